"""Helper of test_gpu_parity: runs one fixed prefill call with whichever prefill kernel EKV_PREFILL_IMPL selects
(the choice is read once per process), checks it against the oracle and saves the output.  Usage: probe OUT.pt"""
import os
import sys

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path[:0] = [os.path.dirname(HERE), HERE]

import ekv_inputs as I  # noqa: E402
import oracle  # noqa: E402
from test_gpu_parity import DEV, Case, check_close, rand_q  # noqa: E402

shape = I.LLAMA8B
case = Case(shape, [700, 45], 64, 93)
cu = torch.tensor([0, 300, 345], dtype=torch.int32)
q = rand_q(94, 345, shape)
out = case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, 0.088)
want = oracle.attn_prefill_chunk(case.host, 32, 8, 16, 128, q, case.tables, cu, case.lengths, 0.088)
check_close(out, want, os.environ.get("EKV_PREFILL_IMPL", "default") + " prefill kernel")
torch.save(out.cpu(), sys.argv[1])
case.close()
