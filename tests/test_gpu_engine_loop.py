"""A miniature serving loop on the GPU that uses the library the way the paper's engine does: the
controller decides one step ahead, a commit is ekv_grow + admit, a decommit is gate -> drain plan ->
ekv_move_blocks -> table rewrite -> drain commit -> ekv_shrink, and attention keeps reading one pointer per
layer throughout.  Every attention result is checked against the oracle on a host mirror that follows the
same writes and moves; moving blocks must not change a single output bit."""
import math

import numpy as np
import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import bf16_bits, cache_view

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MAX_ABS, MEAN_ABS = 2e-2, 2e-3
NL = 2


def check_close(got, want, what):
    err = np.abs(got.float().cpu().numpy().astype(np.float64) - want)
    assert np.isfinite(err).all() and err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (what, err.max(), err.mean())


class Engine:
    def __init__(self):
        self.s = I.LLAMA8B
        s = self.s
        self.pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=128,
                             elastic_blocks=64, num_layers=NL)
        info = self.pool.info
        self.base, self.el = info.base_blocks, info.elastic_blocks
        self.bp = ekv.ekv_blockpool_create(self.base, self.el)
        self.ctrl = ekv.ekv_controller_create(3, 64)
        self.host = [np.full((self.base + self.el) * s.block_elems, 0x7FC0, dtype=np.uint16) for _ in range(NL)]
        for l in range(NL):
            self.pool.layer_tensor(l).view(torch.int16).fill_(0x7FC0)
        self.seqs = {}   # name -> dict(blocks=[...], len=int)
        self.scale = 1 / math.sqrt(s.head_dim)
        self.tick = 0

    def close(self):
        ekv.ekv_blockpool_destroy(self.bp)
        ekv.ekv_controller_destroy(self.ctrl)
        self.pool.close()

    # -- scheduler boundary
    def boundary(self, next_prefill_tokens):
        act = ekv.ekv_controller_decide(self.ctrl, next_prefill_tokens)
        if act == ekv.EKV_ACT_COMMIT:
            self.pool.grow()
            ekv.ekv_blockpool_admit_elastic(self.bp)
        elif act == ekv.EKV_ACT_DECOMMIT:
            in_use = ekv.ekv_blockpool_gate_elastic(self.bp)
            src, dst = ekv.ekv_blockpool_drain_plan(self.bp, self.el)
            assert len(src) == in_use
            if src:
                ekv.ekv_move_blocks(self.pool.handle, torch.tensor(src, dtype=torch.int32, device=DEV),
                                    torch.tensor(dst, dtype=torch.int32, device=DEV))
                remap = dict(zip(src, dst))
                for q in self.seqs.values():
                    q["blocks"] = [remap.get(b, b) for b in q["blocks"]]
                for l in range(NL):                                   # the mirror follows the move
                    v = cache_view(self.host[l], self.s)
                    v[dst] = v[src]
            ekv.ekv_blockpool_drain_commit(self.bp)
            self.pool.shrink()
        assert ekv.ekv_blockpool_stats(self.bp).num_gpu_blocks == self.pool.info.live_blocks
        return act

    # -- requests
    def append(self, name, n_tokens):
        """Allocate blocks for n more tokens of a request and write their K/V in every layer."""
        s = self.s
        q = self.seqs.setdefault(name, {"blocks": [], "len": 0})
        need = (q["len"] + n_tokens + 15) // 16 - len(q["blocks"])
        q["blocks"] += ekv.ekv_blockpool_alloc(self.bp, need)
        row = torch.tensor(q["blocks"], dtype=torch.int32)
        slots = I.position_slots(row, q["len"], n_tokens, 16)
        for l in range(NL):
            self.tick += 1
            n = n_tokens * s.num_kv_heads * s.head_dim
            K = I.normal_bf16(900 + self.tick, 1, 0, n).view(n_tokens, s.num_kv_heads, s.head_dim)
            V = I.normal_bf16(900 + self.tick, 2, 0, n).view(n_tokens, s.num_kv_heads, s.head_dim)
            self.pool.write_kv(l, K.to(DEV), V.to(DEV), slots.to(DEV))
            assert oracle.write_kv(self.host[l], self.pool.info.live_blocks, s.num_kv_heads, 16, s.head_dim, K, V, slots) == 0
        q["len"] += n_tokens

    def finish(self, name):
        ekv.ekv_blockpool_free(self.bp, self.seqs.pop(name)["blocks"])

    def tables(self, names):
        width = max(len(self.seqs[n]["blocks"]) for n in names)
        t = torch.full((len(names), width), -1, dtype=torch.int32)
        for i, n in enumerate(names):
            t[i, :len(self.seqs[n]["blocks"])] = torch.tensor(self.seqs[n]["blocks"], dtype=torch.int32)
        return t, torch.tensor([self.seqs[n]["len"] for n in names], dtype=torch.int32)

    def decode(self, names, layer, check=True):
        s = self.s
        t, lens = self.tables(names)
        q = I.normal_bf16(77, 3, 0, len(names) * s.num_q_heads * s.head_dim).view(len(names), s.num_q_heads, s.head_dim)
        out = self.pool.attn_decode(layer, q.to(DEV), t.to(DEV), lens.to(DEV), self.scale)
        if check:
            want = oracle.attn_decode(self.host[layer], s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q, t, lens, self.scale)
            check_close(out, want, f"decode {names} layer {layer}")
        return out

    def prefill(self, name, c, layer):
        s = self.s
        t, lens = self.tables([name])
        q = I.normal_bf16(78, 3, 0, c * s.num_q_heads * s.head_dim).view(c, s.num_q_heads, s.head_dim)
        cu = torch.tensor([0, c], dtype=torch.int32)
        out = self.pool.attn_prefill_chunk(layer, q.to(DEV), t.to(DEV), cu.to(DEV), cu, lens.to(DEV), self.scale)
        want = oracle.attn_prefill_chunk(self.host[layer], s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q, t, cu, lens, self.scale)
        check_close(out, want, f"prefill {name} layer {layer}")


def test_controller_driven_commit_drain_decommit_cycle():
    e = Engine()
    try:
        bp = e.bp
        for name in ("a", "b", "c"):
            e.append(name, 600)                                        # 38 blocks each, all base
        assert ekv.ekv_blockpool_stats(bp).free_base == e.base - 114
        acts = [e.boundary(0) for _ in range(3)]                       # three decode-only steps ahead
        assert acts == [ekv.EKV_ACT_NONE, ekv.EKV_ACT_NONE, ekv.EKV_ACT_COMMIT]
        assert e.pool.info.grown and ekv.ekv_blockpool_stats(bp).admitted
        e.append("d", 700)                                             # 44 blocks: the last 30 come from the elastic range
        st = ekv.ekv_blockpool_stats(bp)
        assert st.elastic_in_use == 44 - (e.base - 114) and st.free_base == 0
        assert max(e.seqs["d"]["blocks"]) >= e.base                    # peak live block id exceeds the base range ...
        before = [e.decode(["a", "b", "c", "d"], l) for l in range(NL)]   # ... and is served in a single kernel call
        for step in range(4):                                          # a few decode steps while the reserve is lent
            assert e.boundary(0) == ekv.EKV_ACT_NONE
            for n in ("a", "b", "c", "d"):
                e.append(n, 1)
            e.decode(["a", "b", "c", "d"], step % NL)
        e.finish("a")                                                  # a request completes: base blocks come back
        ref = [e.decode(["b", "c", "d"], l) for l in range(NL)]
        assert e.boundary(128) == ekv.EKV_ACT_DECOMMIT                 # the next step carries a 128-token prefill
        st = ekv.ekv_blockpool_stats(bp)
        assert not e.pool.info.grown and st.elastic_in_use == 0 and not st.admitted and not st.draining
        assert max(max(q["blocks"]) for q in e.seqs.values()) < e.base
        after = [e.decode(["b", "c", "d"], l) for l in range(NL)]
        for x, y in zip(ref, after):
            assert torch.equal(x, y), "draining to base blocks changed the output bits"
        e.append("p", 128)                                             # the prefill chunk: write, then attend
        for l in range(NL):
            e.prefill("p", 128, l)
        with pytest.raises(ekv.EkvError) as err:                       # gated: no elastic id, and base is nearly full
            ekv.ekv_blockpool_alloc(bp, 64)
        assert err.value.status == ekv.Status.ERR_OOM
        acts = [e.boundary(0) for _ in range(3)]
        assert acts[-1] == ekv.EKV_ACT_COMMIT and e.pool.info.grown    # and the reserve is lent again
        e.append("f", 300)
        e.decode(["b", "c", "d", "p", "f"], 1)
        torch.cuda.synchronize()
        assert e.pool.poll_status() == ekv.Status.OK
        assert len(before) == NL
    finally:
        e.close()


def test_move_blocks_is_a_bit_exact_copy_in_every_layer_and_guards_the_live_limit():
    s = I.LLAMA8B
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=64,
                    elastic_blocks=32, num_layers=3, start_grown=True)
    try:
        for l in range(3):
            I.fill_pool_layer_(pool.layer_tensor(l), 5, layer=l)
        before = [pool.layer_tensor(l).cpu() for l in range(3)]
        src = torch.tensor([70, 95, 64, 3], dtype=torch.int32, device=DEV)
        dst = torch.tensor([1, 10, 63, 80], dtype=torch.int32, device=DEV)
        ekv.ekv_move_blocks(pool.handle, src, dst)
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        for l in range(3):
            want = before[l].clone()
            want[dst.cpu().long()] = before[l][src.cpu().long()]
            assert torch.equal(pool.layer_tensor(l).cpu(), want)
        pool.shrink(keep_physical=True)
        ekv.ekv_move_blocks(pool.handle, src, dst)                     # ids >= base are no longer live: skipped, latched
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.ERR_BLOCK_OOB
    finally:
        pool.close()
