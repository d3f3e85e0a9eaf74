"""Plain model of the gated block pool and the one-step-ahead controller -- TEST INFRASTRUCTURE ONLY.

Written from the paper's description (section "An Elastic KV Mechanism"):
  * the block pool is an integer free list with no runtime allocation (section "Background and
    Motivation", "KV allocation in vLLM");
  * the top elastic block-id range is gated: those ids are only handed out while the elastic slice is
    committed ("Two handles, one virtual range");
  * committing grows num_gpu_blocks and admits the top ids; decommitting first drains them
    ("Controller");
  * the controller commits during decode-only phases and decommits at the boundary before a prefill,
    with hysteresis ("Controller").
Readings this build adds (the paper gives no detail): base ids are preferred over elastic ids; free
lists are stacks whose initial order hands out ascending ids; hysteresis = a number of consecutive
quiet steps before a commit; a step is "a prefill that needs the reserve" when its prefill tokens
reach a threshold; a decommit is decided immediately.

Everything is lists and sets; no code is shared with the C++ implementation.
"""


class BlockPoolModel:
    def __init__(self, base, elastic):
        self.base, self.elastic = base, elastic
        self.free_base = list(range(base - 1, -1, -1))            # pop() hands out the lowest id first
        self.free_elastic = list(range(base + elastic - 1, base - 1, -1))
        self.used = set()
        self.admitted = False
        self.plan = None

    def alloc(self, n):
        avail = len(self.free_base) + (len(self.free_elastic) if self.admitted else 0)
        if n > avail:
            return None                                            # all or nothing
        out = []
        for _ in range(n):
            out.append(self.free_base.pop() if self.free_base else self.free_elastic.pop())
        self.used.update(out)
        return out

    def free(self, ids):
        """True / False (nothing freed) / "state" (an id of the outstanding drain plan: nothing freed)."""
        if len(set(ids)) != len(ids) or any(i not in self.used for i in ids):
            return False
        if self.plan and any(i in self.plan[0] or i in self.plan[1] for i in ids):
            return "state"
        for i in ids:
            self.used.discard(i)
            (self.free_base if i < self.base else self.free_elastic).append(i)
        return True

    def elastic_in_use(self):
        return sorted(i for i in self.used if i >= self.base)

    def admit(self):
        if self.plan:
            return False
        self.admitted = True
        return True

    def gate(self):
        self.admitted = False
        return len(self.elastic_in_use())

    def drain_plan(self):
        """Returns 'state' / 'oom' / (from_ids, to_ids)."""
        if self.admitted or self.plan:
            return "state"
        src = self.elastic_in_use()
        if len(src) > len(self.free_base):
            return "oom"
        dst = [self.free_base.pop() for _ in src]
        self.used.update(dst)
        self.plan = (src, dst)
        return src, dst

    def drain_commit(self):
        if self.plan:
            for i in self.plan[0]:
                self.used.discard(i)
                self.free_elastic.append(i)
        self.plan = None

    def num_gpu_blocks(self):
        return self.base + (self.elastic if self.admitted else 0)


class ControllerModel:
    NONE, COMMIT, DECOMMIT = 0, 1, 2

    def __init__(self, commit_after_decode_steps, reserve_prefill_tokens, committed=False):
        self.n, self.thr, self.committed, self.streak = commit_after_decode_steps, reserve_prefill_tokens, committed, 0

    def decide(self, next_prefill_tokens):
        if next_prefill_tokens >= self.thr:                        # the next step needs the reserve back
            self.streak = 0
            if self.committed:
                self.committed = False
                return self.DECOMMIT
            return self.NONE
        self.streak += 1
        if not self.committed and self.streak >= self.n:
            self.committed = True
            return self.COMMIT
        return self.NONE
