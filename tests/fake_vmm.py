"""A host-only model of the CUDA VMM calls the pool makes (reserve / create / map / set-access /
unmap / release / free), with the driver's rules enforced and failures injectable.  It is plugged
into libekv through ekv_set_vmm_backend so the pool's state machine runs without a GPU."""
import paper_2608_23658_b200 as ekv

OK, FAIL, OOM = 0, 1, 2


class FakeVmm:
    def __init__(self, granularity=2 << 20, capacity=None):
        self.gran = granularity
        self.capacity = capacity          # bytes of "physical memory", None = unlimited
        self.reserved = {}                # va -> size
        self.handles = {}                 # handle -> size
        self.mapped = {}                  # va -> (size, handle)
        self.access = set()               # va of mappings that were granted access
        self.log = []
        self.fail_create_at = None        # fail the k-th create call from now (0-based)
        self.fail_map_at = None
        self.fail_access_at = None
        self.fail_unmap_at = None
        self._next_va = 0x7000_0000_0000
        self._next_h = 101
        self.violations = []

    # -- helpers
    def used(self):
        return sum(self.handles.values())

    def _bad(self, msg):
        self.violations.append(msg)
        return FAIL

    def _tick(self, attr):
        k = getattr(self, attr)
        if k is None:
            return False
        if k == 0:
            setattr(self, attr, None)
            return True
        setattr(self, attr, k - 1)
        return False

    def _inside_reservation(self, va, size):
        return any(b <= va and va + size <= b + s for b, s in self.reserved.items())

    # -- the table
    def granularity(self, user, device, out):
        out[0] = self.gran
        return OK

    def reserve(self, user, size, align, out):
        if size % self.gran or size == 0:
            return self._bad(f"reserve size {size} not a granule multiple")
        va = self._next_va
        self._next_va += size + (64 << 30)
        self.reserved[va] = size
        out[0] = va
        self.log.append(("reserve", va, size))
        return OK

    def unreserve(self, user, va, size):
        if self.reserved.get(va) != size:
            return self._bad("free of an unknown reservation")
        if any(va <= m < va + size for m in self.mapped):
            return self._bad("free of a range that is still mapped")
        del self.reserved[va]
        self.log.append(("free", va, size))
        return OK

    def create(self, user, size, device, out):
        if size % self.gran or size == 0:
            return self._bad(f"create size {size} not a granule multiple")
        if self._tick("fail_create_at") or (self.capacity is not None and self.used() + size > self.capacity):
            self.log.append(("create-oom", size))
            return OOM
        h = self._next_h
        self._next_h += 1
        self.handles[h] = size
        out[0] = h
        self.log.append(("create", h, size))
        return OK

    def release(self, user, handle):
        if handle not in self.handles:
            return self._bad("release of an unknown handle")
        if any(h == handle for _, h in self.mapped.values()):
            return self._bad("release of a handle that is still mapped")
        del self.handles[handle]
        self.log.append(("release", handle))
        return OK

    def map(self, user, va, size, handle):
        if self.handles.get(handle) != size:
            return self._bad("map size differs from the handle's size (offset must be 0)")
        if not self._inside_reservation(va, size) or va % self.gran:
            return self._bad("map outside a reservation or misaligned")
        if any(m < va + size and va < m + s for m, (s, _) in self.mapped.items()):
            return self._bad("map overlaps an existing mapping")
        if self._tick("fail_map_at"):
            return FAIL
        self.mapped[va] = (size, handle)
        self.log.append(("map", va, size, handle))
        return OK

    def unmap(self, user, va, size):
        if va not in self.mapped or self.mapped[va][0] != size:
            return self._bad("unmap must cover exactly one whole mapping")
        if self._tick("fail_unmap_at"):
            self.log.append(("unmap-refused", va, size))
            return FAIL
        del self.mapped[va]
        self.access.discard(va)
        self.log.append(("unmap", va, size))
        return OK

    def set_access(self, user, va, size, device):
        if va not in self.mapped or self.mapped[va][0] != size:
            return self._bad("set_access on a range that is not one whole mapping")
        if self._tick("fail_access_at"):
            return FAIL
        self.access.add(va)
        return OK

    def table(self):
        return ekv.VmmBackend.from_callables(self.granularity, self.reserve, self.unreserve, self.create,
                                             self.release, self.map, self.unmap, self.set_access)
