"""Failures made on the host, handled on the GPU machine: an allocator callback
that returns NULL on its k-th call (a simulated out-of-memory condition) for
every k until the call succeeds.  Each failing call must report GCNSA_ERR_OOM,
hand back everything it was given (the callback counts), and leave the context
usable for the next call.  Nothing here faults, traps or hangs the GPU."""
import ctypes as C

import numpy as np
import pytest
import torch

from gen import configs
from paper_2012_04930_b200 import gcnsa

pytestmark = pytest.mark.gpu


class FailingAllocator:
    """gcnsa_env callbacks on top of torch's caching allocator; call number `fail_at` (1-based) returns NULL."""

    def __init__(self):
        self.calls, self.fail_at, self.live = 0, 0, {}
        self.alloc_cb = gcnsa.ALLOC_FN(self._alloc)
        self.free_cb = gcnsa.FREE_FN(self._free)

    def arm(self, fail_at):
        self.calls, self.fail_at = 0, fail_at

    def _alloc(self, nbytes, user):
        self.calls += 1
        if self.calls == self.fail_at:
            return None
        p = torch.cuda.caching_allocator_alloc(int(nbytes), stream=torch.cuda.current_stream())
        self.live[p] = int(nbytes)
        return p

    def _free(self, ptr, user):
        assert ptr in self.live, "free of a pointer the allocator never handed out (or a second free)"
        del self.live[ptr]
        torch.cuda.caching_allocator_delete(ptr)

    def env(self):
        e = gcnsa.make_env(0)
        e.alloc, e.free = self.alloc_cb, self.free_cb
        return e


def _until_success(alloc, call, keeps=False, limit=400):
    """Runs call() with the k-th allocation failing for k = 1, 2, ...; returns (k of the first success, result).
    keeps: the object under test may keep what a failed call had already obtained (buffers made on first use)."""
    for k in range(1, limit):
        alloc.arm(k)
        live_before = set(alloc.live)
        try:
            out = call()
        except gcnsa.GcnsaError as e:
            assert e.code == gcnsa.ERR_OOM, (k, e)
            assert alloc.calls >= k
            torch.cuda.synchronize()
            if not keeps:
                leaked = set(alloc.live) - live_before
                assert not leaked, f"allocation {k} failed and {len(leaked)} buffers were not handed back"
            continue
        assert alloc.calls < k, "the call succeeded although one of its allocations was refused"
        return k, out
    raise AssertionError("no success within the limit")


@pytest.mark.parametrize("builder", [gcnsa.BUILD_DEVICE, gcnsa.BUILD_HOST])
def test_out_of_memory_while_building_partitions(builder, tiny_wl):
    w = tiny_wl
    alloc = FailingAllocator()
    env = alloc.env()

    def build():
        return gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                           w.part_mode, w.user_part, w.loss_on_halo, builder=builder)

    k, parts = _until_success(alloc, build)
    assert k > 10, "the build makes many allocations: each of them was made to fail once"
    alloc.arm(0)
    # the object built right after the failures is a good one: same structure as a build with torch's allocator
    good = gcnsa.Parts(gcnsa.make_env(0), w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                       w.part_mode, w.user_part, w.loss_on_halo, builder=builder)
    for p in range(w.m):
        a, b = parts.export(p), good.export(p)
        for key in a:
            assert np.array_equal(a[key], b[key]), key
    good.close()
    parts.close()
    torch.cuda.synchronize()
    assert not alloc.live, "destroy releases every buffer"


@pytest.mark.parametrize("agg_mode,cache_ax", [(gcnsa.AGG_GRAD_AVG, 0), (gcnsa.AGG_PARAM_AVG, 1)])
def test_out_of_memory_while_creating_and_using_a_model(agg_mode, cache_ax, tiny_wl):
    w = tiny_wl
    alloc = FailingAllocator()
    env = alloc.env()
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    held = set(alloc.live)

    def create():
        return gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, agg_mode=agg_mode, cache_ax=cache_ax,
                           **{**gcnsa.MEASURED, "epoch_graph": 0})

    k, model = _until_success(alloc, create)
    assert k > 10
    alloc.arm(0)
    loss = torch.zeros(1, device="cuda")
    model.epoch(loss.data_ptr())
    first = loss.item()
    assert np.isfinite(first)
    # the buffers evaluation and the host-buffer epoch allocate on first use: a failure there is an error code, and
    # the call works when it is made again
    k_ev, (correct, total, _) = _until_success(alloc, lambda: model.evaluate(parts, 0), keeps=True)
    assert k_ev >= 2 and 0 <= correct <= total == parts.info(0).n
    xs = [np.ascontiguousarray(w.x[parts.members(p)]) for p in range(w.m)]
    loss_h = np.zeros(1, np.float32)
    k_eh, _ = _until_success(alloc, lambda: model.epoch_host([x.ctypes.data for x in xs], loss_h), keeps=True)
    assert k_eh >= 2 and np.isfinite(loss_h[0]) and loss_h[0] <= first
    alloc.arm(0)
    model.close()
    torch.cuda.synchronize()
    assert held <= set(alloc.live) and len(set(alloc.live) - held) <= 2   # the partitions and their two staging buffers
    parts.close()
    torch.cuda.synchronize()
    assert not alloc.live
