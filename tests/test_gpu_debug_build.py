"""The checking build of the library (-DGCNSA_DEBUG): the same scenario runs
once on the regular library (this process) and once on libgcnsa_debug.so (a
child process, because a process loads one build), and must give bit-identical
results with no check recorded.  The scenario: the tiny workload trained in
the plain and in the measured configuration, and partition builds of random
graphs under every assignment mode."""
import hashlib
import json
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

pytestmark = pytest.mark.gpu


def _digest(arrays):
    h = hashlib.sha256()
    for a in arrays:
        h.update(np.ascontiguousarray(a).tobytes())
    return h.hexdigest()


def scenario():
    import torch
    from gen import configs, graphs
    from paper_2012_04930_b200 import gcnsa
    out = {}
    w = configs.tiny()
    side = torch.cuda.Stream()
    for name, opts, stream in (("plain", gcnsa.PLAIN, torch.cuda.current_stream()), ("measured", gcnsa.MEASURED, side)):
        with torch.cuda.stream(stream):
            env = gcnsa.make_env(0)
            parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                                w.part_mode, w.user_part, w.loss_on_halo)
            model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, **opts)
            loss = torch.zeros(1, device="cuda")
            losses = []
            for _ in range(3):
                model.epoch(loss.data_ptr())
                stream.synchronize()
                losses.append(float(loss.item()))
            out[name] = {"losses": losses,
                         "params": _digest([model.get(what, l) for what in (gcnsa.GET_W, gcnsa.GET_B) for l in range(2)])}
            correct, total, pred = model.evaluate(parts, 1)
            out[name]["eval"] = [correct, total, _digest([pred])]
            model.close(); parts.close()
    rng = np.random.default_rng(11)
    builds = []
    for n, prob, m, o_ppm, mode in ((300, 0.03, 3, 300_000, gcnsa.PART_HASH), (900, 0.01, 5, 100_000, gcnsa.PART_RANGE),
                                    (64, 0.2, 2, 1_000_000, gcnsa.PART_USER), (500, 0.004, 4, 500_000, gcnsa.PART_HASH)):
        rowptr, col = graphs.erdos_renyi(n, prob, n)
        x = rng.standard_normal((n, 5)).astype(np.float32)
        y = rng.integers(0, 3, n).astype(np.int32)
        mask = (rng.random(n) < 0.5).astype(np.uint8)
        user = (np.arange(n) % m).astype(np.int32) if mode == gcnsa.PART_USER else None
        parts = gcnsa.Parts(gcnsa.make_env(0), rowptr, col, x, y, mask, 3, m, o_ppm, 17, mode, user, 1)
        arrays = [parts.assignment()]
        for p in range(m):
            e, sc = parts.export(p), parts.export_schedule(p)
            arrays += [e[k] for k in sorted(e)] + [sc[k] for k in sorted(sc) if isinstance(sc[k], np.ndarray)]
        builds.append(_digest(arrays))
        parts.close()
    out["builds"] = builds
    out["debug_status"] = list(gcnsa.debug_status())
    out["tc_status"] = gcnsa.tc_status()
    return out


def test_checking_build_gives_identical_results_and_records_nothing():
    from paper_2012_04930_b200 import build
    build.build()
    lib_debug = build.build(debug=True)
    child = subprocess.run([sys.executable, os.path.abspath(__file__), "--child", lib_debug], capture_output=True, text=True,
                           timeout=900)
    assert child.returncode == 0, child.stderr[-2000:]
    got = json.loads(child.stdout.strip().splitlines()[-1])
    want = scenario()
    assert got["debug_status"] == [True, 0, 0], "the checking build recorded a violation (code, value)"
    assert want["debug_status"] == [False, 0, 0]
    for key in ("plain", "measured", "builds", "tc_status"):
        assert got[key] == want[key], key


if __name__ == "__main__":
    if len(sys.argv) == 3 and sys.argv[1] == "--child":
        from paper_2012_04930_b200 import gcnsa
        gcnsa.use_library(sys.argv[2])
        print(json.dumps(scenario()))
