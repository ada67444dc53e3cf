"""Helpers shared by the GPU parity suites (no method arithmetic)."""
import numpy as np

TOL = 1e-4   # fp32 tensors: max |got - want| <= TOL * max |want|


def close(got, want, tol=TOL, what=""):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if want.size == 0:
        return
    scale = max(np.abs(want).max(), 1e-30)
    err = np.abs(got - want).max()
    assert err <= tol * scale, f"{what}: max err {err:.3e} vs scale {scale:.3e}"


def ambiguous_units(zs, rel=1e-5):
    """Per hidden layer, the units whose pre-activation is so close to zero
    (|z| < rel * max|z| of the layer, the checker's own fp64 values) that its
    sign is not determined in fp32.  Nothing of the kernel enters here."""
    return [np.abs(z) < rel * np.abs(z).max() for z in zs]


def relu_decisions(fw, h_gpu):
    """ReLU on / off per hidden unit for the checker's backward pass
    (ReLU'(z) = [z > 0]): the checker's own sign of z everywhere except on
    ambiguous_units(), where the kernel's decision is taken after checking that
    the kernel's value is equally tiny.  Away from zero both sides must agree,
    and the ambiguous units must be at most 1e-3 of all hidden units."""
    zs = fw["Z"][:-1]
    assert len(h_gpu) == len(zs)
    amb = ambiguous_units(zs)
    out, n_amb = [], 0
    for z, h, a in zip(zs, h_gpu, amb):
        assert np.all(np.abs(h[a]) < 2e-5 * np.abs(z).max())
        assert np.array_equal((h > 0)[~a], (z > 0)[~a]), "ReLU decisions differ away from zero"
        out.append(np.where(a, h > 0, z > 0))
        n_amb += int(a.sum())
    assert n_amb <= 1e-3 * sum(z.size for z in zs) + 2
    return out
