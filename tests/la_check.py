"""Error metrics shared by the parity tests (numpy, fp64)."""
import numpy as np

TOL_BF16 = 2e-2   # max|err| <= 2e-2 * RMS(ref) for bf16 inputs with fp32 accumulation
TOL_F32 = 1e-4    # the fp32 workload


def head_err(got, ref):
    """Largest max|got-ref| / RMS(ref) over the (b,h) slices, plus the whole-tensor ratio."""
    if hasattr(got, "detach"):
        got = got.detach().double().cpu().numpy()
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    B, H = ref.shape[:2]
    g = got.reshape(B, H, -1)
    r = ref.reshape(B, H, -1)
    assert np.all(np.isfinite(g)), "non-finite values in the GPU result"
    err = np.max(np.abs(g - r), axis=2)
    rms = np.sqrt(np.mean(r * r, axis=2))
    per_head = err / np.maximum(rms, 1e-300)
    whole = np.max(np.abs(g - r)) / max(np.sqrt(np.mean(r * r)), 1e-300)
    return float(per_head.max()), float(whole)


def assert_close(got, ref, tol, what=""):
    per_head, whole = head_err(got, ref)
    assert per_head <= tol, "%s: per-head max|err|/RMS = %.3e > %.1e (whole tensor %.3e)" % (
        what, per_head, tol, whole)
    return per_head
