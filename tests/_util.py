"""Shared helpers of the GPU parity tests (argument marshalling and error metrics only)."""
import numpy as np

# tolerances of the build target, relative to RMS(oracle out)
TOL = {"f32": dict(max=1e-4, mean=None), "bf16": dict(max=2e-2, mean=2e-3), "bf16_f32out": dict(max=2e-4, mean=None)}


def to_dev(a, dev="cuda:0"):
    import torch
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
    return torch.from_numpy(a).to(dev)


def bits(t):
    """Device tensor -> host array in the oracle's storage convention."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def as_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def metrics(got64, ref64):
    """max abs, mean abs, RMSE (all relative to RMS(ref)), cosine, non-finite count."""
    rms = float(np.sqrt(np.mean(ref64 ** 2)))
    rms = rms if rms > 0 else 1.0
    err = np.abs(got64 - ref64)
    g, r = got64.ravel(), ref64.ravel()
    den = float(np.linalg.norm(g) * np.linalg.norm(r))
    return dict(max=float(err.max()) / rms, mean=float(err.mean()) / rms,
                rmse=float(np.sqrt(np.mean(err ** 2))) / rms,
                cos=float(np.dot(g, r) / den) if den > 0 else 1.0,
                nonfinite=int(np.count_nonzero(~np.isfinite(got64))), rms=rms)


def check(got64, ref64, kind):
    m = metrics(got64, ref64)
    tol = TOL[kind]
    assert m["nonfinite"] == 0, m
    assert m["max"] <= tol["max"], (kind, m)
    if tol["mean"] is not None:
        assert m["mean"] <= tol["mean"], (kind, m)
    return m
