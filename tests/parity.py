"""Comparison rules shared by the GPU parity tests (all arithmetic in float64).

rel_fro = ||X - X_ref||_F / ||X_ref||_F          <= 5e-3
max_abs = max|X - X_ref| / s                      <= 3e-2   (s makes the output unit scale:
          rms(C_ref) for GEMM, 1 for attention outputs, which are convex combinations of N(0,1) values)
max|LSE - LSE_ref|                                <= 1e-3
"""
import numpy as np

REL_FRO_TOL = 5e-3
MAX_ABS_TOL = 3e-2
LSE_TOL = 1e-3


def errors(x: np.ndarray, ref: np.ndarray, unit: float | None = None):
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert x.shape == ref.shape, (x.shape, ref.shape)
    assert np.isfinite(x).all(), "non-finite output"
    diff = x - ref
    nref = np.linalg.norm(ref)
    rel = np.linalg.norm(diff) / nref if nref > 0 else np.linalg.norm(diff)
    if unit is None:
        unit = 1.0
    mx = np.abs(diff).max() / unit if diff.size else 0.0
    return rel, mx


def check_gemm(c: np.ndarray, ref: np.ndarray, what=""):
    rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 1.0
    rel, mx = errors(c, ref, unit=rms if rms > 0 else 1.0)
    assert rel <= REL_FRO_TOL, f"{what}: rel_fro {rel:.3e}"
    assert mx <= MAX_ABS_TOL, f"{what}: max_abs/rms {mx:.3e}"
    return rel, mx


def check_mha(o, lse, o_ref, lse_ref, what="", unit=1.0):
    rel, mx = errors(o, o_ref, unit=unit)
    assert rel <= REL_FRO_TOL, f"{what}: O rel_fro {rel:.3e}"
    assert mx <= MAX_ABS_TOL, f"{what}: O max_abs {mx:.3e}"
    dl = float(np.abs(np.asarray(lse, np.float64) - lse_ref).max()) if lse_ref.size else 0.0
    assert np.isfinite(np.asarray(lse)).all()
    assert dl <= LSE_TOL, f"{what}: LSE max_abs {dl:.3e}"
    return rel, mx, dl


def log_line(text: str) -> None:
    """Appends one line to the parity log of this run (full-output comparisons are recorded there): the file named
    by MLT_PARITY_LOG, else parity_full_configs.log in the repository's untracked output folder.  Never fails a test."""
    import os
    path = os.environ.get("MLT_PARITY_LOG")
    if not path:
        root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
        path = os.path.join(root, "gpurun_out", "parity_full_configs.log")
    try:
        os.makedirs(os.path.dirname(path), exist_ok=True)
        with open(path, "a") as f:
            f.write(text.rstrip("\n") + "\n")
    except OSError:
        pass


class RunningErrors:
    """rel_fro / max_abs accumulated over chunks of rows, for outputs too large to hold twice in float64."""

    def __init__(self):
        self.d2 = self.r2 = 0.0
        self.max_abs = 0.0
        self.n = 0

    def add(self, x, ref):
        import numpy as np
        x = np.asarray(x, dtype=np.float64)
        ref = np.asarray(ref, dtype=np.float64)
        assert x.shape == ref.shape, (x.shape, ref.shape)
        assert np.isfinite(x).all(), "non-finite output"
        diff = x - ref
        self.d2 += float(np.sum(diff * diff))
        self.r2 += float(np.sum(ref * ref))
        if diff.size:
            self.max_abs = max(self.max_abs, float(np.abs(diff).max()))
        self.n += diff.size

    def rel_fro(self):
        return (self.d2 / self.r2) ** 0.5 if self.r2 > 0 else self.d2 ** 0.5

    def rms_ref(self):
        return (self.r2 / self.n) ** 0.5 if self.n else 1.0
