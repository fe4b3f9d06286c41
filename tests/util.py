"""Shared helpers for the GPU parity tests (marshalling and error metrics only)."""
import numpy as np

REL_F_TOL = 5e-3      # relative Frobenius error bound stated for this path
MAX_ABS_TOL = 3e-2    # max elementwise abs error bound; applied to |gpu-oracle| / max(1, rms(oracle))
                      # for bf16 outputs (a correctly rounded bf16 value above 8 is already off by
                      # more than 3e-2), and literally for fp32 outputs of unit scale


def to_dev(bits_or_f32):
    """numpy uint16 (bf16 bit patterns) -> cuda bf16 tensor; numpy float32 -> cuda fp32 tensor."""
    import torch
    a = np.ascontiguousarray(bits_or_f32)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def to_f64(t):
    """cuda tensor (bf16 or fp32) -> numpy fp64, exact widening."""
    return t.detach().double().cpu().numpy()


def errors(gpu, ref):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), "non-finite values (unwritten output?)"
    d = np.abs(gpu - ref)
    relf = float(np.linalg.norm(d) / max(np.linalg.norm(ref), 1e-30))
    rms = float(np.sqrt(np.mean(ref * ref)))
    return relf, float(d.max()), float(d.max() / max(1.0, rms))


def assert_close(gpu, ref, name="", relf_tol=REL_F_TOL, abs_tol=MAX_ABS_TOL):
    relf, maxabs, maxabs_norm = errors(gpu, ref)
    assert relf <= relf_tol, "%s: rel Frobenius %.3e > %.1e" % (name, relf, relf_tol)
    assert maxabs_norm <= abs_tol, "%s: max abs (scale-normalised) %.3e > %.1e (raw %.3e)" % (
        name, maxabs_norm, abs_tol, maxabs)
    return relf, maxabs


class Guarded:
    """A device buffer with canary bands before and after the payload, NaN-prefilled payload."""

    def __init__(self, shape, dtype, band=1024):
        import torch
        self.n = int(np.prod(shape))
        self.band = band
        self.shape = shape
        self.raw = torch.empty(self.n + 2 * band, dtype=dtype, device="cuda")
        self.raw.fill_(1234.5)
        self.t = self.raw[band:band + self.n].view(*shape)
        self.t.fill_(float("nan"))

    def check(self):
        assert bool((self.raw[:self.band] == 1234.5).all()), "write before the buffer"
        assert bool((self.raw[self.band + self.n:] == 1234.5).all()), "write past the buffer"
