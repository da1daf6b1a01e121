"""Helpers of the GPU parity tests: the two error measures and guarded device buffers.

Error measures, both against the fp64 oracle b:
  * rel-L2 = ||a - b|| / ||b|| over the whole tensor (the stated tolerances: 1e-5 merged weights,
    1e-4 fp32 outputs, 2e-2 bf16 outputs);
  * an element-wise bound |a - b| <= rtol * |b| + atol * rms(b), which a localised fault (one wrong
    pixel, a dropped tap on a tile seam, a stale row) cannot hide under.

bf16 bound: the oracle and the GPU read the same bf16-rounded input, so an output element errs by
(i) the bf16 rounding of the merged weights, sum_i w_i eps_i x_i with |eps_i| <= 2^-9, whose standard
deviation is about 2^-9 / sqrt(3) * rms(b) = 1.1e-3 rms(b) whatever the reduction length, (ii) fp32
accumulation (negligible) and (iii) the rounding of the output itself, <= 2^-9 |b|.  Measured
rel-L2 is 2-3e-3, i.e. sigma ~ 2.5e-3 rms(b).  rtol = 2^-7 and atol = 2^-5 (12 sigma; the largest
tensor here has 1.3e7 elements, whose extreme is ~5.5 sigma) leave room for rounding only: any
error above 4 % of the tensor's rms at a single element fails.  `scale` multiplies both terms for
paths that round intermediate maps as well (an unmerged block: 3; the whole network: stated there).
fp32 bound: rtol = atol = 1e-4 (fp32 FMA accumulation errs by ~1e-6 rms(b)).
"""
import numpy as np

RTOL_BF16, ATOL_BF16 = 2.0 ** -7, 2.0 ** -5
RTOL_F32, ATOL_F32 = 1e-4, 1e-4


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = float(np.sqrt(np.sum(b * b)))
    return float(np.sqrt(np.sum((a - b) ** 2))) / (den if den > 0 else 1.0)


def elementwise_excess(a, b, bf16=True, scale=1.0):
    """(worst ratio of |a-b| to its bound, index of that element, max abs error)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    rtol, atol = (RTOL_BF16, ATOL_BF16) if bf16 else (RTOL_F32, ATOL_F32)
    rms = float(np.sqrt(np.mean(b * b))) if b.size else 0.0
    err = np.abs(a - b)
    bound = scale * (rtol * np.abs(b) + atol * rms) + 1e-30
    ratio = err / bound
    if ratio.size == 0:
        return 0.0, (), 0.0
    idx = np.unravel_index(int(np.argmax(np.where(np.isnan(ratio), np.inf, ratio))), ratio.shape)
    worst = float(ratio[idx])
    return (np.inf if np.isnan(worst) else worst), idx, float(np.nanmax(err))


def assert_close(a, b, tol, bf16=True, scale=1.0, what=""):
    """Both measures; on failure names the worst element (NCHW index for feature maps)."""
    assert tuple(np.shape(a)) == tuple(np.shape(b)), (what, np.shape(a), np.shape(b))
    r = rel_l2(a, b)
    worst, idx, max_abs = elementwise_excess(a, b, bf16=bf16, scale=scale)
    assert r <= tol, "%s: rel-L2 %.3e > %.1e (max abs error %.3e at %s)" % (what, r, tol, max_abs, idx)
    assert worst <= 1.0, ("%s: element %s is off by %.2f x its bound: got %r, oracle %r (rel-L2 %.3e, max abs %.3e)"
                          % (what, idx, worst, float(np.asarray(a)[idx]), float(np.asarray(b)[idx]), r, max_abs))
    return r, worst, max_abs


class Guarded:
    """A device tensor in the middle of a larger allocation whose two flanks hold a sentinel
    pattern: a kernel that writes outside the tensor it was given changes a flank.  Stands in for a
    memory checker on the buffers the library writes (outputs, merged weights, packed copies,
    workspaces)."""
    GUARD = 64 * 1024            # bytes on each side
    SENTINEL = 0xA5

    def __init__(self, torch, shape, dtype, fill=None):
        self.torch = torch
        esize = torch.empty((), dtype=dtype).element_size()
        n = 1
        for d in shape:
            n *= int(d)
        nbytes = ((n * esize + 255) // 256) * 256
        self.raw = torch.full((2 * self.GUARD + nbytes,), self.SENTINEL, dtype=torch.uint8, device="cuda")
        self.nbytes = n * esize
        body = self.raw[self.GUARD:self.GUARD + n * esize]
        self.t = body.view(dtype).view(*shape) if n else torch.empty(shape, dtype=dtype, device="cuda")
        if fill is not None and n:
            self.t.fill_(fill)

    def check(self, what=""):
        front = self.raw[:self.GUARD]
        back = self.raw[self.GUARD + self.nbytes:]
        for name, band in (("before", front), ("after", back)):
            bad = (band != self.SENTINEL).nonzero()
            assert bad.numel() == 0, "%s: %d bytes written %s the buffer (first at offset %d of the band)" % (
                what, bad.numel(), name, int(bad[0]))
