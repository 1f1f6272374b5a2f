"""Helpers shared by the GPU parity tests (marshalling and comparators only)."""
import numpy as np

# Tolerances of the layer output against the fp32/fp64 oracle given the oracle's
# mask: max-abs 2e-2 and relative Frobenius 1e-2 for bf16 outputs.
MAX_ABS = 2e-2
REL_FRO = 1e-2
SCORE_BAND = 1e-6  # tokens whose score is this close to the threshold are excluded


def rel_fro(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def bf16_ulp(v):
    """Spacing of bf16 numbers at magnitude |v| (8 significand bits)."""
    v = np.abs(np.asarray(v, np.float64))
    e = np.floor(np.log2(np.maximum(v, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def assert_layer_close(out, ref, strict=True):
    """bf16 layer output against the oracle.  strict: the stated max-abs bound;
    otherwise the bound is widened to one bf16 ulp where |ref| is so large that
    half an ulp alone exceeds it (7B-sized activations beyond |x| >= 8)."""
    out = np.asarray(out, np.float64)
    ref = np.asarray(ref, np.float64)
    err = np.abs(out - ref)
    bound = np.full(ref.shape, MAX_ABS) if strict else np.maximum(MAX_ABS, bf16_ulp(ref))
    worst = float((err - bound).max())
    assert worst <= 0, "max-abs violated by %.4g (max err %.4g)" % (worst, err.max())
    rf = rel_fro(out, ref)
    assert rf <= REL_FRO, "relative Frobenius %.4g" % rf


def assert_selection_matches(idx_gpu, n_gpu, scores_ref, mask_ref, threshold=None):
    """Index sets must agree bit for bit, except tokens whose score lies within
    SCORE_BAND of the threshold."""
    got = np.zeros(mask_ref.shape[0], bool)
    got[np.asarray(idx_gpu[:n_gpu], np.int64)] = True
    assert np.all(np.diff(idx_gpu[:n_gpu]) > 0), "index list must be strictly ascending"
    diff = got != mask_ref.astype(bool)
    if threshold is not None:
        diff &= np.abs(scores_ref.astype(np.float64) - threshold) > SCORE_BAND
    assert not diff.any(), "selection differs at tokens %s" % np.nonzero(diff)[0][:10]


def round_act(a, act_dtype):
    """float32 values rounded to the 16-bit activation format (0 = bf16, 1 = fp16)."""
    a = np.asarray(a, np.float32)
    if act_dtype == 1:
        return a.astype(np.float16).astype(np.float32)
    b = a.view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def act_eps(act_dtype):
    """Half an ulp, relative, of the 16-bit activation format."""
    return 2.0 ** -12 if act_dtype == 1 else 2.0 ** -9
