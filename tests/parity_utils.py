"""Comparison rules shared by the GPU parity tests.

fp32 paths:  |gpu - ref| <= 1e-4 |ref| + 1e-4 rms(ref)   (max relative error 1e-4, with elements near
             zero judged at the tensor's scale).
bf16 paths:  max |LN0(gpu) - LN0(ref)| <= 2e-2, LN0 = parameter-free LayerNorm over the channel axis in
             float64 ("max abs error 2e-2 after LayerNorm").  An output that already is a LayerNorm
             output (the pair broadcast) is compared directly.
Integer outputs are compared bit-exactly by the tests themselves.
"""
import numpy as np

F32_RTOL = 1e-4
BF16_ATOL_AFTER_LN = 2e-2


def ln0(a):
    a = np.asarray(a, dtype=np.float64)
    mu = a.mean(-1, keepdims=True)
    var = ((a - mu) ** 2).mean(-1, keepdims=True)
    return (a - mu) / np.sqrt(var + 1e-12)


def check_f32(gpu, ref, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (what, gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), what
    rms = np.sqrt(np.mean(ref ** 2)) if ref.size else 0.0
    err = np.abs(gpu - ref)
    bound = F32_RTOL * np.abs(ref) + F32_RTOL * rms
    worst = float((err / np.maximum(bound, 1e-300)).max()) if ref.size else 0.0
    assert worst <= 1.0, f"{what}: error is {worst:.3f}x the fp32 bound"
    return worst


def check_bf16(gpu, ref, what="", already_normalised=False):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (what, gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), what
    if not ref.size:
        return 0.0
    err = np.abs(gpu - ref) if already_normalised else np.abs(ln0(gpu) - ln0(ref))
    worst = float(err.max())
    assert worst <= BF16_ATOL_AFTER_LN, f"{what}: max abs error after LN {worst:.4f} > {BF16_ATOL_AFTER_LN}"
    return worst


def check(dtype, gpu, ref, what="", already_normalised=False):
    if dtype == "f32":
        return check_f32(gpu, ref, what)
    return check_bf16(gpu, ref, what, already_normalised)
