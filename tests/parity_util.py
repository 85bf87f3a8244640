"""Helpers shared by the GPU parity tests: tolerances, error metrics, device upload."""
import numpy as np

# Tolerances of the bf16 tensor-core path (bf16 inputs, fp32 accumulation) and of the
# fp32 debug path, per output tensor over the whole [B, H, N, D].
BF16_MAX_ABS = 2e-2
BF16_REL_FRO = 5e-3
FP32_REL = 1e-5


def rel_fro(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    num = np.linalg.norm((got - ref).ravel())
    return num / den if den > 0 else num


def max_abs(got, ref):
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - np.asarray(ref, dtype=np.float64))))


def assert_bf16_close(got, ref, name):
    got = np.asarray(got, dtype=np.float64)
    assert np.all(np.isfinite(got)), f"{name}: non-finite values"
    ma, rf = max_abs(got, ref), rel_fro(got, ref)
    assert ma <= BF16_MAX_ABS, f"{name}: max-abs {ma:.3e} > {BF16_MAX_ABS}"
    assert rf <= BF16_REL_FRO, f"{name}: rel-Frobenius {rf:.3e} > {BF16_REL_FRO}"
    # no single head may hide behind the others
    B, H = got.shape[:2]
    for b in range(B):
        for h in range(H):
            r = rel_fro(got[b, h], ref[b, h])
            assert r <= 2 * BF16_REL_FRO, f"{name}[{b},{h}]: per-head rel-Frobenius {r:.3e}"
    return ma, rf


def assert_fp32_close(got, ref, name):
    got = np.asarray(got, dtype=np.float64)
    assert np.all(np.isfinite(got)), f"{name}: non-finite values"
    rf = rel_fro(got, ref)
    ma = max_abs(got, ref)
    assert rf <= FP32_REL, f"{name}: rel-Frobenius {rf:.3e} > {FP32_REL}"
    assert ma <= FP32_REL * float(np.max(np.abs(ref))) + 1e-30, f"{name}: max-abs {ma:.3e}"
    return ma, rf


def to_device(x_f32, dtype):
    """float32 numpy array (already holding bf16-representable values for bf16) -> CUDA tensor."""
    import torch
    from paper_2409_04431_b200 import inputs
    if dtype == "bf16":
        bits = inputs.f32_to_bf16_bits(x_f32)
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()
    return torch.from_numpy(np.ascontiguousarray(x_f32, dtype=np.float32)).cuda()


def to_host(t):
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)
