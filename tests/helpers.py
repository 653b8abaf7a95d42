"""Shared helpers of the GPU parity tests: device staging and the tolerance checks."""
import numpy as np
import torch

from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200.workloads import pad8

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        _ctx = B.Context(0)
    return _ctx


def to_dev_padded(t: torch.Tensor, ld: int, dtype=torch.bfloat16, fill=float("nan")) -> torch.Tensor:
    """[..., C] fp32 host tensor -> [..., ld] device tensor; pad lanes hold `fill` (they must never be read)."""
    C = t.shape[-1]
    out = torch.full(tuple(t.shape[:-1]) + (ld,), fill, dtype=torch.float32)
    out[..., :C] = t
    return out.to(dtype).cuda()


def out_buffer(shape_no_c, C, ld, f32: bool, canary=7680.0):
    t = torch.full(tuple(shape_no_c) + (ld,), canary, dtype=torch.float32 if f32 else torch.bfloat16, device="cuda")
    return t


def elem_bound(ref: np.ndarray, rms: float, is_bf16: bool) -> np.ndarray:
    """Per-element bound: 1e-2 * rms(ref). Storing a value v as bf16 costs up to half a bf16 ulp,
    2^(floor(log2|v|) - 8), which exceeds 1e-2 * rms for |v| above a few rms whatever the kernel does. So for
    bf16 OUTPUTS the bound of an element is max(1e-2 * rms, half ulp of the reference + 1e-3 * rms of
    accumulation error). fp32 outputs always get the plain bound, and the tests also require the bf16
    output to be the round-to-nearest-even of the fp32 output bit for bit."""
    b = np.full(ref.shape, 1e-2 * rms)
    if is_bf16:
        a = np.abs(ref)
        half_ulp = np.where(a > 0, np.exp2(np.floor(np.log2(np.maximum(a, 1e-300))) - 8.0), 0.0)
        b = np.maximum(b, half_ulp + 1e-3 * rms)
    return b


def check_conv(out_dev: torch.Tensor, C: int, ref: np.ndarray, canary=7680.0, what=""):
    """spec tolerance: relative Frobenius error <= 5e-3 and per-element |err| <= 1e-2 * rms(ref)
    (see elem_bound for bf16 outputs beyond 5 rms); pad lanes must still hold the canary."""
    got = out_dev.float().cpu().numpy().astype(np.float64)
    if got.shape[-1] > C:
        pad = got[..., C:]
        # pad lanes are never read; the TMA-store epilogue may zero those sharing the last 16-byte granule
        assert np.all((pad == canary) | (pad == 0)), what + ": pad lanes hold something other than the canary or zero"
    got = got[..., :C]
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.all(np.isfinite(got)), what + ": non-finite output"
    err = got - ref
    fro = np.linalg.norm(ref.ravel())
    rms = np.sqrt(np.mean(ref.ravel() ** 2))
    rel = np.linalg.norm(err.ravel()) / max(fro, 1e-300)
    mx = np.abs(err).max()
    assert rel <= 5e-3, f"{what}: rel Frobenius {rel:.3e}"
    bound = elem_bound(ref, rms, out_dev.dtype == torch.bfloat16)
    bad = np.abs(err) > bound
    assert not bad.any(), f"{what}: {int(bad.sum())} elements over the bound, worst |err| {mx:.3e} vs 1e-2*rms {1e-2 * rms:.3e}"
    return rel, mx / max(rms, 1e-300)


def check_samples(got: np.ndarray, ref: np.ndarray, rms: float, is_bf16: bool, what=""):
    err = got.astype(np.float64) - ref
    rel = np.linalg.norm(err) / max(np.linalg.norm(ref), 1e-300)
    assert rel <= 5e-3, f"{what}: sampled rel Frobenius {rel:.3e}"
    bad = np.abs(err) > elem_bound(ref, rms, is_bf16)
    assert not bad.any(), f"{what}: {int(bad.sum())} sampled elements over the bound, worst {np.abs(err).max():.3e}, 1e-2*rms {1e-2 * rms:.3e}"


def check_update(got: torch.Tensor, ref: np.ndarray, what=""):
    """fp32 update tolerance: relative Frobenius error <= 1e-5 and |err| <= 1e-5 * max(|ref|, rms(ref)) per element."""
    g = got.detach().float().cpu().numpy().astype(np.float64)
    err = g - ref
    fro = np.linalg.norm(ref.ravel())
    if fro == 0:
        assert np.all(g == 0), what
        return
    rms = np.sqrt(np.mean(ref.ravel() ** 2))
    assert np.linalg.norm(err.ravel()) / fro <= 1e-5, f"{what}: rel {np.linalg.norm(err.ravel()) / fro:.3e}"
    bound = 1e-5 * np.maximum(np.abs(ref), rms)
    assert np.all(np.abs(err) <= bound), f"{what}: max ratio {(np.abs(err) / bound).max():.3f}"


def conv_ws(desc, which):
    n = B.pt_conv_workspace_bytes(ctx(), desc, which)
    return torch.empty(max(n, 16), dtype=torch.uint8, device="cuda") if n else None


def run_conv_all(N, H, W, C, K, R, stride, pad, x, w, dy, algo=0, out_f32=0):
    """Runs fwd, dgrad, wgrad through the C ABI on padded device copies; returns device outputs + desc."""
    ldx, ldy, ldw = pad8(C), pad8(K), pad8(C)
    d = B.make_conv_desc(N, H, W, C, K, R, R, stride, pad, ldx, ldy, ldw, out_f32, algo)
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - R) // stride + 1
    xd, wd, dyd = to_dev_padded(x, ldx), to_dev_padded(w, ldw), to_dev_padded(dy, ldy)
    y = out_buffer((N, P, Q), K, ldy, out_f32)
    dx = out_buffer((N, H, W), C, ldx, out_f32)
    dw = torch.full((K, R, R, C), 7680.0, dtype=torch.float32, device="cuda")
    B.pt_conv_fwd(ctx(), d, xd, wd, y, conv_ws(d, B.PT_CONV_FWD))
    B.pt_conv_dgrad(ctx(), d, dyd, wd, dx, conv_ws(d, B.PT_CONV_DGRAD))
    B.pt_conv_wgrad(ctx(), d, xd, dyd, dw, conv_ws(d, B.PT_CONV_WGRAD))
    torch.cuda.synchronize()
    ctx().poll()
    return y, dx, dw, d
