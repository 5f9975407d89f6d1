"""Shared helpers of the GPU parity tests: move seeded inputs to the device, call the C ABI through
the binding, run the oracle on the same host buffers, and apply the stated tolerances."""
import numpy as np
import torch

from paper_2501_13629_b200 import workloads as W


def device_cache(api, inp, device="cuda", unused_page=0):
    """KVCache on the device for a workloads.DecodeInputs (same bytes as the host buffers)."""
    k, v = W.to_torch(inp.k, device), W.to_torch(inp.v, device)
    seqlens = torch.from_numpy(inp.seqlens).to(device)
    pt = None
    if inp.page_table is not None:
        pt = torch.from_numpy(inp.page_table).to(device)
    return api.KVCache(k, v, seqlens, int(inp.max_seqlen), page_table=pt, page_size=inp.cfg.page_size,
                       k_strides=inp.k_strides, v_strides=inp.v_strides,
                       num_blocks=inp.num_pages if pt is not None else inp.cfg.batch)


def oracle_cache(oracle, inp):
    return oracle.Cache(inp.k, inp.v, inp.k_strides, inp.v_strides, inp.seqlens, inp.page_table,
                        inp.cfg.page_size)


def run_decode(api, inp, num_splits=0, out_dtype=torch.float32, gqa=False, want_lse=True):
    cfg = inp.cfg
    dev = "cuda"
    q = W.to_torch(inp.q, dev)
    cache = device_cache(api, inp, dev)
    lse = torch.full((cfg.batch, cfg.n_q), float("nan"), dtype=torch.float32, device=dev) if want_lse else None
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if gqa:
        out = api.gqa_decode(q, cache, cfg.n_k, cfg.scale, num_splits=num_splits, lse=lse, dev_status=status,
                             out_dtype=out_dtype)
    else:
        out = api.diffqkv_decode(q, cache, cfg.n_k, cfg.n_v, cfg.scale, num_splits=num_splits, lse=lse,
                                 dev_status=status, out_dtype=out_dtype)
    torch.cuda.synchronize()
    return (out.float().cpu().numpy().astype(np.float64),
            None if lse is None else lse.cpu().numpy().astype(np.float64), int(status.item()))


def run_oracle(oracle, inp, pairs=None):
    cfg = inp.cfg
    return oracle.decode(inp.q, oracle_cache(oracle, inp), cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v,
                         cfg.scale, pairs=pairs)


def check_bf16(out, ref, what=""):
    """bf16 cache, fp32 accumulation: max |err| <= 2e-2 absolute and <= 1e-2 of max |ref|,
    and element-wise |err| <= 2e-2 + 1e-2 |ref|."""
    err = np.abs(out - ref)
    scale = max(np.abs(ref).max(), 1e-30)
    assert err.max() <= 2e-2, f"{what}: max abs err {err.max():.3e}"
    assert err.max() / scale <= 1e-2, f"{what}: max err / max|ref| {err.max() / scale:.3e}"
    assert np.all(err <= 2e-2 + 1e-2 * np.abs(ref)), what
    return float(err.max())


def check_f32(out, ref, what=""):
    """fp32 mode: max |err| / max |ref| <= 1e-5."""
    err = np.abs(out - ref).max()
    scale = max(np.abs(ref).max(), 1e-30)
    assert err / scale <= 1e-5, f"{what}: max err / max|ref| {err / scale:.3e}"
    return float(err / scale)


def check_lse(lse, ref, tol, what=""):
    both_inf = np.isneginf(lse) & np.isneginf(ref)
    with np.errstate(invalid="ignore"):
        d = np.where(both_inf, 0.0, np.abs(lse - ref))
    assert np.all(np.isfinite(d)) and d.max() <= tol, f"{what}: lse err {d.max()}"


def check_proj(out, ref, what="", c_abs=2e-2):
    """Projection chains (bf16 operands and result, fp32 accumulation; the oracle rounds nothing).

    Three checks: max |err| <= 1e-2 max |ref|; rms(err) <= 4e-3 rms(ref); and element-wise
    |err| <= 2^-8 |ref| + c_abs * rms(ref row).  The last one follows from the arithmetic: an output element is a sum
    of products whose operands were rounded to bf16 (relative error at most 2^-9 each, independent), so its error
    scales with the typical magnitude of its row (about 2e-3 of the row's rms over the three rounded stages of the
    aug-Q chain), not with the element itself, plus 2^-9 |ref| from rounding the result; c_abs = 2e-2 leaves ten
    standard deviations, and an element of small magnitude that is simply wrong (by its row's rms) fails it.
    `out` and `ref` are [rows, columns] (or reshaped to that)."""
    out = np.asarray(out, dtype=np.float64).reshape(-1, out.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(out.shape)
    err = np.abs(out - ref)
    assert np.isfinite(out).all(), what
    big = np.abs(ref).max()
    assert err.max() <= 1e-2 * big, f"{what}: max err {err.max():.3e} vs max|ref| {big:.3e}"
    rms_all = np.sqrt(np.mean(ref ** 2))
    rms = np.sqrt(np.mean(err ** 2)) / max(rms_all, 1e-300)
    assert rms <= 4e-3, f"{what}: rms err / rms ref = {rms:.3e}"
    row_rms = np.sqrt(np.mean(ref ** 2, axis=1, keepdims=True))
    bound = 2.0 ** -8 * np.abs(ref) + c_abs * row_rms
    worst = (err / np.maximum(bound, 1e-300)).max()
    assert worst <= 1.0, f"{what}: element-wise bound exceeded by {worst:.2f}x"
    return float(worst)
