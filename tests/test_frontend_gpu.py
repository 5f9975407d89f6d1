"""GPU parity of the steps around the cache update in the paper's attention listing: the key / value projections
(diffqkv_project), the rotary embedding fused into the projection and into the augmented-Q epilogue
(diffqkv_augq_rope), and the cache update on its own (diffqkv_cache_append), against the float64 oracle through
the C ABI.  Tolerances as in test_augq_gpu.py (bf16 rounding of the result, fp32 accumulation); the cache update is
pure byte movement and must match bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_proj, device_cache, run_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def _check(out, ref, what):
    check_proj(out, ref, what)


def _tables(oracle, pos, d, theta):
    c, s = oracle.rope_tables(pos, d, theta)
    return (torch.from_numpy(c.astype(np.float32)).cuda().contiguous(), torch.from_numpy(s.astype(np.float32)).cuda().contiguous())


@pytest.mark.parametrize("T", [1, 4, 16, 17, 50, 64, 65, 200, 1000])
@pytest.mark.parametrize("heads,d", [(4, 128), (3, 128), (8, 64), (6, 64)])
def test_projection_with_and_without_rotation(api, oracle, T, heads, d):
    """d_out = heads * d ends in a half-filled 256-column tile for odd head counts at d 128."""
    d_in, theta = 256, 50000.0
    x = W.normal(31, (T, d_in))
    w = W.normal(32, (heads * d, d_in), std=d_in ** -0.5)
    pos = np.random.Generator(np.random.Philox(key=33)).integers(0, 70000, size=T)
    plain = oracle.linear(x, w)
    y = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"))
    torch.cuda.synchronize()
    _check(y.float().cpu().numpy().astype(np.float64), plain, "plain projection")
    cos, sin = _tables(oracle, pos, d, theta)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    yr = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"), d, cos, sin, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.rope(plain.reshape(T, heads, d), pos, theta).reshape(T, heads * d)
    _check(yr.float().cpu().numpy().astype(np.float64), ref, "rotated projection")


@pytest.fixture
def tensor_gemm(api):
    """Switches the projections to the tensor-core GEMM for any row count and back."""
    yield api.force_tensor_gemm
    api.force_tensor_gemm(False)


@pytest.mark.parametrize("T", [3, 16, 40])
def test_few_rows_on_either_kernel(api, oracle, tensor_gemm, T):
    """Up to 64 rows take the weight-streaming kernel, the tensor-core GEMM computes the same thing: both against the
    oracle, for a K that is not a multiple of the 512-column stage and the three epilogues."""
    d_in, heads, d, theta = 896, 6, 64, 500000.0
    x = W.normal(61, (T, d_in))
    w = W.normal(62, (heads * d, d_in), std=d_in ** -0.5)
    pos = np.arange(T) * 7 + 3
    cos, sin = _tables(oracle, pos, d, theta)
    plain = oracle.linear(x, w)
    ref_rot = oracle.rope(plain.reshape(T, heads, d), pos, theta).reshape(T, heads * d)
    h = W.normal(63, (T, 256), std=1.0)
    ws = [W.normal(64, (384, 256), std=256 ** -0.5), W.normal(65, (640, 384), std=384 ** -0.5),
          W.normal(66, (640, 384), std=384 ** -0.5), W.normal(67, (256, 640), std=640 ** -0.5)]
    ref_q = oracle.augq(h, *ws)
    for on in (False, True):
        tensor_gemm(on)
        y = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"))
        yr = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"), d, cos, sin)
        q = api.diffqkv_augq(W.to_torch(h, "cuda"), *(W.to_torch(a, "cuda") for a in ws))
        torch.cuda.synchronize()
        _check(y.float().cpu().numpy().astype(np.float64), plain, f"plain, tensor_gemm={on}")
        _check(yr.float().cpu().numpy().astype(np.float64), ref_rot, f"rotated, tensor_gemm={on}")
        _check(q.float().cpu().numpy().astype(np.float64), ref_q, f"aug-Q, tensor_gemm={on}")


def test_rotation_at_position_zero_is_the_plain_projection(api, oracle):
    T, d_in, heads, d = 130, 128, 2, 128
    x, w = W.normal(41, (T, d_in)), W.normal(42, (heads * d, d_in), std=d_in ** -0.5)
    cos, sin = _tables(oracle, np.zeros(T, np.int64), d, 50000.0)
    a = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"))
    b = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"), d, cos, sin)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_augq_with_rotation(api, oracle):
    T, d_model, n_q, d, d_aug, theta = 300, 256, 4, 128, 384, 500000.0
    d_q0 = n_q * d
    h = W.normal(51, (T, d_model))
    ws = [W.normal(52, (d_q0, d_model), std=d_model ** -0.5), W.normal(53, (d_aug, d_q0), std=d_q0 ** -0.5),
          W.normal(54, (d_aug, d_q0), std=d_q0 ** -0.5), W.normal(55, (d_q0, d_aug), std=d_aug ** -0.5)]
    pos = np.arange(1000, 1000 + T)
    cos, sin = _tables(oracle, pos, d, theta)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q = api.diffqkv_augq_rope(W.to_torch(h, "cuda"), *(W.to_torch(w, "cuda") for w in ws), d, cos, sin, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.rope(oracle.augq(h, *ws).reshape(T, n_q, d), pos, theta).reshape(T, d_q0)
    _check(q.float().cpu().numpy().astype(np.float64), ref, "augq + rope")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("paged", [0, 16])
def test_cache_append_is_bit_exact(api, oracle, dtype, paged):
    cfg = W.DecodeConfig("t", batch=3, n_q=8, n_k=2, n_v=4, d_qk=64, d_v=128, kv_len=96, dtype=dtype, seed=61)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([0, 17, 60], np.int32))
    if paged:
        inp = W.paginate(inp, paged, seed=5)
    q_len = 30
    k_new = W.normal(62, (cfg.batch, q_len, cfg.n_k, cfg.d_qk), dtype=dtype)
    v_new = W.normal(63, (cfg.batch, q_len, cfg.n_v, cfg.d_v), dtype=dtype)
    cache = device_cache(api, inp)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.diffqkv_cache_append(W.to_torch(k_new, "cuda"), W.to_torch(v_new, "cuda"), cache, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    k_ref, v_ref = inp.k.copy(), inp.v.copy()
    oracle.cache_append(k_new, v_new, oracle.Cache(k_ref, v_ref, inp.k_strides, inp.v_strides, inp.seqlens,
                                                   inp.page_table, inp.cfg.page_size))
    view = torch.uint16 if dtype == "bf16" else torch.float32
    assert np.array_equal(cache.k.view(view).cpu().numpy(), k_ref)
    assert np.array_equal(cache.v.view(view).cpu().numpy(), v_ref)


def test_append_past_the_end_is_reported_not_written(api):
    cfg = W.DecodeConfig("t", batch=1, n_q=4, n_k=2, n_v=2, d_qk=64, d_v=64, kv_len=64, seed=71)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([60], np.int32))
    cache = device_cache(api, inp)
    before_k = cache.k.clone()
    k_new, v_new = W.normal(72, (1, 8, 2, 64)), W.normal(73, (1, 8, 2, 64))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.diffqkv_cache_append(W.to_torch(k_new, "cuda"), W.to_torch(v_new, "cuda"), cache, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << api.ERR_INDEX
    assert torch.equal(cache.k[:, :, :60], before_k[:, :, :60])  # rows 60..63 were written, nothing else moved


def test_decode_step_through_the_front_end(api, oracle):
    """One decode step the way a model layer runs it: project the new token's hidden state to k and v (k rotated),
    append, then attend with the augmented, rotated query; every stage on the GPU, the oracle chained alongside."""
    n_q, n_k, n_v, d, d_model, d_aug, theta, batch, S = 8, 2, 4, 128, 256, 384, 50000.0, 2, 300
    cfg = W.DecodeConfig("t", batch=batch, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, kv_len=S, seed=81)
    lens = np.array([S - 1, 100], np.int32)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    h = W.normal(82, (batch, d_model))
    w_k = W.normal(83, (n_k * d, d_model), std=d_model ** -0.5)
    w_v = W.normal(84, (n_v * d, d_model), std=d_model ** -0.5)
    ws = [W.normal(85, (n_q * d, d_model), std=d_model ** -0.5), W.normal(86, (d_aug, n_q * d), std=(n_q * d) ** -0.5),
          W.normal(87, (d_aug, n_q * d), std=(n_q * d) ** -0.5), W.normal(88, (n_q * d, d_aug), std=d_aug ** -0.5)]
    pos = lens.astype(np.int64)  # the new token sits at index len
    cos, sin = _tables(oracle, pos, d, theta)
    dev = "cuda"
    th = W.to_torch(h, dev)
    k_new = api.diffqkv_project(th, W.to_torch(w_k, dev), d, cos, sin).view(batch, 1, n_k, d)
    v_new = api.diffqkv_project(th, W.to_torch(w_v, dev)).view(batch, 1, n_v, d)
    q = api.diffqkv_augq_rope(th, *(W.to_torch(w, dev) for w in ws), d, cos, sin).view(batch, n_q, d)
    cache = device_cache(api, inp)
    api.diffqkv_cache_append(k_new, v_new, cache)
    cache.seqlens += 1
    out = api.diffqkv_decode(q, cache, n_k, n_v, cfg.scale, out_dtype=torch.float32)
    torch.cuda.synchronize()
    # the oracle attends over the GPU's own bf16 k, v and q, so that the comparison isolates the attention step
    k_host, v_host = inp.k.copy(), inp.v.copy()
    oc = oracle.Cache(k_host, v_host, inp.k_strides, inp.v_strides, lens)
    oracle.cache_append(k_new.view(torch.uint16).cpu().numpy(), v_new.view(torch.uint16).cpu().numpy(), oc)
    oc2 = oracle.Cache(k_host, v_host, inp.k_strides, inp.v_strides, lens + 1)
    ref, _ = oracle.decode(q.view(torch.uint16).cpu().numpy(), oc2, n_q, n_k, n_v, d, d, cfg.scale)
    check_bf16(out.cpu().numpy().astype(np.float64), ref, "decode after front end")
    # and the front-end outputs themselves against the unrounded chain
    k_ref = oracle.rope(oracle.linear(h, w_k).reshape(batch, n_k, d), pos, theta)
    _check(k_new.float().cpu().numpy().astype(np.float64).reshape(batch, n_k, d), k_ref, "k_new")


@pytest.mark.parametrize("batch,paged,rotate", [(2, 0, True), (5, 16, True), (16, 0, False), (33, 64, True), (70, 0, True)])
def test_fused_decode_front_end_equals_the_separate_steps(api, oracle, tensor_gemm, batch, paged, rotate):
    """diffqkv_decode_frontend writes the same cache rows and returns the same queries as diffqkv_project x 2 +
    diffqkv_cache_append + diffqkv_augq_rope, bit for bit when both run on the same kernels (up to 64 sequences the
    weight-streaming kernel, beyond that the tensor-core one), and the new K row matches the oracle's chain."""
    n_q, n_k, n_v, d, d_model, d_aug, theta, S = 8, 2, 4, 128, 256, 384, 50000.0, 200
    cfg = W.DecodeConfig("t", batch=batch, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, kv_len=S, seed=181)
    lens = (np.arange(batch) * 37 % (S - 1)).astype(np.int32)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    if paged:
        inp = W.paginate(inp, paged, seed=5)
    h = W.normal(182, (batch, d_model))
    w_k = W.normal(183, (n_k * d, d_model), std=d_model ** -0.5)
    w_v = W.normal(184, (n_v * d, d_model), std=d_model ** -0.5)
    ws = [W.normal(185, (n_q * d, d_model), std=d_model ** -0.5), W.normal(186, (d_aug, n_q * d), std=(n_q * d) ** -0.5),
          W.normal(187, (d_aug, n_q * d), std=(n_q * d) ** -0.5), W.normal(188, (n_q * d, d_aug), std=d_aug ** -0.5)]
    pos = lens.astype(np.int64)
    cos, sin = _tables(oracle, pos, d, theta) if rotate else (None, None)
    dev = "cuda"
    th, tw = W.to_torch(h, dev), [W.to_torch(w, dev) for w in ws]
    tk, tv = W.to_torch(w_k, dev), W.to_torch(w_v, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # separate steps
    c1 = device_cache(api, inp)
    k_new = (api.diffqkv_project(th, tk, d, cos, sin) if rotate else api.diffqkv_project(th, tk)).view(batch, 1, n_k, d)
    v_new = api.diffqkv_project(th, tv).view(batch, 1, n_v, d)
    api.diffqkv_cache_append(k_new, v_new, c1, dev_status=status)
    q1 = (api.diffqkv_augq_rope(th, *tw, d, cos, sin) if rotate else api.diffqkv_augq(th, *tw)).view(batch, n_q, d)
    # fused
    c2 = device_cache(api, inp)
    q2 = api.diffqkv_decode_frontend(th, *tw, tk, tv, c2, n_q, d, d, cos, sin, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(q1.view(torch.uint16), q2.view(torch.uint16))
    assert torch.equal(c1.k.view(torch.uint16), c2.k.view(torch.uint16))
    assert torch.equal(c1.v.view(torch.uint16), c2.v.view(torch.uint16))
    k_ref = oracle.linear(h, w_k).reshape(batch, n_k, d)
    if rotate:
        k_ref = oracle.rope(k_ref, pos, theta)
    _check(k_new.float().cpu().numpy().astype(np.float64).reshape(batch, n_k, d), k_ref, "k_new")
    if batch <= 64:  # the same entry on the tensor-core kernels agrees within rounding
        tensor_gemm(True)
        c3 = device_cache(api, inp)
        q3 = api.diffqkv_decode_frontend(th, *tw, tk, tv, c3, n_q, d, d, cos, sin, dev_status=status)
        torch.cuda.synchronize()
        assert (q3.float() - q2.float()).abs().max().item() <= 2e-2 * q2.float().abs().max().item()
        assert (c3.k.float() - c2.k.float()).abs().max().item() <= 2e-2 * c2.k.float().abs().max().item()


def test_fused_decode_front_end_reports_a_full_cache(api):
    n_q, n_k, n_v, d, d_model, d_aug = 8, 2, 2, 128, 128, 128
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device="cuda")  # noqa: E731
    lens = torch.tensor([64, 10], dtype=torch.int32, device="cuda")  # sequence 0 is full
    cache = api.KVCache(z(2, n_k, 64, d), z(2, n_v, 64, d), lens, 64)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.diffqkv_decode_frontend(z(2, d_model), z(n_q * d, d_model), z(d_aug, n_q * d), z(d_aug, n_q * d),
                                z(n_q * d, d_aug), z(n_k * d, d_model), z(n_v * d, d_model), cache, n_q, d, d,
                                dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << api.ERR_INDEX
