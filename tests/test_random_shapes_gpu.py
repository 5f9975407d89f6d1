"""Seeded random shapes through every attention entry point, each against the float64 oracle on the same host
buffers: head counts drawn from the divisors of n_q (so n_k > n_v, n_k not dividing n_v and multi-query shapes all
occur), head dimensions 64 / 128 in any combination, ragged and empty sequences, contiguous and paged caches, and the
fused decode front end against its separate steps.  The draws are fixed by the case number, so a failure names a
shape that can be rerun alone."""
import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_lse, check_proj, device_cache, oracle_cache, run_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def _rng(kind, it):
    return np.random.Generator(np.random.Philox(key=1_000_003 * kind + it))


def _heads(rng):
    n_q = int(rng.choice([4, 8, 12, 16, 32]))
    divs = [d for d in range(1, n_q + 1) if n_q % d == 0]
    return n_q, int(rng.choice(divs)), int(rng.choice(divs))


@pytest.mark.parametrize("cluster", [-1, 1])
@pytest.mark.parametrize("it", range(20))
def test_random_decode(api, oracle, it, cluster):
    """cluster = 1 forces the on-chip merge of a row's blocks wherever at least two blocks per row fit on the GPU
    (left to itself the library takes it for some of these shapes only)."""
    api.decode_cluster(cluster)
    try:
        _random_decode(api, oracle, it)
    finally:
        api.decode_cluster(-1)


def _random_decode(api, oracle, it):
    rng = _rng(1, it)
    n_q, n_k, n_v = _heads(rng)
    d_qk, d_v = int(rng.choice([64, 128])), int(rng.choice([64, 128]))
    batch, S = int(rng.integers(1, 6)), int(rng.integers(1, 3000))
    lens = rng.integers(0, S + 1, size=batch).astype(np.int32)
    cfg = W.DecodeConfig("r", batch=batch, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d_qk, d_v=d_v, kv_len=S, seed=11000 + it)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    page = int(rng.choice([0, 16, 32, 64, 128]))
    if page:
        inp = W.paginate(inp, page, seed=it)
    what = f"decode heads {n_q}/{n_k}/{n_v} d {d_qk}/{d_v} lens {lens.tolist()} page {page}"
    q, cache = W.to_torch(inp.q, "cuda"), device_cache(api, inp)
    lse = torch.full((batch, n_q), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = api.diffqkv_decode(q, cache, n_k, n_v, cfg.scale, lse=lse, dev_status=status, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, what
    ref, lse_ref = run_oracle(oracle, inp)
    check_bf16(out.cpu().numpy().astype(np.float64), ref, what)
    check_lse(lse.cpu().numpy().astype(np.float64), lse_ref, 2e-2, what)


@pytest.mark.parametrize("it", range(14))
def test_random_selective_v(api, oracle, it):
    rng = _rng(2, it)
    n_q, n_k, n_v = _heads(rng)
    if n_q // n_k > 32:
        n_k = n_q // 32
    d_qk, d_v = int(rng.choice([64, 128])), int(rng.choice([64, 128]))
    batch, S = int(rng.integers(1, 5)), int(rng.integers(1, 3000))
    lens = rng.integers(0, S + 1, size=batch).astype(np.int32)
    cfg = W.DecodeConfig("r", batch=batch, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d_qk, d_v=d_v, kv_len=S, seed=12000 + it)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    page = int(rng.choice([0, 16, 64, 128]))
    if page:
        inp = W.paginate(inp, page, seed=it)
    k = int(rng.choice([1, 3, 20, 100, 700]))
    what = f"top-{k} heads {n_q}/{n_k}/{n_v} d {d_qk}/{d_v} lens {lens.tolist()} page {page}"
    q, cache = W.to_torch(inp.q, "cuda"), device_cache(api, inp)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = api.diffqkv_decode_topk(q, cache, n_k, n_v, cfg.scale, k, dev_status=status, out_dtype=torch.float32)
    api.topk_general_only(True)
    try:
        out2 = api.diffqkv_decode_topk(q, cache, n_k, n_v, cfg.scale, k, out_dtype=torch.float32)
    finally:
        api.topk_general_only(False)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, what
    assert torch.equal(out, out2), what + ": the two selection paths differ"
    ref, _, _, margin = oracle.decode_topk(inp.q, oracle_cache(oracle, inp), n_q, n_k, n_v, d_qk, d_v, cfg.scale, k)
    clear = margin > 4e-5  # rows whose kept set does not hinge on the last bits of a score
    if clear.any():
        check_bf16(out.cpu().numpy().astype(np.float64)[clear], ref[clear], what)


@pytest.mark.parametrize("it", range(16))
def test_random_prefill(api, oracle, it):
    rng = _rng(3, it)
    n_q, n_k, n_v = _heads(rng)
    d_qk = int(rng.choice([64, 128]))
    d_v = d_qk if rng.random() < 0.7 else int(rng.choice([64, 128]))
    batch, q_len = int(rng.integers(1, 4)), int(rng.integers(1, 500))
    past = rng.integers(0, 400, size=batch).astype(np.int32)
    S = int(past.max() + q_len)
    what = f"prefill heads {n_q}/{n_k}/{n_v} d {d_qk}/{d_v} q_len {q_len} past {past.tolist()}"
    q = W.normal(13000 + it, (batch, q_len, n_q, d_qk))
    k_new, v_new = W.normal(13100 + it, (batch, q_len, n_k, d_qk)), W.normal(13200 + it, (batch, q_len, n_v, d_v))
    k, v = W.normal(13300 + it, (batch, n_k, S, d_qk)), W.normal(13400 + it, (batch, n_v, S, d_v))
    ks, vs = (n_k * S * d_qk, S * d_qk, d_qk), (n_v * S * d_v, S * d_v, d_v)
    oc = oracle.Cache(k.copy(), v.copy(), ks, vs, past)
    oracle.cache_append(k_new, v_new, oc)
    ref, lse_ref = oracle.prefill(q, past, oc, n_k, n_v, d_v, d_qk ** -0.5)
    cache = api.KVCache(W.to_torch(k.copy(), "cuda"), W.to_torch(v.copy(), "cuda"), torch.from_numpy(past).cuda(), S,
                        k_strides=ks, v_strides=vs, num_blocks=batch)
    lse = torch.full((batch, q_len, n_q), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = api.diffqkv_prefill(W.to_torch(q, "cuda"), W.to_torch(k_new, "cuda"), W.to_torch(v_new, "cuda"), cache,
                              d_qk ** -0.5, lse=lse, dev_status=status, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, what
    check_bf16(out.cpu().numpy().astype(np.float64), ref, what)
    check_lse(lse.cpu().numpy().astype(np.float64), lse_ref, 2e-2, what)
    assert np.array_equal(cache.k.view(torch.uint16).cpu().numpy(), oc.k), what + ": K cache"
    assert np.array_equal(cache.v.view(torch.uint16).cpu().numpy(), oc.v), what + ": V cache"


@pytest.mark.parametrize("it", range(10))
def test_random_decode_front_end(api, oracle, it):
    rng = _rng(4, it)
    d = int(rng.choice([64, 128]))
    n_q = int(rng.choice([8, 16]))
    n_k, n_v = int(rng.choice([2, 4])), int(rng.choice([2, 4, 8]))
    batch, S = int(rng.integers(1, 80)), 150
    d_model, d_aug = 128 * int(rng.integers(1, 5)), 128 * int(rng.integers(1, 5))
    page = int(rng.choice([0, 16, 64]))
    theta = 50000.0
    what = f"front end batch {batch} heads {n_q}/{n_k}/{n_v} d {d} d_model {d_model} d_aug {d_aug} page {page}"
    cfg = W.DecodeConfig("r", batch=batch, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, kv_len=S, seed=14000 + it)
    lens = rng.integers(0, S - 1, size=batch).astype(np.int32)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    if page:
        inp = W.paginate(inp, page, seed=it)
    h = W.normal(14100 + it, (batch, d_model))
    w_k = W.normal(14200 + it, (n_k * d, d_model), std=d_model ** -0.5)
    w_v = W.normal(14300 + it, (n_v * d, d_model), std=d_model ** -0.5)
    ws = [W.normal(14400 + it, (n_q * d, d_model), std=d_model ** -0.5),
          W.normal(14500 + it, (d_aug, n_q * d), std=(n_q * d) ** -0.5),
          W.normal(14600 + it, (d_aug, n_q * d), std=(n_q * d) ** -0.5),
          W.normal(14700 + it, (n_q * d, d_aug), std=d_aug ** -0.5)]
    pos = lens.astype(np.int64)
    c, s = oracle.rope_tables(pos, d, theta)
    cos, sin = (torch.from_numpy(c.astype(np.float32)).cuda().contiguous(),
                torch.from_numpy(s.astype(np.float32)).cuda().contiguous())
    th, tw = W.to_torch(h, "cuda"), [W.to_torch(w, "cuda") for w in ws]
    tk, tv = W.to_torch(w_k, "cuda"), W.to_torch(w_v, "cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    c1 = device_cache(api, inp)
    k_new = api.diffqkv_project(th, tk, d, cos, sin).view(batch, 1, n_k, d)
    v_new = api.diffqkv_project(th, tv).view(batch, 1, n_v, d)
    api.diffqkv_cache_append(k_new, v_new, c1, dev_status=status)
    q1 = api.diffqkv_augq_rope(th, *tw, d, cos, sin).view(batch, n_q, d)
    c2 = device_cache(api, inp)
    q2 = api.diffqkv_decode_frontend(th, *tw, tk, tv, c2, n_q, d, d, cos, sin, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, what
    assert torch.equal(q1.view(torch.uint16), q2.view(torch.uint16)), what
    assert torch.equal(c1.k.view(torch.uint16), c2.k.view(torch.uint16)), what
    assert torch.equal(c1.v.view(torch.uint16), c2.v.view(torch.uint16)), what
    q_ref = oracle.rope(oracle.augq(h, *ws).reshape(batch, n_q, d), pos, theta)
    check_proj(q2.float().cpu().numpy().astype(np.float64).reshape(batch, n_q * d), q_ref.reshape(batch, n_q * d), what)
