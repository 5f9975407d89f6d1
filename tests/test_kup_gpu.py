"""GPU parity of the half-width K cache path (Section 2: Attend with different Q and K head dimensions goes through
a feed-forward layer on K; Observation 2: d_k = d_v / 2): diffqkv_fold_k_up folds the layer into the queries, then
diffqkv_decode / diffqkv_prefill score the narrow cache directly.  The oracle does what the paper states: it widens
every cached key through the layer and takes the inner product at full width.  bf16 tolerances of
helpers.check_bf16 (the folded query is rounded to bf16 once more, a relative 2^-9 per element that moves a score
by about 1e-3)."""
import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_lse

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def _strides(n, S, d):
    return (n * S * d, S * d, d)


@pytest.mark.parametrize("heads", [(32, 4, 8), (16, 2, 4), (8, 8, 8)])
def test_decode_over_half_width_keys(api, oracle, heads):
    n_q, n_k, n_v = heads
    d_q, d_k, d_v, S = 128, 64, 128, 3000
    lens = np.array([3000, 1, 777, 0, 2049], np.int32)
    b = len(lens)
    q = W.normal(501, (b, n_q, d_q))
    k = W.normal(502, (b, n_k, S, d_k))
    v = W.normal(503, (b, n_v, S, d_v))
    w = W.normal(504, (n_k, d_q, d_k), std=d_k ** -0.5)
    scale = d_q ** -0.5
    ref, lse_ref = oracle.decode_kup(q, w, oracle.Cache(k, v, _strides(n_k, S, d_k), _strides(n_v, S, d_v), lens),
                                     n_q, n_k, n_v, d_v, scale)
    dev = "cuda"
    qf = api.diffqkv_fold_k_up(W.to_torch(q, dev), W.to_torch(w, dev))
    assert qf.shape == (b, n_q, d_k)
    cache = api.KVCache(W.to_torch(k, dev), W.to_torch(v, dev), torch.from_numpy(lens).to(dev), S)
    lse = torch.full((b, n_q), float("nan"), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = api.diffqkv_decode(qf, cache, n_k, n_v, scale, lse=lse, dev_status=status, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and api.last_decode_kernel() == 2
    check_bf16(out.cpu().numpy().astype(np.float64), ref, f"heads {heads}")
    check_lse(lse.cpu().numpy().astype(np.float64), lse_ref, 2e-2, f"heads {heads}")


@pytest.mark.parametrize("n_q,n_k,d_q,d_k,T", [
    (12, 3, 128, 64, 37),     # tensor-core kernel, 148 rows per K head: one full 128-row tile and a ragged one
    (32, 4, 128, 64, 1000),   # several tiles per block
    (16, 16, 64, 32, 9),      # groups of one head, a single 16-row slab partly filled
    (8, 2, 256, 128, 131),    # the widest layer the tensor-core kernel takes
    (6, 2, 128, 32, 50),      # a group size that does not divide the slab height
    (4, 4, 64, 64, 300),      # square layer
    (8, 2, 96, 48, 21),       # d_k not a multiple of 32: the plain kernel
    (12, 4, 100, 20, 13),     # d_q not a multiple of 16: the plain kernel
    (8, 4, 64, 128, 40),      # a widening layer: the plain kernel
])
def test_folded_queries_match_the_definition(api, n_q, n_k, d_q, d_k, T):
    """q' = W[hk]^T q per head, against the same product in float64: every element within one bf16 rounding of the
    exact value (half a unit in the last of eight significant bits: 2^-8 relative) plus the fp32 accumulation's share."""
    q, w = W.normal(511, (T, n_q, d_q)), W.normal(512, (n_k, d_q, d_k), std=d_k ** -0.5)
    out = torch.full((T, n_q, d_k), float("nan"), dtype=torch.bfloat16, device="cuda")
    api.diffqkv_fold_k_up(W.to_torch(q, "cuda"), W.to_torch(w, "cuda"), out=out)
    got = out.float().cpu().numpy().astype(np.float64)
    qf, wf = W.as_f64(q), W.as_f64(w)
    for h in range(n_q):
        ref = qf[:, h] @ wf[h // (n_q // n_k)]
        err = np.abs(got[:, h] - ref)
        assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 2e-5 * np.abs(ref).max()), (h, err.max())


@pytest.mark.parametrize("q_len,past", [(300, [0, 0]), (257, [100, 31]), (1, [5, 0])])
def test_prefill_over_half_width_keys_runs_on_the_tensor_cores(api, oracle, q_len, past):
    """Prefill row i equals a decode at length past + i + 1 (pinned for the oracle), so sampled rows are checked
    against the oracle's K feed-forward + Attend at that length; the cache update must be exact."""
    n_q, n_k, n_v, d_q, d_k, d_v = 16, 2, 4, 128, 64, 128
    past = np.asarray(past, np.int32)
    b = len(past)
    S = int(past.max()) + q_len
    q = W.normal(521, (b, q_len, n_q, d_q))
    k_new, v_new = W.normal(522, (b, q_len, n_k, d_k)), W.normal(523, (b, q_len, n_v, d_v))
    k, v = W.normal(524, (b, n_k, S, d_k)), W.normal(525, (b, n_v, S, d_v))
    w = W.normal(526, (n_k, d_q, d_k), std=d_k ** -0.5)
    scale = d_q ** -0.5
    dev = "cuda"
    qf = api.diffqkv_fold_k_up(W.to_torch(q, dev), W.to_torch(w, dev))
    kd, vd = W.to_torch(k.copy(), dev), W.to_torch(v.copy(), dev)
    cache = api.KVCache(kd, vd, torch.from_numpy(past).to(dev), S)
    lse = torch.full((b, q_len, n_q), float("nan"), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = api.diffqkv_prefill(qf, W.to_torch(k_new, dev), W.to_torch(v_new, dev), cache, scale, lse=lse,
                              dev_status=status, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and api.last_prefill_kernel() == 2
    k_ref, v_ref = k.copy(), v.copy()
    oc = oracle.Cache(k_ref, v_ref, _strides(n_k, S, d_k), _strides(n_v, S, d_v), past)
    oracle.cache_append(k_new, v_new, oc)
    for bi in range(b):
        n = int(past[bi]) + q_len
        assert np.array_equal(kd.view(torch.uint16).cpu().numpy()[bi, :, :n], k_ref[bi, :, :n])
        assert np.array_equal(vd.view(torch.uint16).cpu().numpy()[bi, :, :n], v_ref[bi, :, :n])
    o, l = out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    for i in sorted({0, 1, 127, 128, 129, 255, 256, q_len - 1} & set(range(q_len))):
        lens = (past + i + 1).astype(np.int32)
        ref, lse_ref = oracle.decode_kup(np.ascontiguousarray(q[:, i]), w,
                                         oracle.Cache(k_ref, v_ref, _strides(n_k, S, d_k), _strides(n_v, S, d_v), lens),
                                         n_q, n_k, n_v, d_v, scale)
        check_bf16(o[:, i], ref, f"row {i}")
        check_lse(l[:, i], lse_ref, 2e-2, f"row {i}")
