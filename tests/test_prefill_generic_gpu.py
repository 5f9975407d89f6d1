"""GPU parity of diffqkv_prefill on the shapes its tensor-core kernel does not take (fp32 storage, head dimensions
other than (128, 128), (64, 64) and (64, 128)): cache update + causal attention on the generic fp32-FMA kernel, against the float64
oracle through the C ABI.  bf16 storage: the bf16 tolerances of helpers.check_bf16; fp32 storage:
max |err| / max |ref| <= 1e-5.  The cache contents after the call must equal the oracle's cache update bit for bit."""
import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_f32, check_lse

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def run_both(api, oracle, seed, batch, q_len, heads, d_qk, d_v, past, dtype):
    n_q, n_k, n_v = heads
    past = np.asarray(past, dtype=np.int32)
    S = int(past.max() + q_len)
    q = W.normal(seed, (batch, q_len, n_q, d_qk), dtype=dtype)
    k_new = W.normal(seed + 1, (batch, q_len, n_k, d_qk), dtype=dtype)
    v_new = W.normal(seed + 2, (batch, q_len, n_v, d_v), dtype=dtype)
    k = W.normal(seed + 3, (batch, n_k, S, d_qk), dtype=dtype)
    v = W.normal(seed + 4, (batch, n_v, S, d_v), dtype=dtype)
    ks, vs = (n_k * S * d_qk, S * d_qk, d_qk), (n_v * S * d_v, S * d_v, d_v)
    scale = d_qk ** -0.5
    # oracle
    k_ref, v_ref = k.copy(), v.copy()
    oc = oracle.Cache(k_ref, v_ref, ks, vs, past)
    oracle.cache_append(k_new, v_new, oc)
    ref, lse_ref = oracle.prefill(q, past, oc, n_k, n_v, d_v, scale)
    # GPU
    dev = "cuda"
    kd, vd = W.to_torch(k.copy(), dev), W.to_torch(v.copy(), dev)
    cache = api.KVCache(kd, vd, torch.from_numpy(past).to(dev), S, k_strides=ks, v_strides=vs, num_blocks=batch)
    lse = torch.full((batch, q_len, n_q), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = api.diffqkv_prefill(W.to_torch(q, dev), W.to_torch(k_new, dev), W.to_torch(v_new, dev), cache, scale,
                              lse=lse, dev_status=status, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert api.last_prefill_kernel() == 1, "these shapes belong to the generic kernel"
    bits = torch.uint16 if dtype == "bf16" else torch.float32
    for b in range(batch):
        n = int(past[b]) + q_len
        assert np.array_equal(kd.view(bits).cpu().numpy()[b, :, :n], k_ref[b, :, :n])
        assert np.array_equal(vd.view(bits).cpu().numpy()[b, :, :n], v_ref[b, :, :n])
    return out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), ref, lse_ref


@pytest.mark.parametrize("d_qk,d_v", [(192, 192), (128, 64), (32, 256)])
@pytest.mark.parametrize("heads", [(8, 2, 4), (4, 4, 1)])
def test_bf16_other_head_dimensions(api, oracle, d_qk, d_v, heads):
    out, lse, ref, lse_ref = run_both(api, oracle, 300 + d_qk + d_v, 2, 150, heads, d_qk, d_v, [0, 37], "bf16")
    check_bf16(out, ref, f"d_qk={d_qk} d_v={d_v} heads={heads}")
    check_lse(lse, lse_ref, 2e-2)


@pytest.mark.parametrize("d", [64, 128])
def test_fp32_storage(api, oracle, d):
    out, lse, ref, lse_ref = run_both(api, oracle, 400 + d, 2, 131, (8, 2, 4), d, d, [5, 200], "f32")
    check_f32(out, ref, f"fp32 d={d}")
    check_lse(lse, lse_ref, 1e-4)


def test_first_row_without_past_is_its_own_v_row(api, oracle):
    out, _, ref, _ = run_both(api, oracle, 500, 1, 9, (4, 2, 2), 64, 64, [0], "f32")
    assert np.abs(out[0, 0] - ref[0, 0]).max() <= 1e-6


def test_tensor_core_shape_still_takes_the_tensor_core_kernel(api):
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device="cuda")  # noqa: E731
    cache = api.KVCache(z(1, 2, 64, 128), z(1, 2, 64, 128), torch.zeros(1, dtype=torch.int32, device="cuda"), 64)
    api.diffqkv_prefill(z(1, 8, 4, 128), z(1, 8, 2, 128), z(1, 8, 2, 128), cache, 0.1)
    torch.cuda.synchronize()
    assert api.last_prefill_kernel() == 2
