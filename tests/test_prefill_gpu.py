"""GPU parity of diffqkv_prefill (cache update + causal tcgen05 attention) against the float64 oracle, called
through the C ABI on the same seeded inputs.  bf16 inputs, fp32 accumulation: the bf16-mode tolerances of
helpers.check_bf16 apply (max |err| <= 2e-2, <= 1e-2 of max |ref|, element-wise 2e-2 + 1e-2 |ref|); the
cache contents after the call must equal the oracle's cache update bit for bit."""
import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_lse

pytestmark = pytest.mark.gpu
D = 128


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


class Case:
    """Seeded prefill problem with a contiguous [batch, head, S, d] cache holding `past` earlier tokens."""

    def __init__(self, seed, batch, q_len, heads, past, S=None, q_std=1.0, garbage=None, d=D, d_v=None):
        n_q, n_k, n_v = heads
        self.d = D = d
        self.d_v = d_v or d
        self.batch, self.q_len, self.heads = batch, q_len, heads
        self.past = np.asarray(past, dtype=np.int32)
        self.S = S or int(self.past.max() + q_len)
        self.q = W.normal(seed, (batch, q_len, n_q, D), std=q_std)
        self.k_new = W.normal(seed + 1, (batch, q_len, n_k, D))
        self.v_new = W.normal(seed + 2, (batch, q_len, n_v, self.d_v))
        self.k = W.normal(seed + 3, (batch, n_k, self.S, D))
        self.v = W.normal(seed + 4, (batch, n_v, self.S, self.d_v))
        if garbage is not None:  # poison everything at and after the first new row
            for b in range(batch):
                self.k[b, :, self.past[b]:] = garbage
                self.v[b, :, self.past[b]:] = garbage
        self.scale = D ** -0.5

    def strides(self, n, d=None):
        d = d or self.d
        return (n * self.S * d, self.S * d, d)


def run_gpu(api, case, paged=None, out_dtype=torch.float32):
    """Returns out, lse, status and the cache pools after the call (as uint16 host arrays, contiguous layout)."""
    dev = "cuda"
    n_q, n_k, n_v = case.heads
    seqlens = torch.from_numpy(case.past).to(dev)
    if paged is None:
        k, v = W.to_torch(case.k.copy(), dev), W.to_torch(case.v.copy(), dev)
        cache = api.KVCache(k, v, seqlens, case.S, k_strides=case.strides(n_k), v_strides=case.strides(n_v, case.d_v),
                            num_blocks=case.batch)
    else:
        inp = W.DecodeInputs(W.DecodeConfig("t", case.batch, n_q, n_k, n_v, case.d, case.d_v, case.S), None, case.k, case.v,
                             case.past, case.strides(n_k), case.strides(n_v, case.d_v), max_seqlen=case.S)
        pg = W.paginate(inp, paged, seed=99)
        k, v = W.to_torch(pg.k, dev), W.to_torch(pg.v, dev)
        cache = api.KVCache(k, v, seqlens, pg.max_seqlen, page_table=torch.from_numpy(pg.page_table).to(dev),
                            page_size=paged, k_strides=pg.k_strides, v_strides=pg.v_strides, num_blocks=pg.num_pages)
    lse = torch.full((case.batch, case.q_len, n_q), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = api.diffqkv_prefill(W.to_torch(case.q, dev), W.to_torch(case.k_new, dev), W.to_torch(case.v_new, dev),
                              cache, case.scale, lse=lse, dev_status=status, out_dtype=out_dtype)
    torch.cuda.synchronize()
    k_after = k.view(torch.uint16).cpu().numpy()
    v_after = v.view(torch.uint16).cpu().numpy()
    if paged is not None:  # gather the pages back into the contiguous layout
        kc, vc = np.zeros_like(case.k), np.zeros_like(case.v)
        pt = pg.page_table
        for b in range(case.batch):
            for pi in range(pt.shape[1]):
                lo, hi = pi * paged, min(case.S, (pi + 1) * paged)
                if lo < hi:
                    kc[b, :, lo:hi] = k_after[pt[b, pi], :, : hi - lo]
                    vc[b, :, lo:hi] = v_after[pt[b, pi], :, : hi - lo]
        k_after, v_after = kc, vc
    return (out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64),
            int(status.item()), k_after, v_after)


def run_oracle(oracle, case, rows=None):
    n_q, n_k, n_v = case.heads
    k, v = case.k.copy(), case.v.copy()
    cache = oracle.Cache(k, v, case.strides(n_k), case.strides(n_v, case.d_v), case.past)
    oracle.cache_append(case.k_new, case.v_new, cache)
    out, lse = oracle.prefill(case.q, case.past, cache, n_k, n_v, case.d_v, case.scale, rows=rows)
    return out, lse, k, v


def check_case(api, oracle, case, what, paged=None):
    ref, lse_ref, k_ref, v_ref = run_oracle(oracle, case)
    out, lse, st, k_after, v_after = run_gpu(api, case, paged=paged)
    assert st == 0, f"{what}: device status {st}"
    check_bf16(out, ref, what)
    check_lse(lse, lse_ref, 2e-2, what)
    for b in range(case.batch):  # rows [0, past + q_len) of the cache are defined; they must match bit for bit
        n = int(case.past[b]) + case.q_len
        assert np.array_equal(k_after[b, :, :n], k_ref[b, :, :n]), f"{what}: K cache differs"
        assert np.array_equal(v_after[b, :, :n], v_ref[b, :, :n]), f"{what}: V cache differs"
    return out


@pytest.mark.parametrize("q_len", [1, 63, 64, 65, 128, 129, 255, 256, 257, 700])
def test_ragged_query_lengths_no_past(api, oracle, q_len):
    check_case(api, oracle, Case(10 + q_len, 2, q_len, (8, 2, 4), [0, 0]), f"q_len={q_len}")


@pytest.mark.parametrize("heads", [(16, 2, 4), (4, 4, 4), (8, 1, 8), (8, 8, 1), (12, 6, 2), (32, 4, 8)])
def test_head_configurations(api, oracle, heads):
    check_case(api, oracle, Case(300, 1, 333, heads, [0]), f"heads={heads}")


@pytest.mark.parametrize("past", [[37, 200], [64, 0], [511, 1]])
def test_cached_prefix_is_attended(api, oracle, past):
    """Bottom-right aligned causal mask: query row i sees tokens 0 .. past + i."""
    check_case(api, oracle, Case(400, 2, 300, (8, 2, 4), past), f"past={past}")


def test_first_row_without_past_is_its_own_v_row(api, oracle):
    case = Case(500, 1, 130, (8, 2, 4), [0])
    out, _, st, _, _ = run_gpu(api, case)
    assert st == 0
    for h in range(8):
        assert np.array_equal(out[0, 0, h], W.as_f64(case.v_new[0, 0, h // 2]))


def test_peaked_softmax_exercises_rescaling(api, oracle):
    """Queries with std 4: scores spread over tens of log2 units, so the running reference maximum is raised
    many times and O is rescaled in tensor memory."""
    check_case(api, oracle, Case(600, 1, 600, (8, 2, 4), [100], q_std=4.0), "peaked")


def test_nearly_uniform_softmax(api, oracle):
    check_case(api, oracle, Case(610, 1, 400, (8, 2, 4), [0], q_std=0.01), "uniform")


def test_nan_garbage_past_the_sequence_end_is_never_read_into_results(api, oracle):
    """Cache rows at and after the first new row start as NaN patterns; rows past past+q_len stay NaN and sit
    in the same KV tile as valid rows (q_len not a multiple of 64)."""
    case = Case(700, 2, 150, (8, 2, 4), [20, 0], S=400, garbage=0x7FC0)
    check_case(api, oracle, case, "garbage tail")


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
def test_paged_cache_equals_contiguous_bitwise(api, oracle, page_size):
    case = Case(800, 2, 200, (8, 2, 4), [50, 0], S=384)
    out_c, lse_c, st, _, _ = run_gpu(api, case)
    assert st == 0
    ref, lse_ref, k_ref, v_ref = run_oracle(oracle, case)
    out_p, lse_p, st, k_after, v_after = run_gpu(api, case, paged=page_size)
    assert st == 0
    assert np.array_equal(out_p, out_c) and np.array_equal(lse_p, lse_c)
    for b in range(2):
        n = int(case.past[b]) + case.q_len
        assert np.array_equal(k_after[b, :, :n], k_ref[b, :, :n]) and np.array_equal(v_after[b, :, :n], v_ref[b, :, :n])
    check_bf16(out_p, ref, f"paged {page_size}")


@pytest.mark.parametrize("scale", [-0.0884, 0.0])
def test_non_positive_scale_matches_the_oracle(api, oracle, scale):
    """A negative scale turns the softmax towards the smallest inner products; zero makes it uniform.  Either must give
    what the definition gives (the tensor-core kernel orders raw scores, so these run on the generic kernel)."""
    case = Case(950, 1, 200, (8, 2, 4), [30])
    case.scale = scale
    check_case(api, oracle, case, f"scale={scale}")
    assert api.last_prefill_kernel() == 1


def test_bf16_output(api, oracle):
    case = Case(900, 1, 200, (8, 2, 4), [0])
    ref, _, _, _ = run_oracle(oracle, case)
    out, _, st, _, _ = run_gpu(api, case, out_dtype=torch.bfloat16)
    assert st == 0
    check_bf16(out, ref, "bf16 out")


def test_prefill_rows_match_decode_kernel(api, oracle):
    """Prefill row i and a decode call at length past + i + 1 on the updated cache agree within tolerance."""
    case = Case(1000, 1, 192, (8, 2, 4), [64])
    out, _, st, k_after, v_after = run_gpu(api, case)
    assert st == 0
    dev = "cuda"
    k, v = W.to_torch(k_after, dev), W.to_torch(v_after, dev)
    for i in (0, 63, 191):
        lens = torch.tensor([64 + i + 1], dtype=torch.int32, device=dev)
        cache = api.KVCache(k, v, lens, case.S, k_strides=case.strides(2), v_strides=case.strides(4), num_blocks=1)
        q = W.to_torch(np.ascontiguousarray(case.q[:, i]), dev)
        dec = api.diffqkv_decode(q, cache, 2, 4, case.scale, out_dtype=torch.float32)
        torch.cuda.synchronize()
        assert np.abs(dec.cpu().numpy().astype(np.float64) - out[:, i]).max() <= 2e-2


def test_config4_full_size_sampled_rows(api, oracle):
    """Config 4: batch 2, 8192 tokens, 32/4/8 heads, d 128, bf16, K and V N(0,1), direct N(0,1) queries; the whole
    problem on the GPU, a sample of (sequence, row, head) outputs through the oracle."""
    cfg = W.CFG4
    heads = (cfg.n_q, cfg.n_k, cfg.n_v)
    case = Case(cfg.seed + 5, cfg.batch, cfg.seq, heads, [0, 0])
    g = np.random.Generator(np.random.Philox(key=4242))
    rows_i = np.concatenate([[0, 1, 63, 64, 127, 128, 255, 256, 4095, 4096, 8190, 8191], g.integers(0, cfg.seq, 40)])
    rows = np.array([(b, i, h) for b in range(cfg.batch) for i in rows_i for h in g.integers(0, cfg.n_q, 6)],
                    dtype=np.int32)
    ref, lse_ref, _, _ = run_oracle(oracle, case, rows=rows)
    out, lse, st, _, _ = run_gpu(api, case)
    assert st == 0
    got = out[rows[:, 0], rows[:, 1], rows[:, 2]]
    check_bf16(got, ref, "cfg4 sampled rows")
    check_lse(lse[rows[:, 0], rows[:, 1], rows[:, 2]], lse_ref, 2e-2, "cfg4 lse")
    assert np.isfinite(out).all()


@pytest.mark.parametrize("q_len,past", [(1, [0, 0]), (129, [0, 70]), (300, [257, 5]), (700, [0, 0])])
def test_head_dimension_64_on_the_tensor_cores(api, oracle, q_len, past):
    """SIGMA-1.5B's head size: the same kernel with half-width tiles."""
    check_case(api, oracle, Case(800 + q_len, 2, q_len, (8, 2, 4), past, d=64), f"d=64 q_len={q_len} past={past}")
    assert api.last_prefill_kernel() == 2


@pytest.mark.parametrize("q_len,past", [(1, [0, 0]), (129, [0, 70]), (300, [257, 5]), (700, [0, 0])])
def test_half_width_keys_on_the_tensor_cores(api, oracle, q_len, past):
    """d_qk = 64 with d_v = 128 (keys cached at half the value width): half-width Q and K tiles, full-width V."""
    check_case(api, oracle, Case(870 + q_len, 2, q_len, (8, 2, 4), past, d=64, d_v=128),
               f"d 64/128 q_len={q_len} past={past}")
    assert api.last_prefill_kernel() == 2


@pytest.mark.parametrize("page", [16, 128])
def test_half_width_keys_paged(api, oracle, page):
    check_case(api, oracle, Case(880 + page, 2, 200, (32, 4, 16), [100, 0], d=64, d_v=128), f"d 64/128 page={page}",
               paged=page)
    assert api.last_prefill_kernel() == 2


@pytest.mark.parametrize("page", [16, 128])
def test_head_dimension_64_paged(api, oracle, page):
    check_case(api, oracle, Case(850 + page, 2, 200, (32, 4, 16), [100, 0], d=64), f"d=64 page={page}", paged=page)


def test_argument_errors(api):
    dev = "cuda"
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device=dev)
    lens = torch.zeros(1, dtype=torch.int32, device=dev)
    cache = api.KVCache(z(1, 2, 64, 64), z(1, 2, 64, 64), lens, 64)
    with pytest.raises(api.DiffQKVError) as e:  # 3 query heads cannot share 2 K heads
        api.diffqkv_prefill(z(1, 8, 3, 64), z(1, 8, 2, 64), z(1, 8, 1, 64), cache, 0.125)
    assert e.value.status == api.ERR_INVALID_ARG
    cache = api.KVCache(z(1, 2, 64, 128), z(1, 2, 64, 128), lens, 64)
    with pytest.raises(api.DiffQKVError) as e:  # more new tokens than the cache can hold
        api.diffqkv_prefill(z(1, 100, 4, 128), z(1, 100, 2, 128), z(1, 100, 2, 128), cache, 0.1)
    assert e.value.status == api.ERR_INVALID_ARG
