"""GPU parity at the sizes, and through the code paths, that the benchmark times.

The prefill configuration as it is defined: hidden states N(0, 0.02) of width 2048 for 2 x 8192 tokens go through the
augmented-Q projection (appendix attention listing: q_proj, then q_down_proj(act(q_gate_proj) * q_up_proj)) on the
tensor cores, and that bf16 q, with K and V N(0, 1), goes through the cache update and the causal attention.  At
16 384 rows every persistent block of the projection kernel walks about 14 output tiles (both tensor-memory
accumulators several times over, the shared-memory ring across tile boundaries); rows are sampled from first, later
and last tiles and compared with the float64 oracle.  The attention is then compared with the oracle fed the very
same bf16 q bits, so that the comparison isolates the attention step, and the cache must match bit for bit.

The weight-streaming kernel that serves up to 64 rows is run at the same widths (2048 -> 4096 -> 3072 -> 4096, eight
512-column stages per weight row, more than one item per block), every element against the oracle's chain.
"""
import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_lse, check_proj

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


@pytest.fixture(scope="module")
def cfg4(api):
    """Config 4's inputs on the host and its augmented queries computed on the GPU (full size)."""
    inp = W.make_prefill_inputs(W.CFG4)
    dev = "cuda"
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    q = api.diffqkv_augq(W.to_torch(inp.h, dev), W.to_torch(inp.W_Q, dev), W.to_torch(inp.W_gate, dev),
                         W.to_torch(inp.W_up, dev), W.to_torch(inp.W_down, dev), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return inp, q


def test_config4_augq_full_size_sampled_rows(api, oracle, cfg4):
    inp, q = cfg4
    cfg = inp.cfg
    T = cfg.batch * cfg.seq
    assert q.shape == (T, cfg.n_q * cfg.d_qk)
    g = np.random.Generator(np.random.Philox(key=4141))
    # first tile, tile edges, the rows where a wave of 148 tiles ends (16 column tiles per 128 rows in the plain
    # products, 24 in the fused gate/up product), rows that only a block's 3rd or later tile reaches, the last tile
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 129, 767, 768, 1151, 1152, 1183, 1184, 2431, 2432, 8191, 8192,
                                      12000, 12287, 12288, 16255, 16256, 16383], g.integers(2432, T, 8)])).astype(np.int64)
    ref = oracle.augq(inp.h, inp.W_Q, inp.W_gate, inp.W_up, inp.W_down, rows=rows)
    got = q[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    check_proj(got, ref, "cfg4 aug-Q at 16384 rows")
    assert torch.isfinite(q.float()).all()


def test_config4_prefill_on_the_augmented_queries(api, oracle, cfg4):
    """h ~ N(0, 0.02) makes tiny queries and a nearly uniform softmax over up to 8192 tokens: late rows are close to
    the mean of the visible V rows, so besides the stated tolerances every sampled row is also held to 1e-2 of its
    own largest reference value."""
    inp, q2d = cfg4
    cfg = inp.cfg
    dev = "cuda"
    B, S, n_q, n_k, n_v, d = cfg.batch, cfg.seq, cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk
    q = q2d.view(B, S, n_q, d)
    q_bits = q.view(torch.uint16).cpu().numpy()
    past = np.zeros(B, np.int32)
    k = torch.zeros((B, n_k, S, d), dtype=torch.bfloat16, device=dev)
    v = torch.zeros((B, n_v, S, d), dtype=torch.bfloat16, device=dev)
    cache = api.KVCache(k, v, torch.from_numpy(past).to(dev), S)
    lse = torch.full((B, S, n_q), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = api.diffqkv_prefill(q, W.to_torch(inp.k_new, dev), W.to_torch(inp.v_new, dev), cache, cfg.scale, lse=lse,
                              dev_status=status, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert api.last_prefill_kernel() == 2
    # oracle: same cache update, then attention on the GPU's own bf16 queries
    k_ref = np.zeros((B, n_k, S, d), np.uint16)
    v_ref = np.zeros((B, n_v, S, d), np.uint16)
    oc = oracle.Cache(k_ref, v_ref, (n_k * S * d, S * d, d), (n_v * S * d, S * d, d), past)
    oracle.cache_append(inp.k_new, inp.v_new, oc)
    assert np.array_equal(k.view(torch.uint16).cpu().numpy(), k_ref), "K cache differs"
    assert np.array_equal(v.view(torch.uint16).cpu().numpy(), v_ref), "V cache differs"
    g = np.random.Generator(np.random.Philox(key=4343))
    rows_i = np.concatenate([[0, 1, 63, 64, 127, 128, 255, 256, 257, 4095, 4096, 8063, 8064, 8190, 8191],
                             g.integers(0, S, 33)])
    rows = np.array([(b, i, h) for b in range(B) for i in rows_i for h in g.integers(0, n_q, 6)], dtype=np.int32)
    ref, lse_ref = oracle.prefill(q_bits, past, oc, n_k, n_v, d, cfg.scale, rows=rows)
    o = out.cpu().numpy().astype(np.float64)
    got = o[rows[:, 0], rows[:, 1], rows[:, 2]]
    check_bf16(got, ref, "cfg4 prefill on aug-Q queries")
    check_lse(lse.cpu().numpy().astype(np.float64)[rows[:, 0], rows[:, 1], rows[:, 2]], lse_ref, 2e-2, "cfg4 lse")
    per_row = np.abs(got - ref).max(axis=1) / np.abs(ref).max(axis=1)
    assert per_row.max() <= 1e-2, f"worst row: err / max|ref row| = {per_row.max():.3e}"
    assert np.isfinite(o).all()


def _tables(oracle, pos, d, theta):
    c, s = oracle.rope_tables(pos, d, theta)
    return (torch.from_numpy(c.astype(np.float32)).cuda().contiguous(),
            torch.from_numpy(s.astype(np.float32)).cuda().contiguous())


@pytest.mark.parametrize("T", [1, 4, 16, 64])
def test_weight_streaming_kernel_at_config4_widths(api, oracle, T):
    """Decode row counts at the prefill configuration's widths, rotary embedding on: the aug-Q chain, the key and value
    projections, and the fused front end of a decode step, every element against the oracle's chain."""
    cfg = W.CFG4
    n_q, n_k, n_v, d, theta = cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, 500000.0
    d_q0 = n_q * d
    dev = "cuda"
    h = W.normal(9100 + T, (T, cfg.d_model), std=1.0)
    ws = [W.normal(9001, (d_q0, cfg.d_model), std=cfg.d_model ** -0.5),
          W.normal(9002, (cfg.d_aug, d_q0), std=d_q0 ** -0.5),
          W.normal(9003, (cfg.d_aug, d_q0), std=d_q0 ** -0.5),
          W.normal(9004, (d_q0, cfg.d_aug), std=cfg.d_aug ** -0.5)]
    w_k = W.normal(9005, (n_k * d, cfg.d_model), std=cfg.d_model ** -0.5)
    w_v = W.normal(9006, (n_v * d, cfg.d_model), std=cfg.d_model ** -0.5)
    S = 96
    lens = ((np.arange(T) * 29 + 5) % (S - 1)).astype(np.int32)
    pos = lens.astype(np.int64)
    cos, sin = _tables(oracle, pos, d, theta)
    th, tw = W.to_torch(h, dev), [W.to_torch(w, dev) for w in ws]
    tk, tv = W.to_torch(w_k, dev), W.to_torch(w_v, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    q_ref = oracle.rope(oracle.augq(h, *ws).reshape(T, n_q, d), pos, theta).reshape(T, d_q0)
    k_plain = oracle.linear(h, w_k)
    k_ref = oracle.rope(k_plain.reshape(T, n_k, d), pos, theta).reshape(T, n_k * d)
    v_ref = oracle.linear(h, w_v)

    q = api.diffqkv_augq_rope(th, *tw, d, cos, sin, dev_status=status)
    kp = api.diffqkv_project(th, tk, dev_status=status)
    kr = api.diffqkv_project(th, tk, d, cos, sin, dev_status=status)
    vp = api.diffqkv_project(th, tv, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)  # noqa: E731
    check_proj(f64(q), q_ref, f"aug-Q + rope, {T} rows")
    check_proj(f64(kp), k_plain, f"key projection, {T} rows")
    check_proj(f64(kr), k_ref, f"rotated key projection, {T} rows")
    check_proj(f64(vp), v_ref, f"value projection, {T} rows")

    # the fused front end of a decode step: q as above, k and v written straight into the cache row of the new token
    kc = W.normal(9007, (T, n_k, S, d))
    vc = W.normal(9008, (T, n_v, S, d))
    k_dev, v_dev = W.to_torch(kc, dev), W.to_torch(vc, dev)
    cache = api.KVCache(k_dev, v_dev, torch.from_numpy(lens).to(dev), S)
    q2 = api.diffqkv_decode_frontend(th, *tw, tk, tv, cache, n_q, d, d, cos, sin, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_proj(f64(q2).reshape(T, d_q0), q_ref, f"front end q, {T} rows")
    k_after, v_after = k_dev.view(torch.uint16).cpu().numpy(), v_dev.view(torch.uint16).cpu().numpy()
    k_row = np.stack([k_after[b, :, lens[b]] for b in range(T)])  # [T, n_k, d]
    v_row = np.stack([v_after[b, :, lens[b]] for b in range(T)])
    check_proj(W.as_f64(k_row).reshape(T, n_k * d), k_ref, f"front end K row, {T} rows")
    check_proj(W.as_f64(v_row).reshape(T, n_v * d), v_ref, f"front end V row, {T} rows")
    for b in range(T):  # nothing but the new token's row moved
        k_after[b, :, lens[b]] = kc[b, :, lens[b]]
        v_after[b, :, lens[b]] = vc[b, :, lens[b]]
    assert np.array_equal(k_after, kc) and np.array_equal(v_after, vc)


def _rows_of_every_tile(T, seed):
    g = np.random.Generator(np.random.Philox(key=seed))
    rows = []
    for m0 in range(0, T, 128):
        hi = min(T, m0 + 128)
        rows += [m0, hi - 1, int(g.integers(m0, hi))]
    return np.unique(np.array(rows, dtype=np.int64))


@pytest.mark.parametrize("rotate", [False, True])
def test_projection_kernel_blocks_walk_many_tiles(api, oracle, rotate):
    """4000 x 4096 outputs are 32 x 16 = 512 tiles of 128 x 256: every persistent block walks three or four, so both
    accumulators are used a second time; six 64-column K blocks per tile make the 4-stage ring wrap inside and across
    tiles.  Three rows of every row tile, all columns, against the oracle (rows are independent in a projection)."""
    T, d_in, heads, d, theta = 4000, 384, 32, 128, 50000.0
    x = W.normal(9201, (T, d_in))
    w = W.normal(9202, (heads * d, d_in), std=d_in ** -0.5)
    pos = np.random.Generator(np.random.Philox(key=9203)).integers(0, 100000, size=T)
    rows = _rows_of_every_tile(T, 9204)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if rotate:
        cos, sin = _tables(oracle, pos, d, theta)
        y = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"), d, cos, sin, dev_status=status)
    else:
        y = api.diffqkv_project(W.to_torch(x, "cuda"), W.to_torch(w, "cuda"), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.linear(np.ascontiguousarray(x[rows]), w)
    if rotate:
        ref = oracle.rope(ref.reshape(len(rows), heads, d), pos[rows], theta).reshape(len(rows), heads * d)
    got = y[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    check_proj(got, ref, f"projection over 512 tiles, rotate={rotate}")


def test_fused_gate_up_kernel_blocks_walk_many_tiles(api, oracle):
    """The fused silu-gate product with 32 x 16 = 512 tiles of 128 x (128 gate + 128 up) columns, and the two plain
    products around it, at 4000 rows."""
    T, d_model, d_q0, d_aug, d_out = 4000, 384, 640, 2048, 1024
    h = W.normal(9301, (T, d_model), std=1.0)
    ws = [W.normal(9302, (d_q0, d_model), std=d_model ** -0.5), W.normal(9303, (d_aug, d_q0), std=d_q0 ** -0.5),
          W.normal(9304, (d_aug, d_q0), std=d_q0 ** -0.5), W.normal(9305, (d_out, d_aug), std=d_aug ** -0.5)]
    rows = _rows_of_every_tile(T, 9306)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q = api.diffqkv_augq(W.to_torch(h, "cuda"), *(W.to_torch(w, "cuda") for w in ws), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.augq(h, *ws, rows=rows)
    got = q[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    check_proj(got, ref, "aug-Q over 512 fused tiles")


def test_fold_of_the_k_layer_at_config4_rows(api):
    """diffqkv_fold_k_up over config 4's 16 384 query rows of 32 heads (every block of the tensor-core kernel walks
    several 128-row tiles and the last block a ragged one: T is taken one row short): sampled rows, every head and
    channel, against the float64 product (Section 2: K brought to the query width by a feed-forward layer)."""
    n_q, n_k, d_q, d_k, T = 32, 4, 128, 64, 16383
    q, w = W.normal(9101, (T, n_q, d_q)), W.normal(9102, (n_k, d_q, d_k), std=d_k ** -0.5)
    out = torch.full((T, n_q, d_k), float("nan"), dtype=torch.bfloat16, device="cuda")
    api.diffqkv_fold_k_up(W.to_torch(q, "cuda"), W.to_torch(w, "cuda"), out=out)
    torch.cuda.synchronize()
    rows = np.unique(np.concatenate([np.arange(0, 40), np.arange(8000, 8040), np.arange(T - 40, T),
                                     np.random.default_rng(5).integers(0, T, 200)]))
    got = out[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    assert not torch.isnan(out.float()).any(), "rows left unwritten"
    qf, wf = W.as_f64(q[rows]), W.as_f64(w)
    for h in range(n_q):
        ref = qf[:, h] @ wf[h // (n_q // n_k)]
        err = np.abs(got[:, h] - ref)
        assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 2e-5 * np.abs(ref).max()), (h, err.max())
