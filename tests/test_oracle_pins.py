"""Pins of the float64 oracle against things other than itself.

Each test ties one part of ``oracle/diffqkv_oracle.c`` to a fact the paper or the
mathematics fixes: a library routine in a special case, a closed form, an invariant, a
pure-Python brute force, or a value the paper prints.  No GPU is involved.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _contig_cache(oracle, k, v, seqlens):
    b, n_k, S, d_qk = k.shape
    _, n_v, _, d_v = v.shape
    return oracle.Cache(k, v, (n_k * S * d_qk, S * d_qk, d_qk), (n_v * S * d_v, S * d_v, d_v),
                        np.ascontiguousarray(seqlens, dtype=np.int32))


def _rand(seed, shape, dtype="f32"):
    return W.normal(seed, shape, dtype=dtype)


# --------------------------------------------------------------------------- whole attention
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_equal_heads_is_textbook_mha(oracle, dtype):
    """n_q = n_k = n_v reduces to standard multi-head attention (Appendix B.1): compare with
    torch's softmax and matmul in float64."""
    b, n, S, d = 3, 4, 37, 16
    q = _rand(1, (b, n, d), dtype)
    k = _rand(2, (b, n, S, d), dtype)
    v = _rand(3, (b, n, S, d), dtype)
    lens = np.array([37, 1, 20], dtype=np.int32)
    scale = 0.37
    out, lse = oracle.decode(q, _contig_cache(oracle, k, v, lens), n, n, n, d, d, scale)
    tq, tk, tv = (torch.from_numpy(W.as_f64(a)) for a in (q, k, v))
    for bi in range(b):
        L = int(lens[bi])
        s = torch.einsum("hd,hjd->hj", tq[bi], tk[bi, :, :L]) * scale
        ref = torch.einsum("hj,hjd->hd", torch.softmax(s, dim=-1), tv[bi, :, :L])
        assert np.allclose(out[bi], ref.numpy(), rtol=0, atol=1e-13)
        assert np.allclose(lse[bi], torch.logsumexp(s, dim=-1).numpy(), rtol=0, atol=1e-12)


def test_bf16_widening_is_exact(oracle):
    """A single visible token returns its V row exactly; bf16 bits widen as torch widens them."""
    v = _rand(5, (1, 2, 3, 8), "bf16")
    k = _rand(6, (1, 2, 3, 8), "bf16")
    q = _rand(7, (1, 4, 8), "bf16")
    out, lse = oracle.decode(q, _contig_cache(oracle, k, v, [1]), 4, 2, 2, 8, 8, 1.0)
    tv = torch.from_numpy(v).view(torch.bfloat16).double().numpy()
    for h in range(4):
        assert np.array_equal(out[0, h], tv[0, h // 2, 0])


# --------------------------------------------------------------------------- head map
def _replicate_adjacent(x, n_rep):
    """The paper's KV Group Sharing listing: expand then reshape puts the copies of one head
    next to each other (head h of the result is head h // n_rep of the input)."""
    t = torch.from_numpy(x)
    b, n, s, d = t.shape
    return t[:, :, None].expand(b, n, n_rep, s, d).reshape(b, n * n_rep, s, d).contiguous().numpy()


@pytest.mark.parametrize("n_q,n_k,n_v", [(16, 2, 4), (32, 4, 16), (8, 1, 8), (12, 6, 2), (8, 4, 1)])
def test_group_sharing_identity(oracle, n_q, n_k, n_v):
    """DiffQKV on the compact cache == GQA on the cache with the scarcer side replicated
    the way the paper's own listing replicates it.  Pins the direction and order of Eq. (idx)."""
    b, S, d = 2, 19, 8
    q = _rand(11, (b, n_q, d))
    k = _rand(12, (b, n_k, S, d))
    v = _rand(13, (b, n_v, S, d))
    lens = [19, 7]
    out, lse = oracle.decode(q, _contig_cache(oracle, k, v, lens), n_q, n_k, n_v, d, d, 0.5)
    if n_k < n_v:
        k2, v2 = _replicate_adjacent(k, n_v // n_k), v
    else:
        k2, v2 = k, _replicate_adjacent(v, n_k // n_v)
    n2 = max(n_k, n_v)
    out2, lse2 = oracle.decode(q, _contig_cache(oracle, k2, v2, lens), n_q, n2, n2, d, d, 0.5)
    assert np.allclose(out, out2, rtol=0, atol=1e-14)
    assert np.allclose(lse, lse2, rtol=0, atol=1e-14)
    # the same GQA result must come from the textbook formula with the map h -> h // (n_q / n2)
    tq, tk, tv = (torch.from_numpy(W.as_f64(a)) for a in (q, k2, v2))
    g = n_q // n2
    for bi, L in enumerate(lens):
        for h in range(n_q):
            s = (tk[bi, h // g, :L] @ tq[bi, h]) * 0.5
            ref = torch.softmax(s, 0) @ tv[bi, h // g, :L]
            assert np.allclose(out2[bi, h], ref.numpy(), rtol=0, atol=1e-13)


def test_interleaved_grouping_would_differ(oracle):
    """The identity above has teeth: replicating K in interleaved order (h % n_k) gives another result."""
    b, S, d, n_q, n_k, n_v = 1, 9, 4, 8, 2, 4
    q, k, v = _rand(21, (b, n_q, d)), _rand(22, (b, n_k, S, d)), _rand(23, (b, n_v, S, d))
    out, _ = oracle.decode(q, _contig_cache(oracle, k, v, [S]), n_q, n_k, n_v, d, d, 1.0)
    k_inter = np.ascontiguousarray(np.tile(k, (1, n_v // n_k, 1, 1)))
    out2, _ = oracle.decode(q, _contig_cache(oracle, k_inter, v, [S]), n_q, n_v, n_v, d, d, 1.0)
    assert np.abs(out - out2).max() > 1e-3


def test_head_index_formula():
    """Eq. (idx) with integer floor equals h // (n_q / n_i) whenever n_i divides n_q."""
    for n_q in (1, 2, 4, 8, 12, 16, 32):
        for n_i in [d for d in range(1, n_q + 1) if n_q % d == 0]:
            for h in range(n_q):
                assert (h * n_i) // n_q == h // (n_q // n_i)


def test_indivisible_heads_rejected(oracle):
    q, k, v = _rand(1, (1, 6, 4)), _rand(2, (1, 4, 3, 4)), _rand(3, (1, 3, 3, 4))
    with pytest.raises(ValueError):
        oracle.decode(q, _contig_cache(oracle, k, v, [3]), 6, 4, 3, 4, 4, 1.0)


# --------------------------------------------------------------------------- softmax weights
def test_identical_keys_give_mean_of_v(oracle):
    b, n_q, n_k, n_v, S, d = 2, 8, 2, 4, 33, 8
    q = _rand(31, (b, n_q, d))
    krow = _rand(32, (b, n_k, 1, d))
    k = np.ascontiguousarray(np.broadcast_to(krow, (b, n_k, S, d)))
    v = _rand(33, (b, n_v, S, d))
    lens = [33, 10]
    scale = 0.25
    out, lse = oracle.decode(q, _contig_cache(oracle, k, v, lens), n_q, n_k, n_v, d, d, scale)
    for bi, L in enumerate(lens):
        for h in range(n_q):
            mean = W.as_f64(v[bi, h // 2, :L]).mean(axis=0)
            s = scale * float(W.as_f64(q[bi, h]) @ W.as_f64(krow[bi, h // 4, 0]))
            assert np.allclose(out[bi, h], mean, rtol=0, atol=1e-14)
            assert abs(lse[bi, h] - (s + math.log(L))) < 1e-12


def test_constant_v_and_convex_hull(oracle):
    b, n_q, n_k, n_v, S, d = 1, 4, 1, 2, 50, 8
    q, k = _rand(41, (b, n_q, d)), _rand(42, (b, n_k, S, d))
    ones = np.ones((b, n_v, S, d), dtype=np.float32)
    out, _ = oracle.decode(q, _contig_cache(oracle, k, ones, [S]), n_q, n_k, n_v, d, d, 1.0)
    assert np.allclose(out, 1.0, rtol=0, atol=1e-15)
    v = _rand(43, (b, n_v, S, d))
    out, _ = oracle.decode(q, _contig_cache(oracle, k, v, [S]), n_q, n_k, n_v, d, d, 1.0)
    for h in range(n_q):
        vv = W.as_f64(v[0, h // 2])
        assert np.all(out[0, h] <= vv.max(axis=0) + 1e-15) and np.all(out[0, h] >= vv.min(axis=0) - 1e-15)


def test_dominant_key_returns_its_v_row(oracle):
    """One key equal to c*q with a large c: the output is that V row up to (len-1) e^-gap."""
    n_q, n_k, n_v, S, d = 4, 2, 4, 40, 8
    q = _rand(51, (1, n_q, d))
    k = (0.01 * _rand(52, (1, n_k, S, d))).astype(np.float32)
    v = _rand(53, (1, n_v, S, d))
    star = 17
    # K head hk serves query heads 2hk and 2hk+1: make the key dominant for head 2hk
    for hk in range(n_k):
        k[0, hk, star] = 30.0 * q[0, 2 * hk]
    out, _ = oracle.decode(q, _contig_cache(oracle, k, v, [S]), n_q, n_k, n_v, d, d, 1.0)
    for hk in range(n_k):
        h = 2 * hk
        s = W.as_f64(k[0, hk]) @ W.as_f64(q[0, h])
        gap = s[star] - np.max(np.delete(s, star))
        assert gap > 20
        bound = (S - 1) * math.exp(-gap) * 2 * np.abs(W.as_f64(v[0, h])).max()
        assert np.abs(out[0, h] - W.as_f64(v[0, h, star])).max() <= bound + 1e-15


def test_two_token_closed_form(oracle):
    """q = e0, keys a*e0 and b*e0: weights are the logistic function of scale*(a-b)."""
    a, b_, scale = 1.5, -0.5, 0.5
    q = np.array([[[1.0, 0.0]]], dtype=np.float32)
    k = np.array([[[[a, 0.3], [b_, -0.7]]]], dtype=np.float32)
    v = np.array([[[[2.0, 4.0], [-6.0, 8.0]]]], dtype=np.float32)
    out, lse = oracle.decode(q, _contig_cache(oracle, k, v, [2]), 1, 1, 1, 2, 2, scale)
    w0 = 1.0 / (1.0 + math.exp(-scale * (a - b_)))
    assert np.allclose(out[0, 0], [w0 * 2.0 + (1 - w0) * -6.0, w0 * 4.0 + (1 - w0) * 8.0], rtol=0, atol=1e-15)
    assert abs(lse[0, 0] - math.log(math.exp(scale * a) + math.exp(scale * b_))) < 1e-15


def test_empty_sequence(oracle):
    q, k, v = _rand(1, (2, 2, 4)), _rand(2, (2, 1, 5, 4)), _rand(3, (2, 2, 5, 4))
    out, lse = oracle.decode(q, _contig_cache(oracle, k, v, [0, 5]), 2, 1, 2, 4, 4, 1.0)
    assert np.all(out[0] == 0.0) and np.all(np.isneginf(lse[0]))
    assert np.all(np.isfinite(out[1])) and np.all(np.isfinite(lse[1]))


# --------------------------------------------------------------------------- brute force
def _brute(q, k, v, lens, n_q, n_k, n_v, scale):
    """Pure-Python restatement of Section 2's formulas, one scalar at a time."""
    b = len(lens)
    d_qk, d_v = len(q[0][0]), len(v[0][0][0])
    out = [[[0.0] * d_v for _ in range(n_q)] for _ in range(b)]
    for bi in range(b):
        for h in range(n_q):
            hk, hv = (h * n_k) // n_q, (h * n_v) // n_q
            scores = []
            for j in range(lens[bi]):
                scores.append(scale * sum(q[bi][h][c] * k[bi][hk][j][c] for c in range(d_qk)))
            z = sum(math.exp(s) for s in scores)
            for j in range(lens[bi]):
                a = math.exp(scores[j]) / z
                for c in range(d_v):
                    out[bi][h][c] += a * v[bi][hv][j][c]
    return np.array(out)


def test_brute_force_all_divisor_pairs(oracle):
    S, d_qk, d_v = 7, 3, 4
    for n_q in (1, 2, 4):
        divs = [x for x in range(1, n_q + 1) if n_q % x == 0]
        for n_k, n_v in itertools.product(divs, divs):
            q = _rand(100 + n_q, (2, n_q, d_qk))
            k = _rand(200 + n_k, (2, n_k, S, d_qk))
            v = _rand(300 + n_v, (2, n_v, S, d_v))
            lens = [7, 3]
            out, _ = oracle.decode(q, _contig_cache(oracle, k, v, lens), n_q, n_k, n_v, d_qk, d_v, 0.6)
            ref = _brute(W.as_f64(q).tolist(), W.as_f64(k).tolist(), W.as_f64(v).tolist(), lens,
                         n_q, n_k, n_v, 0.6)
            assert np.allclose(out, ref, rtol=0, atol=1e-13), (n_q, n_k, n_v)


# --------------------------------------------------------------------------- splits / combine
def test_split_then_combine_equals_unsplit(oracle):
    b, n_q, n_k, n_v, S, d = 2, 8, 2, 4, 100, 16
    q, k, v = _rand(61, (b, n_q, d)), _rand(62, (b, n_k, S, d)), _rand(63, (b, n_v, S, d))
    cache = _contig_cache(oracle, k, v, [100, 41])
    full, lse_full = oracle.decode(q, cache, n_q, n_k, n_v, d, d, 0.3)
    for cuts in ([0, 100], [0, 1, 2, 50, 100], [0, 33, 33, 64, 97, 100], [0, 41, 60, 100]):
        op, lp = oracle.decode_splits(q, cache, n_q, n_k, n_v, d, d, 0.3, cuts)
        out, lse = oracle.combine(op, lp)
        assert np.allclose(out, full, rtol=0, atol=1e-13)
        assert np.allclose(lse, lse_full, rtol=0, atol=1e-12)


def test_combine_closed_forms(oracle):
    """Equal lse: plain average. One split -inf: skipped. All -inf: zero and -inf."""
    o = np.array([[[1.0, 2.0], [3.0, 6.0]]])
    out, lse = oracle.combine(o, np.array([[0.7, 0.7]]))
    assert np.allclose(out, [[2.0, 4.0]], atol=1e-15) and abs(lse[0] - (0.7 + math.log(2))) < 1e-15
    out, lse = oracle.combine(o, np.array([[-np.inf, 0.2]]))
    assert np.array_equal(out, [[3.0, 6.0]]) and lse[0] == 0.2
    out, lse = oracle.combine(o, np.array([[-np.inf, -np.inf]]))
    assert np.all(out == 0) and np.isneginf(lse[0])
    # weights exp(lse_s) / sum: lse = log 1, log 3 -> 1/4, 3/4
    out, lse = oracle.combine(o, np.array([[0.0, math.log(3.0)]]))
    assert np.allclose(out, [[2.5, 5.0]], atol=1e-15) and abs(lse[0] - math.log(4.0)) < 1e-15


# --------------------------------------------------------------------------- paging
@pytest.mark.parametrize("page_size", [1, 4, 16])
def test_paging_is_pure_addressing(oracle, page_size):
    cfg = W.DecodeConfig("t", batch=3, n_q=8, n_k=2, n_v=4, d_qk=8, d_v=8, kv_len=45, dtype="bf16", seed=77)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([45, 16, 1], dtype=np.int32))
    ref, lse_ref = oracle.decode(inp.q, oracle.Cache(inp.k, inp.v, inp.k_strides, inp.v_strides, inp.seqlens),
                                 8, 2, 4, 8, 8, cfg.scale)
    for identity in (True, False):
        pg = W.paginate(inp, page_size, seed=5, identity=identity)
        cache = oracle.Cache(pg.k, pg.v, pg.k_strides, pg.v_strides, pg.seqlens, pg.page_table, page_size)
        out, lse = oracle.decode(pg.q, cache, 8, 2, 4, 8, 8, cfg.scale)
        assert np.array_equal(out, ref) and np.array_equal(lse, lse_ref)
    # the shuffled table really is a permutation with distinct pages
    assert len(np.unique(pg.page_table)) == pg.page_table.size


def test_token_major_strides(oracle):
    """The (b, s, n_h, d_h) layout of Section 3.1 read through explicit strides equals head-major."""
    b, n_q, n_k, n_v, S, d = 2, 4, 2, 4, 11, 8
    q, k, v = _rand(71, (b, n_q, d)), _rand(72, (b, n_k, S, d)), _rand(73, (b, n_v, S, d))
    ref, _ = oracle.decode(q, _contig_cache(oracle, k, v, [11, 6]), n_q, n_k, n_v, d, d, 1.0)
    kt = np.ascontiguousarray(k.transpose(0, 2, 1, 3))
    vt = np.ascontiguousarray(v.transpose(0, 2, 1, 3))
    cache = oracle.Cache(kt, vt, (S * n_k * d, d, n_k * d), (S * n_v * d, d, n_v * d),
                         np.array([11, 6], dtype=np.int32))
    out, _ = oracle.decode(q, cache, n_q, n_k, n_v, d, d, 1.0)
    assert np.array_equal(out, ref)


# --------------------------------------------------------------------------- prefill
def test_prefill_rows_equal_decode_and_cache_append(oracle):
    b, T, n_q, n_k, n_v, d, S = 2, 9, 4, 2, 4, 8, 16
    k = np.zeros((b, n_k, S, d), dtype=np.uint16)
    v = np.zeros((b, n_v, S, d), dtype=np.uint16)
    past = np.array([0, 5], dtype=np.int32)
    k[1, :, :5] = _rand(80, (n_k, 5, d), "bf16")
    v[1, :, :5] = _rand(81, (n_v, 5, d), "bf16")
    q = _rand(82, (b, T, n_q, d), "bf16")
    k_new, v_new = _rand(83, (b, T, n_k, d), "bf16"), _rand(84, (b, T, n_v, d), "bf16")
    cache = _contig_cache(oracle, k, v, past)
    oracle.cache_append(k_new, v_new, cache)
    for bi in range(b):
        p = int(past[bi])
        assert np.array_equal(k[bi, :, p:p + T], k_new[bi].transpose(1, 0, 2))
        assert np.array_equal(v[bi, :, p:p + T], v_new[bi].transpose(1, 0, 2))
    assert not k[0, :, T:].any() and not v[1, :, 5 + T:].any()
    out, lse = oracle.prefill(q, past, cache, n_k, n_v, d, 0.4)
    # row 0 with no past sees exactly one token: its V row, bit for bit
    for h in range(n_q):
        assert np.array_equal(out[0, 0, h], W.as_f64(v_new[0, 0, h]))
    for i in range(T):
        lens = past + i + 1
        dec, dlse = oracle.decode(np.ascontiguousarray(q[:, i]), _contig_cache(oracle, k, v, lens),
                                  n_q, n_k, n_v, d, d, 0.4)
        assert np.array_equal(out[:, i], dec) and np.array_equal(lse[:, i], dlse)
    rows = np.array([[1, 8, 3], [0, 0, 0], [1, 2, 1]], dtype=np.int32)
    o2, l2 = oracle.prefill(q, past, cache, n_k, n_v, d, 0.4, rows=rows)
    for r, (bi, i, h) in enumerate(rows):
        assert np.array_equal(o2[r], out[bi, i, h]) and l2[r] == lse[bi, i, h]


def test_prefill_is_causal_textbook(oracle):
    """Equal heads, no past: torch's masked softmax attention in float64."""
    T, n, d = 12, 3, 8
    q = _rand(90, (1, T, n, d))
    k_new, v_new = _rand(91, (1, T, n, d)), _rand(92, (1, T, n, d))
    k = np.zeros((1, n, T, d), dtype=np.float32)
    v = np.zeros((1, n, T, d), dtype=np.float32)
    cache = _contig_cache(oracle, k, v, [0])
    oracle.cache_append(k_new, v_new, cache)
    out, _ = oracle.prefill(q, np.array([0]), cache, n, n, d, 0.5)
    tq, tk, tv = (torch.from_numpy(a.astype(np.float64)[0]).transpose(0, 1) for a in (q, k_new, v_new))
    s = tq @ tk.transpose(1, 2) * 0.5
    s = s.masked_fill(torch.triu(torch.ones(T, T, dtype=torch.bool), 1), float("-inf"))
    ref = (torch.softmax(s, -1) @ tv).transpose(0, 1).numpy()
    assert np.allclose(out[0], ref, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- augmented Q
def test_augq_closed_forms(oracle):
    # 1x1 chain by hand: x = 2*3 = 6, g = 6*0.5 = 3, u = 6*(-1) = -6, q = silu(3)*(-6)*4
    one = lambda val: np.array([[val]], dtype=np.float32)
    out = oracle.augq(one(2.0), one(3.0), one(0.5), one(-1.0), one(4.0))
    assert abs(out[0, 0] - (3.0 / (1.0 + math.exp(-3.0))) * -6.0 * 4.0) < 1e-14
    # zero gate weights: silu(0) = 0 kills the product
    h, wq = _rand(1, (5, 6)), _rand(2, (4, 6))
    wg, wu, wd = np.zeros((7, 4), np.float32), _rand(3, (7, 4)), _rand(4, (4, 7))
    assert np.all(oracle.augq(h, wq, wg, wu, wd) == 0.0)
    # silu is odd-plus-identity: silu(g) - silu(-g) = g, so flipping the gate sign changes q by (g*u) W_down^T
    wg = _rand(5, (7, 4))
    a = oracle.augq(h, wq, wg, wu, wd)
    b_ = oracle.augq(h, wq, -wg, wu, wd)
    x = W.as_f64(h) @ W.as_f64(wq).T
    lin = ((x @ W.as_f64(wg).T) * (x @ W.as_f64(wu).T)) @ W.as_f64(wd).T
    assert np.allclose(a - b_, lin, rtol=0, atol=1e-12)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_augq_matches_library_matmul(oracle, dtype):
    T, dm, dq0, da, do = 9, 12, 10, 14, 10
    h, wq = _rand(1, (T, dm), dtype), _rand(2, (dq0, dm), dtype)
    wg, wu, wd = _rand(3, (da, dq0), dtype), _rand(4, (da, dq0), dtype), _rand(5, (do, da), dtype)
    out = oracle.augq(h, wq, wg, wu, wd)
    th, twq, twg, twu, twd = (torch.from_numpy(W.as_f64(a)) for a in (h, wq, wg, wu, wd))
    x = th @ twq.T
    ref = (torch.nn.functional.silu(x @ twg.T) * (x @ twu.T)) @ twd.T
    assert np.allclose(out, ref.numpy(), rtol=1e-12, atol=1e-12)
    rows = np.array([8, 0, 3])
    assert np.array_equal(oracle.augq(h, wq, wg, wu, wd, rows=rows), out[rows])


# --------------------------------------------------------------------------- half-width keys (K feed-forward + Attend)
def _kup_case(seed, b, n_q, n_k, n_v, S, d_q, d_k, d_v, dtype="f32"):
    q = _rand(seed, (b, n_q, d_q), dtype)
    k = _rand(seed + 1, (b, n_k, S, d_k), dtype)
    v = _rand(seed + 2, (b, n_v, S, d_v), dtype)
    w = W.normal(seed + 3, (n_k, d_q, d_k), std=d_k ** -0.5, dtype=dtype)
    return q, k, v, w


def test_kup_with_identity_layer_is_plain_decode(oracle):
    """W = I (d_q = d_k) leaves the keys as they are: the function must reduce to oracle_decode exactly."""
    b, n_q, n_k, n_v, S, d = 2, 8, 2, 4, 33, 16
    q, k, v, _ = _kup_case(301, b, n_q, n_k, n_v, S, d, d, d)
    w = np.broadcast_to(np.eye(d, dtype=np.float32), (n_k, d, d)).copy()
    cache = _contig_cache(oracle, k, v, [S, 7])
    out, lse = oracle.decode_kup(q, w, cache, n_q, n_k, n_v, d, 0.41)
    ref, lse_ref = oracle.decode(q, cache, n_q, n_k, n_v, d, d, 0.41)
    assert np.array_equal(out, ref) and np.array_equal(lse, lse_ref)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_kup_matches_numpy_restatement(oracle, dtype):
    """Widen every key with numpy's matmul, then textbook softmax attention per head (per-head weights, so a
    transposed or head-shared W would fail; d_q != d_k != d_v so swapped dimensions fail)."""
    b, n_q, n_k, n_v, S, d_q, d_k, d_v = 2, 8, 2, 4, 29, 12, 6, 10
    q, k, v, w = _kup_case(311, b, n_q, n_k, n_v, S, d_q, d_k, d_v, dtype)
    lens = [S, 11]
    out, lse = oracle.decode_kup(q, w, _contig_cache(oracle, k, v, lens), n_q, n_k, n_v, d_v, 0.3)
    qf, kf, vf, wf = (W.as_f64(a) for a in (q, k, v, w))
    for bi in range(b):
        for h in range(n_q):
            hk, hv, L = h // (n_q // n_k), h // (n_q // n_v), lens[bi]
            kw = kf[bi, hk, :L] @ wf[hk].T  # [L, d_q]
            s = 0.3 * (kw @ qf[bi, h])
            p = np.exp(s - s.max())
            assert np.allclose(out[bi, h], (p / p.sum()) @ vf[bi, hv, :L], rtol=0, atol=1e-13)
            assert abs(lse[bi, h] - (s.max() + math.log(p.sum()))) < 1e-12


def test_kup_fold_identity_justifies_scoring_the_half_width_cache(oracle):
    """<q, W k> = <W^T q, k>: decoding with the layer equals plain decode over the narrow cache with the folded
    queries q' = W[hk]^T q (here folded in float64 and fed as fp32-exact small integers so that both sides see
    the same stored values)."""
    b, n_q, n_k, n_v, S, d_q, d_k, d_v = 1, 4, 2, 2, 21, 8, 4, 8
    g = np.random.Generator(np.random.Philox(key=321))
    q = g.integers(-3, 4, size=(b, n_q, d_q)).astype(np.float32)
    w = g.integers(-2, 3, size=(n_k, d_q, d_k)).astype(np.float32)
    k = g.integers(-3, 4, size=(b, n_k, S, d_k)).astype(np.float32) / 4
    v = _rand(322, (b, n_v, S, d_v))
    cache = _contig_cache(oracle, k, v, [S])
    out, lse = oracle.decode_kup(q, w, cache, n_q, n_k, n_v, d_v, 0.125)
    folded = np.stack([[w[h // (n_q // n_k)].T @ q[bi, h] for h in range(n_q)] for bi in range(b)]).astype(np.float32)
    ref, lse_ref = oracle.decode(folded, cache, n_q, n_k, n_v, d_k, d_v, 0.125)
    assert np.allclose(out, ref, rtol=0, atol=1e-13) and np.allclose(lse, lse_ref, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- selective V fetching
def test_topk_keeps_everything_when_k_covers_the_sequence(oracle):
    n_q, n_k, n_v, d, S = 8, 2, 4, 16, 40
    q, k, v = _rand(201, (2, n_q, d)), _rand(202, (2, n_k, S, d)), _rand(203, (2, n_v, S, d))
    cache = _contig_cache(oracle, k, v, [40, 13])
    full, lse_full = oracle.decode(q, cache, n_q, n_k, n_v, d, d, 0.3)
    for topk in (40, 64):
        out, lse, sel, margin = oracle.decode_topk(q, cache, n_q, n_k, n_v, d, d, 0.3, topk)
        assert np.allclose(out, full, rtol=0, atol=1e-13) and np.allclose(lse, lse_full, rtol=0, atol=1e-13)
        assert np.all(np.isinf(margin)) and np.all(np.sort(sel[0, 0][sel[0, 0] >= 0]) == np.arange(40))
        assert np.all(sel[1, :, 13:] == -1)


def test_top1_returns_the_v_row_of_the_best_key(oracle):
    n_q, n_k, n_v, d, S = 4, 2, 4, 8, 30
    q, k, v = _rand(211, (1, n_q, d)), _rand(212, (1, n_k, S, d)), _rand(213, (1, n_v, S, d))
    cache = _contig_cache(oracle, k, v, [S])
    out, lse, sel, _ = oracle.decode_topk(q, cache, n_q, n_k, n_v, d, d, 1.0, 1)
    for h in range(n_q):
        s = W.as_f64(k[0, h // 2]) @ W.as_f64(q[0, h])
        j = int(np.argmax(s))
        assert sel[0, h, 0] == j and np.array_equal(out[0, h], W.as_f64(v[0, h, j])) and abs(lse[0, h] - s[j]) < 1e-13


def test_topk_matches_numpy_selection_and_error_bound(oracle):
    """Independent restatement with numpy's sort; and the distance to full attention is bounded by twice the
    probability mass that was dropped times the largest |V|."""
    n_q, n_k, n_v, d, S, topk = 8, 2, 4, 16, 200, 20
    q, k, v = _rand(221, (1, n_q, d)), _rand(222, (1, n_k, S, d)), _rand(223, (1, n_v, S, d))
    cache = _contig_cache(oracle, k, v, [S])
    out, lse, sel, margin = oracle.decode_topk(q, cache, n_q, n_k, n_v, d, d, 0.5, topk)
    full, _ = oracle.decode(q, cache, n_q, n_k, n_v, d, d, 0.5)
    for h in range(n_q):
        s = 0.5 * (W.as_f64(k[0, h // 4]) @ W.as_f64(q[0, h]))
        order = np.argsort(-s, kind="stable")
        keep = order[:topk]
        assert np.array_equal(sel[0, h], keep)
        p = np.exp(s[keep] - s[keep].max())
        ref = (p / p.sum()) @ W.as_f64(v[0, h // 2])[keep]
        assert np.allclose(out[0, h], ref, rtol=0, atol=1e-13)
        assert abs(margin[0, h] - (s[order[topk - 1]] - s[order[topk]])) < 1e-13
        pf = np.exp(s - s.max())
        dropped = 1.0 - pf[keep].sum() / pf.sum()
        assert np.abs(out[0, h] - full[0, h]).max() <= 2.0 * dropped * np.abs(W.as_f64(v[0, h // 2])).max() + 1e-12


def test_topk_ties_take_the_earlier_token(oracle):
    d = 4
    q = np.ones((1, 1, d), np.float32)
    k = np.ones((1, 1, 6, d), np.float32)  # every score equal
    v = np.arange(6 * d, dtype=np.float32).reshape(1, 1, 6, d)
    out, _, sel, margin = oracle.decode_topk(q, _contig_cache(oracle, k, v, [6]), 1, 1, 1, d, d, 1.0, 3)
    assert np.array_equal(sel[0, 0], [0, 1, 2]) and margin[0, 0] == 0.0
    assert np.allclose(out[0, 0], v[0, 0, :3].mean(axis=0))


# --------------------------------------------------------------------------- projections and rotary embedding
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_linear_matches_library_matmul(oracle, dtype):
    x, w = _rand(1, (7, 12), dtype), _rand(2, (5, 12), dtype)
    ref = torch.from_numpy(W.as_f64(x)) @ torch.from_numpy(W.as_f64(w)).T
    assert np.allclose(oracle.linear(x, w), ref.numpy(), rtol=1e-13, atol=1e-13)
    # one-hot input picks a column of W^T
    e = np.zeros((1, 12), np.float32)
    e[0, 3] = 1.0
    assert np.array_equal(oracle.linear(e, _rand(2, (5, 12))), W.as_f64(_rand(2, (5, 12)))[:, 3][None])


def test_rope_closed_forms(oracle):
    d, theta = 8, 50000.0
    x = np.random.default_rng(3).standard_normal((6, 3, d))
    pos = np.array([0, 1, 2, 7, 100, 4095])
    y = oracle.rope(x, pos, theta)
    assert np.array_equal(y[0], x[0])  # position 0 rotates by nothing
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)  # a rotation
    # pair 0 turns by exactly `pos` radians (theta^0 = 1): check one element by hand
    t, h = 3, 1
    a, b = x[t, h, 0], x[t, h, d // 2]
    assert abs(y[t, h, 0] - (a * math.cos(7.0) - b * math.sin(7.0))) < 1e-14
    assert abs(y[t, h, d // 2] - (b * math.cos(7.0) + a * math.sin(7.0))) < 1e-14
    # the last pair turns by pos * theta^(-2 (d/2 - 1) / d)
    ang = 100.0 * theta ** (-2.0 * (d // 2 - 1) / d)
    a, b = x[4, 0, d // 2 - 1], x[4, 0, d - 1]
    assert abs(y[4, 0, d // 2 - 1] - (a * math.cos(ang) - b * math.sin(ang))) < 1e-13
    # tables are the same angles
    c, s_ = oracle.rope_tables(pos, d, theta)
    assert abs(c[4, d // 2 - 1] - math.cos(ang)) < 1e-15 and abs(s_[3, 0] - math.sin(7.0)) < 1e-15


def test_rope_scores_depend_on_relative_position_only(oracle):
    d, theta = 16, 500000.0
    rng = np.random.default_rng(5)
    q, k = rng.standard_normal((1, 1, d)), rng.standard_normal((1, 1, d))
    dots = []
    for m, n in ((10, 3), (107, 100), (5007, 5000)):
        dots.append(float(np.sum(oracle.rope(q, np.array([m]), theta) * oracle.rope(k, np.array([n]), theta))))
    assert max(dots) - min(dots) < 1e-9
    other = float(np.sum(oracle.rope(q, np.array([10]), theta) * oracle.rope(k, np.array([4]), theta)))
    assert abs(other - dots[0]) > 1e-6  # and they do depend on it


def test_rope_is_the_complex_rotation(oracle):
    """Pair (x_i, x_{i+d/2}) as a complex number is multiplied by e^{i angle}: numpy's complex arithmetic."""
    d, theta = 32, 50000.0
    rng = np.random.default_rng(8)
    x = rng.standard_normal((5, 2, d))
    pos = np.array([1, 17, 300, 9999, 65535])
    z = x[..., : d // 2] + 1j * x[..., d // 2:]
    ang = pos[:, None] * theta ** (-2.0 * np.arange(d // 2) / d)[None, :]
    zr = z * np.exp(1j * ang)[:, None, :]
    ref = np.concatenate([zr.real, zr.imag], axis=-1)
    assert np.allclose(oracle.rope(x, pos, theta), ref, rtol=0, atol=1e-12)


# --------------------------------------------------------------------------- cost model
def test_cache_cost_model_matches_paper(oracle):
    """Eq. (imp_t): SIGMA-1.5B against the 16/16 GQA model saves (32-20)/32 of the cache traffic."""
    with open(os.path.join(GOLDEN, "cache_cost_model.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for n_k, n_v, gk, gv, d, red in rows:
        n_k, n_v, gk, gv, d = map(int, (n_k, n_v, gk, gv, d))
        lens = np.array([4096, 123], dtype=np.int32)
        ours = oracle.kv_bytes(lens, n_k, n_v, d, d, 2)
        gqa = oracle.kv_bytes(lens, gk, gv, d, d, 2)
        assert ours == 4219 * (n_k + n_v) * d * 2
        assert abs((gqa - ours) / gqa - float(red)) < 1e-15
    # the benchmark shapes (n_k = n_v/2 against n_k = n_v) save exactly one quarter
    for cfg in (W.CFG2, W.CFG3):
        lens = W.draw_lengths(cfg)
        tw = cfg.gqa_twin()
        a = oracle.kv_bytes(lens, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v, 2)
        g = oracle.kv_bytes(lens, tw.n_k, tw.n_v, tw.d_qk, tw.d_v, 2)
        assert (g - a) / g == 0.25
    assert oracle.kv_bytes(W.draw_lengths(W.CFG3), 4, 8, 128, 128, 2) == 402653184.0


# --------------------------------------------------------------------------- input generator
def test_generator_is_deterministic_and_rounds_to_nearest_even():
    a = W.normal(3, (1000,), dtype="bf16")
    assert np.array_equal(a, W.normal(3, (1000,), dtype="bf16"))
    assert not np.array_equal(a, W.normal(4, (1000,), dtype="bf16"))
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.3895314e38], dtype=np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(W.f32_to_bf16_bits(x), ref)
    big = W.normal(9, (3_000_000,), dtype="f32")
    assert abs(big.mean()) < 5e-3 and abs(big.std() - 1) < 5e-3
    lens = W.draw_lengths(W.CFG5)
    assert lens.min() >= 1024 and lens.max() <= 65536 and len(lens) == 64
