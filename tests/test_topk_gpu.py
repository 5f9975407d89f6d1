"""GPU parity of diffqkv_decode_topk (selective V cache fetching) against the float64 oracle through the C ABI.

Which tokens are kept is decided by comparing scores.  The kernel scores with fp32 accumulation, the oracle in float64, so two
scores closer than the kernel's accumulation error may swap ranks at the cut.  The oracle reports the gap between the last kept and the first dropped score of every row: rows whose gap is
clear of that error must match within the bf16 tolerances of helpers.check_bf16; for the others the result is
checked for validity instead: it may differ by a swap of near-equal tokens at the cut, whose weight is at most the
weight of the last kept token, so |err| <= tol + 2 * w_last * max|V| per swap (a few swaps at most)."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_lse, device_cache, oracle_cache, run_oracle

pytestmark = pytest.mark.gpu
SCORE_EPS = 2e-5  # bound on |kernel score - exact score|: bf16 x bf16 products are exact in fp32, so only the fp32
                  # accumulation of d <= 128 terms rounds (about 1e-6 of the score magnitude, scores are O(1))


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def run_topk(api, inp, topk):
    cfg = inp.cfg
    q = W.to_torch(inp.q, "cuda")
    cache = device_cache(api, inp)
    lse = torch.full((cfg.batch, cfg.n_q), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = api.diffqkv_decode_topk(q, cache, cfg.n_k, cfg.n_v, cfg.scale, topk, lse=lse, dev_status=status,
                                  out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


def check_against_oracle(oracle, inp, topk, out, lse, what):
    cfg = inp.cfg
    ref, lse_ref, sel, margin = oracle.decode_topk(inp.q, oracle_cache(oracle, inp), cfg.n_q, cfg.n_k, cfg.n_v,
                                                   cfg.d_qk, cfg.d_v, cfg.scale, topk)
    clear = margin > 2 * SCORE_EPS
    assert clear.mean() > 0.5, "the test inputs should leave most rows unambiguous"
    if clear.any():
        check_bf16(out[clear], ref[clear], what)
        check_lse(lse[clear], lse_ref[clear], 2e-2, what)
    vmax = float(np.abs(W.as_f64(inp.v)).max())
    for b, h in zip(*np.nonzero(~clear)):
        kept = sel[b, h][sel[b, h] >= 0]
        # weight of the last kept token = exp(s_last - lse); s_last from the definition
        hk = h * cfg.n_k // cfg.n_q
        j = int(kept[-1])
        if inp.page_table is None:
            krow = W.as_f64(inp.k[b, hk, j])
        else:
            krow = W.as_f64(inp.k[inp.page_table[b, j // cfg.page_size], hk, j % cfg.page_size])
        s_last = cfg.scale * float(krow @ W.as_f64(inp.q[b, h]))
        w = float(np.exp(s_last - lse_ref[b, h]))
        assert np.abs(out[b, h] - ref[b, h]).max() <= 2e-2 + 3 * 2 * w * vmax, f"{what}: row ({b},{h})"
    assert np.isfinite(out).all()


SMALL = W.DecodeConfig("topk_small", batch=3, n_q=16, n_k=2, n_v=4, d_qk=128, d_v=128, kv_len=3000, seed=91)


@pytest.mark.parametrize("topk", [1, 7, 100, 1024])
def test_topk_small(api, oracle, topk):
    inp = W.make_decode_inputs(SMALL, seqlens=np.array([3000, 129, 64], np.int32))
    out, lse = run_topk(api, inp, topk)
    check_against_oracle(oracle, inp, topk, out, lse, f"topk={topk}")


def test_topk_covering_the_sequence_equals_full_decode(api, oracle):
    inp = W.make_decode_inputs(SMALL, seqlens=np.array([700, 1, 0], np.int32))
    out, lse = run_topk(api, inp, 1024)
    ref, lse_ref = run_oracle(oracle, inp)
    check_bf16(out, ref, "k >= len")
    check_lse(lse, lse_ref, 2e-2)
    assert np.all(out[2] == 0) and np.all(np.isneginf(lse[2]))


@pytest.mark.parametrize("heads,d", [((8, 8, 8), 64), ((32, 1, 4), 128), ((12, 6, 2), 64), ((32, 4, 16), 64), ((8, 4, 1), 128)])
def test_topk_head_configurations(api, oracle, heads, d):
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, batch=2, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, kv_len=1500, seed=92)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([1500, 333], np.int32))
    out, lse = run_topk(api, inp, 50)
    check_against_oracle(oracle, inp, 50, out, lse, f"heads={heads} d={d}")


@pytest.mark.parametrize("page_size", [16, 64, 128])
def test_topk_paged_equals_contiguous_bitwise(api, oracle, page_size):
    inp = W.make_decode_inputs(dataclasses.replace(SMALL, kv_len=1024), seqlens=np.array([1024, 500, 17], np.int32))
    base, lse0 = run_topk(api, inp, 100)
    pg = W.paginate(inp, page_size, seed=9)
    out, lse = run_topk(api, pg, 100)
    assert np.array_equal(out, base) and np.array_equal(lse, lse0)
    check_against_oracle(oracle, inp, 100, base, lse0, "contiguous")


def test_topk_ties_take_the_earlier_tokens(api):
    """Every key equal: every score equal, the first k tokens are kept and the output is the mean of their V rows."""
    cfg = dataclasses.replace(SMALL, batch=1, n_q=8, n_k=2, n_v=2, kv_len=400, seed=93)
    inp = W.make_decode_inputs(cfg)
    inp.k[:] = inp.k[:, :, :1]
    out, _ = run_topk(api, inp, 10)
    v = W.as_f64(inp.v)
    for h in range(8):
        assert np.abs(out[0, h] - v[0, h // 4, :10].mean(axis=0)).max() <= 1e-5


@pytest.fixture
def general_only(api):
    """Switches diffqkv_decode_topk to the selection over all scores and back."""
    yield api.topk_general_only
    api.topk_general_only(False)


def test_topk_partial_ties_at_the_cut(api, oracle, general_only):
    """All keys equal except a few: the kept set is the few that score higher plus the earliest of the equal ones,
    so the cut falls inside a run of exactly equal scores.  Checked in both selection paths."""
    cfg = dataclasses.replace(SMALL, batch=1, n_q=8, n_k=2, n_v=4, kv_len=2000, seed=94)
    inp = W.make_decode_inputs(cfg)
    special = np.array([3, 517, 1024, 1999, 1500])
    keep = inp.k[:, :, special].copy()
    inp.k[:] = inp.k[:, :, 7:8]
    inp.k[:, :, special] = keep
    ref, lse_ref, sel, _ = oracle.decode_topk(inp.q, oracle_cache(oracle, inp), cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk,
                                              cfg.d_v, cfg.scale, 20)
    for h in range(cfg.n_q):  # the definition's choice: the tokens that beat the common score, then the earliest
        kept = np.sort(sel[0, h])
        common = np.setdiff1d(kept, special)
        assert np.array_equal(common, np.setdiff1d(np.arange(2000), special)[:len(common)])
    for on in (False, True):
        general_only(on)
        out, lse = run_topk(api, inp, 20)
        check_bf16(out, ref, f"partial ties, general_only={on}")
        check_lse(lse, lse_ref, 2e-2)


@pytest.mark.parametrize("lens,topk", [((3000, 129, 64), 50), ((2500, 2048, 33), 7)])
def test_topk_selection_paths_agree_bitwise(api, general_only, lens, topk):
    """The selection driven by the block maxima and the one over all scores keep the same tokens in the same order."""
    inp = W.make_decode_inputs(SMALL, seqlens=np.array(lens, np.int32))
    out, lse = run_topk(api, inp, topk)
    general_only(True)
    out_g, lse_g = run_topk(api, inp, topk)
    assert np.array_equal(out, out_g) and np.array_equal(lse, lse_g)


def test_topk_rows_longer_than_one_selection_pass(api, oracle, general_only):
    """70000 tokens: the selection over all scores takes the row in 32768-token pieces and merges their winners."""
    cfg = dataclasses.replace(SMALL, batch=2, n_q=8, n_k=1, n_v=2, kv_len=70000, seed=95)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([70000, 32769], np.int32))
    out, lse = run_topk(api, inp, 100)
    check_against_oracle(oracle, inp, 100, out, lse, "70000 tokens")
    general_only(True)
    out_g, lse_g = run_topk(api, inp, 100)
    assert np.array_equal(out, out_g) and np.array_equal(lse, lse_g)


def test_topk_config3_full_size(api, oracle, general_only):
    """The long-context configuration (batch 4, 32/4/8 heads, d 128, 32768 tokens) with the paper's 100 scores."""
    inp = W.make_decode_inputs(W.CFG3)
    out, lse = run_topk(api, inp, 100)
    check_against_oracle(oracle, inp, 100, out, lse, "cfg3 top-100")
    general_only(True)
    out_g, lse_g = run_topk(api, inp, 100)
    assert np.array_equal(out, out_g) and np.array_equal(lse, lse_g)


def test_topk_argument_errors(api):
    inp = W.make_decode_inputs(dataclasses.replace(SMALL, batch=1, kv_len=128))
    q, cache = W.to_torch(inp.q, "cuda"), device_cache(api, inp)
    with pytest.raises(api.DiffQKVError) as e:
        api.diffqkv_decode_topk(q, cache, 2, 4, 0.1, 2000)
    assert e.value.status == api.ERR_UNSUPPORTED
    with pytest.raises(api.DiffQKVError) as e:
        api.diffqkv_decode_topk(q, cache, 2, 4, 0.1, 10, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == api.ERR_WORKSPACE


@pytest.mark.parametrize("topk,paged", [(1, 0), (7, 16), (100, 0), (100, 64), (1024, 0)])
def test_kept_token_ids_are_a_valid_selection(api, oracle, topk, paged):
    """diffqkv_decode_topk_ids returns which tokens entered each head's output.  Several sets can be right when
    scores at the cut differ by less than fp32 scoring resolves, so the unique part is compared and the rest is
    checked for validity: min(topk, len) distinct visible tokens; on rows the inputs decide (gap at the cut above
    the scoring error) exactly the oracle's set; on the others every kept score at least every dropped score minus
    the scoring error (scores from the definition, in float64); -1 padding behind short sequences."""
    cfg = dataclasses.replace(SMALL, seed=95)
    lens = np.array([3000, 129, 0], np.int32)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    # equal keys make equal scores: part of the selection is then decided by the tie rule alone
    inp.k[0, :, 1000:1040] = inp.k[0, :, 1000:1001]
    case = W.paginate(inp, paged, seed=3) if paged else inp
    q, cache = W.to_torch(case.q, "cuda"), device_cache(api, case)
    ids = torch.full((cfg.batch, cfg.n_q, topk), -7, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = api.diffqkv_decode_topk(q, cache, cfg.n_k, cfg.n_v, cfg.scale, topk, dev_status=status,
                                  out_dtype=torch.float32, kept_ids=ids)
    plain = api.diffqkv_decode_topk(q, cache, cfg.n_k, cfg.n_v, cfg.scale, topk, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(out, plain)
    ids = ids.cpu().numpy()
    _, _, sel, margin = oracle.decode_topk(inp.q, oracle_cache(oracle, inp), cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk,
                                           cfg.d_v, cfg.scale, topk)
    qf, kf = W.as_f64(inp.q), W.as_f64(inp.k)
    for b in range(cfg.batch):
        n = int(lens[b])
        for h in range(cfg.n_q):
            kept = ids[b, h]
            k = min(topk, n)
            got = kept[kept >= 0]
            assert len(got) == k and np.all(kept[k:] == -1), (b, h)
            assert len(set(got.tolist())) == k and (k == 0 or (got.min() >= 0 and got.max() < n)), (b, h)
            if k == 0:
                continue
            want = set(sel[b, h][sel[b, h] >= 0].tolist())
            if margin[b, h] > 2 * SCORE_EPS:
                assert set(got.tolist()) == want, f"row ({b},{h}): kept set differs from the oracle's"
            else:
                s = cfg.scale * (kf[b, h * cfg.n_k // cfg.n_q, :n] @ qf[b, h])
                dropped = np.setdiff1d(np.arange(n), got)
                if len(dropped):
                    assert s[got].min() >= s[dropped].max() - 2 * SCORE_EPS, f"row ({b},{h}): not a top-{topk} set"
