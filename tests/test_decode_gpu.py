"""GPU parity of diffqkv_decode / gqa_decode / diffqkv_combine against the float64 oracle,
called through the C ABI on the same seeded inputs."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, check_f32, check_lse, device_cache, run_decode, run_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def test_cfg1_fp32_small(api, oracle):
    """Config 1: batch 1, 16/2/4 heads, d 64, 512 tokens, fp32 cache, seed 0, scale 1/8."""
    inp = W.make_decode_inputs(W.CFG1)
    ref, lse_ref = run_oracle(oracle, inp)
    for splits in (0, 1, 3, 8):
        out, lse, st = run_decode(api, inp, num_splits=splits)
        assert st == 0
        check_f32(out, ref, f"cfg1 splits={splits}")
        check_lse(lse, lse_ref, 1e-5 * np.abs(lse_ref).max())


@pytest.mark.parametrize("cfg", [W.CFG2, W.CFG3], ids=lambda c: c.name)
def test_full_size_bf16_and_gqa_twin(api, oracle, cfg):
    """Configs 2 and 3 at full size, DiffQKV and the n_k = n_v twin, every output element."""
    for c in (cfg, cfg.gqa_twin()):
        inp = W.make_decode_inputs(c)
        ref, lse_ref = run_oracle(oracle, inp)
        gqa = c.n_k == c.n_v
        out, lse, st = run_decode(api, inp, gqa=gqa)
        assert st == 0
        check_bf16(out, ref, c.name)
        check_lse(lse, lse_ref, 2e-2, c.name)
        out_b, _, _ = run_decode(api, inp, out_dtype=torch.bfloat16, gqa=gqa, want_lse=False)
        check_bf16(out_b, ref, c.name + " bf16 out")


SMALL = W.DecodeConfig("small", batch=3, n_q=16, n_k=2, n_v=4, d_qk=128, d_v=128, kv_len=700, seed=42)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("heads", [(16, 2, 4), (8, 8, 8), (8, 1, 1), (8, 1, 8), (12, 6, 2), (32, 4, 16), (4, 4, 2)])
@pytest.mark.parametrize("d", [64, 128])
def test_head_configurations(api, oracle, dtype, heads, d):
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, dtype=dtype)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([700, 1, 333], dtype=np.int32))
    ref, lse_ref = run_oracle(oracle, inp)
    out, lse, st = run_decode(api, inp)
    assert st == 0
    (check_bf16 if dtype == "bf16" else check_f32)(out, ref, str(heads))
    check_lse(lse, lse_ref, 2e-2 if dtype == "bf16" else 1e-4)


def test_mixed_head_dims(api, oracle):
    cfg = dataclasses.replace(SMALL, d_qk=64, d_v=128)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([700, 65, 64], dtype=np.int32))
    ref, _ = run_oracle(oracle, inp)
    out, _, st = run_decode(api, inp)
    assert st == 0
    check_bf16(out, ref)


@pytest.mark.parametrize("heads", [(32, 1, 2), (32, 2, 4), (32, 2, 2), (16, 1, 1), (64, 4, 8), (64, 2, 16)])
@pytest.mark.parametrize("d", [64, 128])
def test_more_than_eight_query_heads_per_kv_head(api, oracle, fixed_owners, heads, d):
    """Multi-query-like shapes: the TMA kernel cuts a unit of 16 to 32 query heads into sub-units of 8 that share
    their K (and V) head; parity with the oracle, contiguous and paged."""
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, batch=2, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, kv_len=900, seed=45)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([900, 130], dtype=np.int32))
    ref, lse_ref = run_oracle(oracle, inp)
    out, lse, st = run_decode(api, inp)
    assert st == 0 and api.last_decode_kernel() == 2
    check_bf16(out, ref, str(heads))
    check_lse(lse, lse_ref, 2e-2)
    out_p, lse_p, st = run_decode(api, W.paginate(inp, 64, seed=4))
    assert st == 0 and np.array_equal(out_p, out) and np.array_equal(lse_p, lse)


@pytest.mark.parametrize("heads", [(32, 4, 16), (16, 2, 4), (8, 4, 4)])
def test_half_width_keys_take_the_tma_kernel(api, oracle, fixed_owners, heads):
    """d_k = d_v / 2 (the paper's other axis of K compression) with SIGMA-1.5B's 4 K / 16 V heads and two smaller
    shapes: the persistent TMA kernel, not the generic fallback."""
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=64, d_v=128, kv_len=1500, seed=44)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([1500, 333, 64], dtype=np.int32))
    ref, lse_ref = run_oracle(oracle, inp)
    out, lse, st = run_decode(api, inp)
    assert st == 0 and api.last_decode_kernel() == 2
    check_bf16(out, ref, str(heads))
    check_lse(lse, lse_ref, 2e-2)
    pg = W.paginate(inp, 16, seed=3)
    out_p, lse_p, st = run_decode(api, pg)
    assert st == 0 and api.last_decode_kernel() == 2
    assert np.array_equal(out_p, out) and np.array_equal(lse_p, lse)


@pytest.mark.parametrize("lens", [[0, 0, 0], [0, 5, 700], [63, 64, 65], [127, 128, 129], [1, 2, 3]])
def test_ragged_and_empty_lengths(api, oracle, lens):
    inp = W.make_decode_inputs(SMALL, seqlens=np.array(lens, dtype=np.int32))
    ref, lse_ref = run_oracle(oracle, inp)
    for splits in (0, 1, 5):
        out, lse, st = run_decode(api, inp, num_splits=splits)
        assert st == 0
        check_bf16(out, ref, f"{lens} splits={splits}")
        check_lse(lse, lse_ref, 2e-2)
        for b, n in enumerate(lens):
            if n == 0:
                assert np.all(out[b] == 0.0) and np.all(np.isneginf(lse[b]))


def test_split_count_invariance(api, oracle):
    """Any split count gives the same result up to fp32 reassociation."""
    inp = W.make_decode_inputs(dataclasses.replace(SMALL, kv_len=3000), seqlens=np.array([3000, 1500, 77], np.int32))
    ref, _ = run_oracle(oracle, inp)
    outs = []
    for splits in (1, 2, 7, 16, 47):
        out, _, st = run_decode(api, inp, num_splits=splits)
        assert st == 0
        check_bf16(out, ref, f"splits={splits}")
        outs.append(out)
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() <= 5e-3


@pytest.mark.parametrize("page_size", [16, 64])
def test_paged_equals_contiguous_bitwise(api, oracle, page_size):
    """Paging is pure addressing: identity table, shuffled table and the contiguous cache give
    bit-identical outputs for the same chunking."""
    inp = W.make_decode_inputs(dataclasses.replace(SMALL, kv_len=1024), seqlens=np.array([1024, 500, 17], np.int32))
    ref, _ = run_oracle(oracle, inp)
    base, lse0, st = run_decode(api, inp, num_splits=4)
    assert st == 0
    check_bf16(base, ref)
    for identity in (True, False):
        pg = W.paginate(inp, page_size, seed=9, identity=identity)
        out, lse, st = run_decode(api, pg, num_splits=4)
        assert st == 0
        assert np.array_equal(out, base) and np.array_equal(lse, lse0)


def test_token_major_layout(api, oracle):
    """The (b, s, n_h, d_h) layout of the paper's cache, expressed through strides."""
    inp = W.make_decode_inputs(SMALL, seqlens=np.array([700, 300, 64], np.int32))
    base, _, _ = run_decode(api, inp)
    c = inp.cfg
    S = c.kv_len
    tm = dataclasses.replace(
        inp, k=np.ascontiguousarray(inp.k.transpose(0, 2, 1, 3)), v=np.ascontiguousarray(inp.v.transpose(0, 2, 1, 3)),
        k_strides=(S * c.n_k * c.d_qk, c.d_qk, c.n_k * c.d_qk), v_strides=(S * c.n_v * c.d_v, c.d_v, c.n_v * c.d_v))
    ref, _ = run_oracle(oracle, tm)
    out, _, st = run_decode(api, tm)
    assert st == 0
    check_bf16(out, ref)
    assert np.abs(out - base).max() <= 5e-3


def test_out_of_range_page_is_reported_not_read(api):
    """A page id outside the pool sets the INDEX bit in dev_status; the kernel skips the read."""
    inp = W.make_decode_inputs(dataclasses.replace(SMALL, kv_len=256), seqlens=np.array([256, 256, 256], np.int32))
    pg = W.paginate(inp, 16, seed=3)
    pg.page_table[1, 3] = pg.num_pages + 5
    pg.page_table[2, 0] = -1
    for splits in (0, 2):  # TMA kernel and generic kernel
        out, lse, st = run_decode(api, pg, num_splits=splits)
        assert st == (1 << api.ERR_INDEX)
        assert np.all(np.isfinite(out))


def test_paged_varlen_config5_shape_reduced(api, oracle):
    """Config 5's structure (16-token pages, shuffled table, uniform lengths) at a reduced length range."""
    cfg = dataclasses.replace(W.CFG5, batch=8, kv_len=4096, len_range=(64, 4096))
    inp = W.make_decode_inputs(cfg)
    ref, lse_ref = run_oracle(oracle, inp)
    out, lse, st = run_decode(api, inp)
    assert st == 0
    check_bf16(out, ref)
    check_lse(lse, lse_ref, 2e-2)


@pytest.fixture
def fixed_owners(api):
    """No tail reserve: every tile has a fixed owner, so results are bitwise reproducible (what the tests that
    compare two runs bit for bit need); the default is restored afterwards."""
    api.set_tail_reserve(0)
    yield
    api.set_tail_reserve(-1)


@pytest.fixture
def tail_reserve(api):
    """Sets the tail reserve of the TMA kernel and always restores the automatic choice."""
    yield api.set_tail_reserve
    api.set_tail_reserve(-1)


@pytest.fixture
def blocks(api):
    """Sets the persistent-block cap of the TMA kernel and always restores the default."""
    yield api.set_max_blocks
    api.set_max_blocks(0)


def test_tma_kernel_is_the_bf16_path(api):
    inp = W.make_decode_inputs(SMALL)
    run_decode(api, inp)
    assert api.last_decode_kernel() == api.KERNEL_TMA
    run_decode(api, inp, num_splits=3)
    assert api.last_decode_kernel() == api.KERNEL_GENERIC
    run_decode(api, W.make_decode_inputs(W.CFG1))
    assert api.last_decode_kernel() == api.KERNEL_GENERIC  # fp32 mode


@pytest.mark.parametrize("heads", [(16, 2, 4), (32, 4, 16), (8, 8, 8), (8, 4, 1), (8, 2, 4)])
@pytest.mark.parametrize("d", [64, 128])
def test_tma_block_partition_invariance(api, oracle, blocks, heads, d):
    """The flat tile list is cut differently for every block count; results agree with the oracle
    and with each other up to fp32 reassociation."""
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, batch=5, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, kv_len=1500)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([1500, 64, 0, 777, 1], dtype=np.int32))
    ref, lse_ref = run_oracle(oracle, inp)
    outs = []
    for nb in (1, 2, 3, 7, 40, 0):
        blocks(nb)
        out, lse, st = run_decode(api, inp)
        assert st == 0 and api.last_decode_kernel() == api.KERNEL_TMA
        check_bf16(out, ref, f"{heads} d={d} blocks={nb}")
        check_lse(lse, lse_ref, 2e-2)
        assert np.all(out[2] == 0) and np.all(np.isneginf(lse[2]))
        outs.append(out)
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() <= 5e-3


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
def test_tma_paged_equals_contiguous_bitwise(api, oracle, blocks, fixed_owners, page_size):
    inp = W.make_decode_inputs(dataclasses.replace(SMALL, kv_len=1024), seqlens=np.array([1024, 500, 17], np.int32))
    ref, _ = run_oracle(oracle, inp)
    for nb in (0, 5):
        blocks(nb)
        base, lse0, st = run_decode(api, inp)
        assert st == 0 and api.last_decode_kernel() == api.KERNEL_TMA
        check_bf16(base, ref)
        for identity in (True, False):
            pg = W.paginate(inp, page_size, seed=9, identity=identity)
            out, lse, st = run_decode(api, pg)
            assert st == 0 and api.last_decode_kernel() == api.KERNEL_TMA
            assert np.array_equal(out, base) and np.array_equal(lse, lse0)


@pytest.mark.parametrize("heads,d_qk,d_v", [((16, 2, 4), 128, 128), ((32, 4, 16), 64, 64), ((8, 4, 1), 128, 128),
                                            ((32, 1, 2), 128, 128), ((16, 2, 4), 64, 128)])
def test_tail_reserve_invariance(api, oracle, blocks, tail_reserve, heads, d_qk, d_v):
    """Tiles drawn from the reserves (the block's own and those of the other blocks of the row) give the same
    attention as fixed owners: against the oracle and against each other up to fp32 reassociation, for several block
    counts (which move the cuts), reserves from one tile to the whole segment, ragged and empty sequences, NaN bit
    patterns behind every sequence end, contiguous and paged."""
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, batch=5, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d_qk, d_v=d_v, kv_len=3000, seed=91)
    lens = np.array([3000, 64, 0, 1777, 1], dtype=np.int32)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    for b, n in enumerate(lens):
        inp.k[b, :, n:] = 0x7FC0  # bf16 NaN
        inp.v[b, :, n:] = 0x7FC0
    ref, lse_ref = run_oracle(oracle, inp)
    outs = []
    for paged in (0, 16):
        case = W.paginate(inp, paged, seed=7) if paged else inp
        for nb in (0, 7, 40):
            blocks(nb)
            for reserve in (0, 1, 3, 4096, -1):
                tail_reserve(reserve)
                out, lse, st = run_decode(api, case)
                what = f"{heads} d={d_qk}/{d_v} paged={paged} blocks={nb} reserve={reserve}"
                assert st == 0 and api.last_decode_kernel() == api.KERNEL_TMA, what
                check_bf16(out, ref, what)
                check_lse(lse, lse_ref, 2e-2, what)
                assert np.all(out[2] == 0) and np.all(np.isneginf(lse[2])), what
                outs.append(out)
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() <= 5e-3


def test_end_of_tail_marker_is_posted_once_every_lane_saw_the_slot_free(api, oracle, blocks, tail_reserve):
    """Blocks with only a few tiles and a one-tile reserve reach the end-of-segment marker while their ring is full:
    the producer's lanes must all have seen the slot free before it is handed on (a lane left polling would run
    into its limit and report a timeout although every result is right).  Repeated, since it is a matter of timing."""
    cfg = dataclasses.replace(SMALL, batch=5, n_q=32, n_k=4, n_v=16, d_qk=64, d_v=64, kv_len=3000, seed=91)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([3000, 64, 0, 1777, 1], dtype=np.int32))
    ref, _ = run_oracle(oracle, inp)
    for nb in (39, 40, 41):
        blocks(nb)
        for reserve in (1, -1):
            tail_reserve(reserve)
            for _ in range(8):
                out, _, st = run_decode(api, inp)
                assert st == 0, f"blocks={nb} reserve={reserve}: device status {st}"
            check_bf16(out, ref, f"blocks={nb} reserve={reserve}")


def test_tail_reserve_full_size_every_tile_drawn(api, oracle, tail_reserve):
    """The headline shape with every tile but one per segment handed out through the counters: a stress of the
    draw protocol at 148 blocks (the automatic reserve runs in test_full_size_bf16_and_gqa_twin)."""
    inp = W.make_decode_inputs(W.CFG3)
    ref, lse_ref = run_oracle(oracle, inp)
    for reserve in (4096, 20):
        tail_reserve(reserve)
        for _ in range(3):
            out, lse, st = run_decode(api, inp)
            assert st == 0
            check_bf16(out, ref, f"cfg3 reserve={reserve}")
            check_lse(lse, lse_ref, 2e-2)


def test_a_device_wait_that_runs_out_is_reported_and_leaves_the_context_usable(api, oracle, fixed_owners):
    """The failure path of the bounded waits, reached without breaking anything: with the wait limit at 2 ms the
    producer of block 0 never requests its first tile (no copy in flight, no completion count), the consumers' wait
    for it runs out, the block reports DIFFQKV_ERR_TIMEOUT, drains and returns.  The same stream then runs an
    ordinary call whose result equals, bit for bit, that of a call made before the failure."""
    inp = W.make_decode_inputs(dataclasses.replace(SMALL, batch=4, kv_len=2000, seed=97))
    ref, _ = run_oracle(oracle, inp)
    clean, lse_clean, st = run_decode(api, inp)
    assert st == 0 and api.last_decode_kernel() == api.KERNEL_TMA
    check_bf16(clean, ref)
    try:
        api.debug_decode_timeout(2_000_000, 0)
        _, _, st = run_decode(api, inp)
    finally:
        api.debug_decode_timeout(0, -1)
    assert st == 1 << api.ERR_TIMEOUT
    again, lse_again, st = run_decode(api, inp)
    assert st == 0
    assert np.array_equal(again, clean) and np.array_equal(lse_again, lse_clean)


def test_tma_tail_rows_with_nan_garbage(api, oracle):
    """Cache rows past a sequence's end may hold anything, NaN bit patterns included."""
    inp = W.make_decode_inputs(SMALL, seqlens=np.array([700, 333, 5], np.int32))
    for b, n in enumerate([700, 333, 5]):
        inp.k[b, :, n:] = 0x7FC0  # bf16 NaN
        inp.v[b, :, n:] = 0x7FC0
    ref, _ = run_oracle(oracle, inp)
    out, _, st = run_decode(api, inp)
    assert st == 0 and api.last_decode_kernel() == api.KERNEL_TMA
    check_bf16(out, ref)


def test_combine_entry_point(api, oracle):
    rng = np.random.Generator(np.random.Philox(key=5))
    o = rng.standard_normal((3, 8, 11, 128)).astype(np.float32)
    l = (3 * rng.standard_normal((3, 8, 11))).astype(np.float32)
    l[0, 0, :] = -np.inf
    l[1, 2, 3:] = -np.inf
    o[1, 2, 3:] = np.nan  # skipped splits must not be read into the result
    ref, lse_ref = oracle.combine(o.astype(np.float64), l.astype(np.float64))
    to, tl = torch.from_numpy(o).cuda(), torch.from_numpy(l).cuda()
    lse = torch.empty((3, 8), dtype=torch.float32, device="cuda")
    out = api.diffqkv_combine(to, tl, out_dtype=torch.float32, lse=lse)
    torch.cuda.synchronize()
    check_f32(out.cpu().numpy().astype(np.float64), ref)
    check_lse(lse.cpu().numpy().astype(np.float64), lse_ref, 1e-5)
    out_b = api.diffqkv_combine(to, tl, out_dtype=torch.bfloat16)
    check_bf16(out_b.float().cpu().numpy().astype(np.float64), ref)


def test_dominant_and_uniform_softmax(api, oracle):
    """Structured inputs: identical keys (uniform weights) and one dominant key (peaked weights)."""
    cfg = dataclasses.replace(SMALL, batch=2, kv_len=600)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([600, 431], np.int32))
    inp.k[:] = inp.k[:, :, :1]  # every token has the same key
    ref, _ = run_oracle(oracle, inp)
    out, _, _ = run_decode(api, inp)
    check_bf16(out, ref, "uniform")
    vf = W.as_f64(inp.v)
    for b, n in enumerate([600, 431]):
        for h in range(cfg.n_q):
            assert np.abs(out[b, h] - vf[b, h // 4, :n].mean(axis=0)).max() <= 2e-2
    inp2 = W.make_decode_inputs(cfg, seqlens=np.array([600, 431], np.int32))
    qf = W.bf16_bits_to_f32(inp2.q)
    inp2.k[:, :, 300] = W.f32_to_bf16_bits(4.0 * qf[:, ::8])  # dominant for the first head of each K group
    ref2, _ = run_oracle(oracle, inp2)
    out2, _, _ = run_decode(api, inp2)
    check_bf16(out2, ref2, "dominant")


def test_config5_full_size_sampled_rows(api, oracle):
    """Config 5 at its full size (64 sequences, lengths uniform in [1024, 65536], 16-token pages, shuffled page
    table, 6.4 GB of cache) in the launch configuration the benchmark times; the oracle recomputes a sample of
    (sequence, query head) rows from the same bytes copied back to the host."""
    import bench
    cfg = W.CFG5
    case = bench.DecodeCase(api, cfg, torch.device("cuda", 0))
    lse = torch.full((cfg.batch, cfg.n_q), float("nan"), dtype=torch.float32, device="cuda")
    out = torch.empty((cfg.batch, cfg.n_q, cfg.d_v), dtype=torch.float32, device="cuda")
    cache = case.caches[0]
    api.diffqkv_decode(case.q, cache, cfg.n_k, cfg.n_v, cfg.scale, workspace=case.workspace, out=out, lse=lse,
                       dev_status=case.status)
    torch.cuda.synchronize()
    assert int(case.status.item()) == 0 and api.last_decode_kernel() == api.KERNEL_TMA
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    k_host = cache.k.view(torch.uint16).cpu().numpy()
    v_host = cache.v.view(torch.uint16).cpu().numpy()
    q_host = case.q.view(torch.uint16).cpu().numpy()
    lens = case.seqlens_host
    ks, vs = tuple(cache.k.stride()[:3]), tuple(cache.v.stride()[:3])
    ocache = oracle.Cache(k_host, v_host, ks, vs, lens, cache.page_table.cpu().numpy(), cfg.page_size)
    g = np.random.Generator(np.random.Philox(key=555))
    seqs = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 0, cfg.batch - 1, *g.integers(0, cfg.batch, 4).tolist()})
    pairs = np.array([(b, h) for b in seqs for h in g.choice(cfg.n_q, 4, replace=False)], dtype=np.int32)
    ref, lse_ref = oracle.decode(q_host, ocache, cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v, cfg.scale, pairs=pairs)
    sel = (pairs[:, 0], pairs[:, 1])
    check_bf16(got[sel], ref[sel], "cfg5 full size")
    check_lse(lse.cpu().numpy().astype(np.float64)[sel], lse_ref[sel], 2e-2, "cfg5 full size")


def test_decode_from_and_to_host_memory(api, oracle, fixed_owners):
    """diffqkv_decode_host: q in pinned host memory, the result back in pinned host memory, same numbers as
    diffqkv_decode on device buffers (bitwise) and within tolerance of the oracle."""
    inp = W.make_decode_inputs(SMALL)
    cfg = inp.cfg
    cache = device_cache(api, inp)
    q_dev_in = W.to_torch(inp.q, "cuda")
    ref_out = api.diffqkv_decode(q_dev_in, cache, cfg.n_k, cfg.n_v, cfg.scale, out_dtype=torch.float32)
    q_host = W.to_torch(inp.q).pin_memory()
    out_host = torch.empty(ref_out.shape, dtype=torch.float32).pin_memory()
    q_dev, out_dev = torch.empty_like(q_dev_in), torch.empty_like(ref_out)
    shape = api.make_shape(cfg.batch, cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v, q_dev.dtype, torch.float32, cfg.scale)
    ws = torch.empty(max(api.diffqkv_decode_workspace_bytes(shape, int(inp.max_seqlen), 0), 256), dtype=torch.uint8,
                     device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(2):
        out_host.fill_(float("nan"))
        api.diffqkv_decode_host(q_host, q_dev, cache, cfg.n_k, cfg.n_v, cfg.scale, ws, out_dev, out_host,
                                dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(out_host, ref_out.cpu())
    ref, _ = run_oracle(oracle, inp)
    check_bf16(out_host.numpy().astype(np.float64), ref, "decode from host memory")


def test_split_counts_beyond_the_combine_limit_are_refused_before_any_launch(api):
    cfg = dataclasses.replace(W.CFG2, batch=1, kv_len=256)
    inp = W.make_decode_inputs(cfg)
    q, cache = W.to_torch(inp.q, "cuda"), device_cache(api, inp)
    launches = api.launch_count()
    with pytest.raises(api.DiffQKVError) as e:
        api.diffqkv_decode(q, cache, cfg.n_k, cfg.n_v, cfg.scale, num_splits=8193,
                           workspace=torch.zeros(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.status == api.ERR_UNSUPPORTED
    assert api.launch_count() == launches


@pytest.fixture
def per_head_only(api):
    """Switches the generic decode path to its one-block-per-query-head kernel and back."""
    yield api.decode_per_head_only
    api.decode_per_head_only(False)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("heads,d_qk,d_v", [((16, 2, 4), 64, 64), ((32, 4, 8), 128, 128), ((12, 6, 2), 128, 64),
                                            ((8, 8, 1), 64, 256), ((8, 1, 8), 256, 128), ((4, 4, 4), 128, 128),
                                            ((8, 2, 2), 64, 128)])
def test_generic_unit_kernel_and_per_head_kernel(api, oracle, per_head_only, dtype, heads, d_qk, d_v):
    """The generic path's unit kernel (every K and V row read once for all query heads of its unit) and its
    one-block-per-head kernel against the oracle and each other: fp32 and bf16 storage, nested head groups in both
    directions, mixed head dimensions, ragged and empty sequences, contiguous and paged, one and several splits."""
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, batch=4, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d_qk, d_v=d_v, kv_len=1100, dtype=dtype,
                              seed=77)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([1100, 1, 0, 517], dtype=np.int32))
    ref, lse_ref = run_oracle(oracle, inp)
    check = check_f32 if dtype == "f32" else check_bf16
    for case in (inp, W.paginate(inp, 16, seed=5)):
        for splits in (1, 5):
            outs = []
            for only in (False, True):
                per_head_only(only)
                out, lse, st = run_decode(api, case, num_splits=splits)
                assert st == 0 and api.last_decode_kernel() == api.KERNEL_GENERIC
                check(out, ref, f"{heads} {d_qk}/{d_v} {dtype} splits={splits} per_head={only}")
                check_lse(lse, lse_ref, 1e-4 if dtype == "f32" else 2e-2)
                assert np.all(out[2] == 0) and np.all(np.isneginf(lse[2]))
                outs.append(out)
            assert np.abs(outs[0] - outs[1]).max() <= (1e-5 if dtype == "f32" else 5e-3) * max(np.abs(ref).max(), 1.0)


@pytest.mark.parametrize("heads,d", [((6, 3, 2), 64), ((16, 2, 4), 96), ((32, 1, 2), 64)])
def test_generic_shapes_the_unit_kernel_does_not_take(api, oracle, heads, d):
    """Head groups that do not nest, head dimensions other than 64 / 128 / 256 and more than eight query heads per
    unit stay on the one-block-per-head kernel (fp32 storage)."""
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, batch=2, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d, d_v=d, kv_len=600, dtype="f32", seed=78)
    inp = W.make_decode_inputs(cfg, seqlens=np.array([600, 77], dtype=np.int32))
    ref, lse_ref = run_oracle(oracle, inp)
    out, lse, st = run_decode(api, inp)
    assert st == 0
    check_f32(out, ref, f"{heads} d={d}")
    check_lse(lse, lse_ref, 1e-4)


def test_unit_kernel_reports_pages_outside_the_pool(api):
    cfg = dataclasses.replace(SMALL, batch=1, kv_len=256, dtype="f32")
    inp = W.paginate(W.make_decode_inputs(cfg), 16, seed=1)
    inp.page_table[0, 3] = inp.num_pages + 5
    _, _, st = run_decode(api, inp)
    assert st == 1 << api.ERR_INDEX


@pytest.fixture
def cluster_mode(api):
    """Sets the on-chip-merge mode of the TMA kernel and always restores the automatic choice."""
    yield api.decode_cluster
    api.decode_cluster(-1)


@pytest.mark.parametrize("heads,d_qk,d_v", [((16, 2, 4), 128, 128), ((32, 4, 16), 64, 64), ((8, 4, 1), 128, 128),
                                            ((32, 1, 2), 128, 128), ((16, 2, 4), 64, 128), ((8, 8, 8), 128, 128)])
def test_rows_merged_on_chip_by_a_cluster(api, oracle, cluster_mode, heads, d_qk, d_v):
    """The blocks of a (sequence, unit) row as a thread-block cluster whose first block merges the others' shares out
    of their shared memory: one launch, no partials in global memory.  Against the oracle and against the two-kernel
    path, with rows of 47 tiles, of one tile (fewer tiles than blocks: most blocks of the cluster have none), of one
    token and empty ones, NaN bit patterns behind every sequence end, contiguous and paged."""
    n_q, n_k, n_v = heads
    cfg = dataclasses.replace(SMALL, batch=5, n_q=n_q, n_k=n_k, n_v=n_v, d_qk=d_qk, d_v=d_v, kv_len=3000, seed=93)
    lens = np.array([3000, 64, 0, 1777, 1], dtype=np.int32)
    inp = W.make_decode_inputs(cfg, seqlens=lens)
    for b, n in enumerate(lens):
        inp.k[b, :, n:] = 0x7FC0  # bf16 NaN
        inp.v[b, :, n:] = 0x7FC0
    ref, lse_ref = run_oracle(oracle, inp)
    for paged in (0, 16, 128):
        case = W.paginate(inp, paged, seed=7) if paged else inp
        cluster_mode(0)
        n0 = api.launch_count()
        out2, lse2, st2 = run_decode(api, case)
        two = api.launch_count() - n0
        cluster_mode(1)
        n0 = api.launch_count()
        out, lse, st = run_decode(api, case)
        one = api.launch_count() - n0
        what = f"{heads} d={d_qk}/{d_v} paged={paged}"
        assert st == 0 and st2 == 0 and api.last_decode_kernel() == api.KERNEL_TMA, what
        assert (one, two) == (1, 2), what + f": launches {one} / {two}"
        check_bf16(out, ref, what)
        check_lse(lse, lse_ref, 2e-2, what)
        assert np.all(out[2] == 0) and np.all(np.isneginf(lse[2])), what
        assert np.abs(out - out2).max() <= 5e-3, what


def test_cluster_merge_is_chosen_for_short_rows_only(api, oracle, cluster_mode):
    """Left to itself the library merges on chip where the fixed costs dominate (16 sequences of 4096 tokens: 32 rows of
    four blocks) and keeps the two-kernel path where the SMs it would leave idle cost more (the same heads at 8 times
    the capacity)."""
    short = dataclasses.replace(SMALL, batch=16, n_q=16, n_k=2, n_v=4, d_qk=128, d_v=128, kv_len=4096, seed=94)
    inp = W.make_decode_inputs(short)
    n0 = api.launch_count()
    out, lse, st = run_decode(api, inp)
    assert st == 0 and api.launch_count() - n0 == 1
    pairs = np.array([(0, 0), (3, 7), (15, 15), (9, 4)], dtype=np.int32)
    ref, _ = run_oracle(oracle, inp, pairs=pairs)
    check_bf16(out[pairs[:, 0], pairs[:, 1]], ref[pairs[:, 0], pairs[:, 1]], "short rows")
    # four sequences of the long-context heads have 16 rows, too few for clusters that fill the GPU: the units are
    # halved (two halves share their K head), which makes 32 rows of four blocks
    halves = dataclasses.replace(SMALL, batch=4, n_q=32, n_k=4, n_v=8, d_qk=128, d_v=128, kv_len=4096, seed=95)
    inp = W.make_decode_inputs(halves, seqlens=np.array([4096, 4000, 77, 2049], dtype=np.int32))
    n0 = api.launch_count()
    out, lse, st = run_decode(api, inp)
    assert st == 0 and api.launch_count() - n0 == 1
    ref, lse_ref = run_oracle(oracle, inp)
    check_bf16(out, ref, "halved units")
    check_lse(lse, lse_ref, 2e-2, "halved units")
    cluster_mode(0)
    out2, _, _ = run_decode(api, inp)
    cluster_mode(-1)
    assert np.abs(out - out2).max() <= 5e-3
    long_rows = dataclasses.replace(short, batch=2, kv_len=262144)
    q = torch.zeros(2, 16, 128, dtype=torch.bfloat16, device="cuda")
    cache = api.KVCache(torch.zeros(2, 2, 262144, 128, dtype=torch.bfloat16, device="cuda"),
                        torch.zeros(2, 4, 262144, 128, dtype=torch.bfloat16, device="cuda"),
                        torch.tensor([5000, 262144], dtype=torch.int32, device="cuda"), 262144)
    n0 = api.launch_count()
    api.diffqkv_decode(q, cache, 2, 4, long_rows.scale)
    torch.cuda.synchronize()
    assert api.launch_count() - n0 == 2


def test_bound_call_is_the_same_call(api, fixed_owners):
    """bind_decode builds the argument structs once; what it launches is the plain call."""
    inp = W.make_decode_inputs(SMALL)
    cfg = inp.cfg
    q, cache = W.to_torch(inp.q, "cuda"), device_cache(api, inp)
    ref = api.diffqkv_decode(q, cache, cfg.n_k, cfg.n_v, cfg.scale)
    shape = api.make_shape(cfg.batch, cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v, q.dtype, q.dtype, cfg.scale)
    ws = torch.empty(api.diffqkv_decode_workspace_bytes(shape, cache.max_seqlen, 0), dtype=torch.uint8, device="cuda")
    out = torch.full_like(ref, float("nan"))
    call = api.bind_decode(q, cache, cfg.n_k, cfg.n_v, cfg.scale, ws, out)
    for _ in range(3):
        assert call() is out
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.uint16), ref.view(torch.uint16))
