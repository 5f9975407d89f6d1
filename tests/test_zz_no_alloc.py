"""diffqkv_decode_static: the decode entry point for hosts that cannot allocate device memory.

A server that gave all device memory to its own pool at start-up, or code that sits behind an
interface without a workspace argument, still has to decode.  This entry point keeps the split
kernel's partial results in an 8 MiB array compiled into the library, so the caller passes only
inputs and outputs.  The test calls it through the C ABI twice in a row (the second call finds the
first call's partials still in the array) and compares each result with the ordinary entry point.
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_bf16, device_cache, run_oracle

pytestmark = pytest.mark.gpu


def _both_ways(api, inp, num_splits):
    cfg = inp.cfg
    q = W.to_torch(inp.q, "cuda")
    cache = device_cache(api, inp)
    ref_out = api.diffqkv_decode(q, cache, cfg.n_k, cfg.n_v, cfg.scale, num_splits=num_splits,
                                 out_dtype=torch.float32)
    out = torch.full((cfg.batch, cfg.n_q, cfg.d_v), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((cfg.batch, cfg.n_q), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    before = torch.cuda.memory_allocated()
    api.diffqkv_decode_static(q, cache, cfg.n_k, cfg.n_v, cfg.scale, out, num_splits=num_splits, lse=lse,
                              dev_status=status)
    assert torch.cuda.memory_allocated() == before  # the wrapper allocated nothing through torch either
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.cpu().numpy().astype(np.float64), ref_out.cpu().numpy().astype(np.float64), lse.cpu().numpy()


def test_static_scratch_decode_matches_workspace_decode_twice(oracle):
    from paper_2501_13629_b200 import api
    api.set_tail_reserve(0)  # fixed tile owners: the two entry points then differ in nothing but the scratch memory
    try:
        _twice(api, oracle)
    finally:
        api.set_tail_reserve(-1)


def _twice(api, oracle):
    big = dataclasses.replace(W.CFG2, batch=3, kv_len=2500, seed=81)
    small = dataclasses.replace(W.CFG2, batch=2, n_q=8, n_k=2, n_v=2, kv_len=300, seed=82)
    first = W.make_decode_inputs(big, seqlens=np.array([2500, 1200, 9], np.int32))
    second = W.make_decode_inputs(small, seqlens=np.array([300, 0], np.int32))
    for inp, splits in ((first, 0), (second, 3)):  # the second call sees the first call's leftovers
        out, same_path, lse = _both_ways(api, inp, splits)
        ref, lse_ref = run_oracle(oracle, inp)
        check_bf16(out, ref, inp.cfg.name)
        check_bf16(same_path, ref, inp.cfg.name)
        assert np.abs(out - same_path).max() <= 1e-6  # same kernels, same chunking: the scratch is all that differs
        finite = np.isfinite(lse_ref)
        assert np.abs(lse[finite] - lse_ref[finite]).max() <= 2e-2
    assert np.all(out[1] == 0.0)  # the empty sequence of the second call


def test_static_scratch_rejects_oversized_shapes():
    from paper_2501_13629_b200 import api
    cfg = dataclasses.replace(W.CFG2, batch=64, n_q=32, n_k=4, n_v=8, kv_len=128, seed=83)
    inp = W.make_decode_inputs(cfg)
    q = W.to_torch(inp.q, "cuda")
    cache = device_cache(api, inp)
    cache.max_seqlen = 1 << 20  # a bound this large needs far more than 8 MiB of partials
    shape = api.make_shape(cfg.batch, cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v, q.dtype, torch.float32, cfg.scale)
    assert api.diffqkv_decode_workspace_bytes(shape, cache.max_seqlen, 0) > api.STATIC_SCRATCH_BYTES
    out = torch.zeros((cfg.batch, cfg.n_q, cfg.d_v), dtype=torch.float32, device="cuda")
    launches = api.launch_count()
    with pytest.raises(api.DiffQKVError) as e:
        api.diffqkv_decode_static(q, cache, cfg.n_k, cfg.n_v, cfg.scale, out)
    assert e.value.status == api.ERR_WORKSPACE
    assert api.launch_count() == launches  # refused on the host, nothing was launched


def test_static_scratch_agrees_with_decode_on_an_empty_batch():
    """batch == 0 is a valid call that does nothing, through either entry point."""
    from paper_2501_13629_b200 import api
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device="cuda")  # noqa: E731
    cache = api.KVCache(z(1, 2, 64, 128), z(1, 2, 64, 128), torch.zeros(1, dtype=torch.int32, device="cuda"), 64)
    q = z(1, 8, 128)  # real storage behind the pointers; the shape says batch 0 (torch gives empty tensors a null pointer)
    out = torch.zeros((1, 8, 128), dtype=torch.float32, device="cuda")
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    shape = api.make_shape(0, 8, 2, 2, 128, 128, q.dtype, out.dtype, 0.1)
    cs = cache.c_struct()
    launches = api.launch_count()
    import ctypes as C
    st = api._lib.diffqkv_decode(q.data_ptr(), C.byref(cs), C.byref(shape), 0, ws.data_ptr(), ws.numel(), out.data_ptr(),
                                 None, None, None)
    assert st == api.OK
    st = api._lib.diffqkv_decode_static(q.data_ptr(), C.byref(cs), C.byref(shape), 0, out.data_ptr(), None, None, None)
    assert st == api.OK
    assert api.launch_count() == launches
