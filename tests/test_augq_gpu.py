"""GPU parity of diffqkv_augq (three tcgen05 GEMMs with the fused silu-gate epilogue) against the float64
oracle, called through the C ABI on the same seeded inputs.

Tolerance.  Products accumulate in fp32; x, a and q are each rounded to bf16 once (relative 2^-9 per element).
The float64 oracle rounds nothing, so the expected deviation is a few 2^-9 of the typical output magnitude:
the tests require max|err| <= 1e-2 * max|ref| (the relative bound of the bf16 mode), an rms error below
4e-3 of the rms of the reference, and element-wise |err| <= 2^-8 |ref| + 2e-2 rms(ref row) (helpers.check_proj).
"""
import numpy as np
import pytest
import torch

from paper_2501_13629_b200 import workloads as W
from helpers import check_proj

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def _weights(seed, d_model, d_q0, d_aug, d_out, gate_gain=1.0):
    return (W.normal(seed + 1, (d_q0, d_model), std=d_model ** -0.5),
            W.normal(seed + 2, (d_aug, d_q0), std=gate_gain * d_q0 ** -0.5),
            W.normal(seed + 3, (d_aug, d_q0), std=d_q0 ** -0.5),
            W.normal(seed + 4, (d_out, d_aug), std=d_aug ** -0.5))


def _run(api, h, ws):
    dev = "cuda"
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    q = api.diffqkv_augq(W.to_torch(h, dev), *(W.to_torch(w, dev) for w in ws), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return q.float().cpu().numpy().astype(np.float64)


def _check(out, ref, what):
    check_proj(out, ref, what)


@pytest.mark.parametrize("T", [1, 5, 16, 33, 64, 128, 300, 1000])
@pytest.mark.parametrize("dims", [(256, 384, 384, 256), (128, 128, 128, 128), (512, 256, 640, 384)])
def test_augq_small_shapes_every_row(api, oracle, T, dims):
    """Ragged row counts (tail tiles) and column counts that end in a half-filled 256-column tile."""
    d_model, d_q0, d_aug, d_out = dims
    h = W.normal(77, (T, d_model), std=1.0)  # unit-variance input: the gate is well inside the nonlinear range
    ws = _weights(100, d_model, d_q0, d_aug, d_out)
    ref = oracle.augq(h, *ws)
    _check(_run(api, h, ws), ref, f"T={T} dims={dims}")


def test_augq_zero_gate_gives_zero(api):
    d_model, d_q0, d_aug, d_out = 128, 256, 128, 128
    h = W.normal(5, (200, d_model))
    wq, _, wu, wd = _weights(7, d_model, d_q0, d_aug, d_out)
    wg = np.zeros((d_aug, d_q0), dtype=np.uint16)
    assert np.all(_run(api, h, (wq, wg, wu, wd)) == 0.0)


def test_augq_config4_widths_sampled_rows(api, oracle):
    """The prefill configuration's widths (hidden 2048 -> 4096 -> 3072 -> 4096) with hidden states N(0, 0.02) and
    seeded N(0, 1/fan_in) weights, 1100 rows on the GPU, a sample of rows through the oracle."""
    cfg = W.CFG4
    T = 1100
    d_q0 = cfg.n_q * cfg.d_qk
    h = W.normal(cfg.seed, (T, cfg.d_model), std=cfg.h_std)
    ws = _weights(cfg.seed, cfg.d_model, d_q0, cfg.d_aug, d_q0)
    rows = np.array([0, 1, 127, 128, 511, 640, 1023, 1024, 1099], dtype=np.int64)
    ref = oracle.augq(h, *ws, rows=rows)
    _check(_run(api, h, ws)[rows], ref, "cfg4 widths")
    # same widths, unit-variance input (a gate that is not nearly linear)
    h1 = W.normal(cfg.seed + 50, (T, cfg.d_model), std=1.0)
    ref1 = oracle.augq(h1, *ws, rows=rows)
    _check(_run(api, h1, ws)[rows], ref1, "cfg4 widths, unit input")


def test_augq_argument_errors(api):
    dev = "cuda"
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device=dev)
    with pytest.raises(api.DiffQKVError) as e:
        api.diffqkv_augq(z(4, 100), z(128, 100), z(128, 128), z(128, 128), z(128, 128))
    assert e.value.status == api.ERR_UNSUPPORTED
    with pytest.raises(api.DiffQKVError) as e:
        api.diffqkv_augq(z(4, 128), z(128, 128), z(128, 128), z(128, 128), z(128, 128),
                         workspace=torch.zeros(256, dtype=torch.uint8, device=dev))
    assert e.value.status == api.ERR_WORKSPACE
