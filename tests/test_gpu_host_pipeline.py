"""fc_compress_host (host buffers in, host buffers out) against the per-stage entry points on
device buffers and against the fp64 oracle.  The kernels are the same, so budgets, indices and
rows must be identical to the per-stage path; the oracle comparison uses the tolerances of
test_gpu_parity.py."""
import numpy as np
import pytest
import torch

from oracle import flashcache_oracle as O
from paper_2511_16786_b200 import synth_kv as S

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-3, torch.float16: 2e-2, torch.bfloat16: 2e-2}


@pytest.fixture(scope="module")
def fc():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2511_16786_b200 import binding
    return binding


def _layers(cfg, pin=True):
    Ks, Vs = [], []
    for l in range(cfg.num_layers):
        k, v = S.make_layer(cfg, l, "cpu")
        Ks.append(k.pin_memory() if pin else k)
        Vs.append(v.pin_memory() if pin else v)
    return Ks, Vs


def _per_stage(fc, cfg, Ks, Vs, per_layer=False, protect=None):
    comp = fc.Compressor(cfg.num_layers, cfg.num_heads, cfg.head_dim, cfg.cu_seqlens, cfg.torch_dtype, cfg.rho,
                         cfg.gamma, cfg.min_keep, per_layer=per_layer,
                         protect=None if protect is None else protect.cuda())
    Kd, Vd = [k.cuda() for k in Ks], [v.cuda() for v in Vs]
    comp.compress(Kd, Vd)
    comp.check_device_status()
    out = (comp.budgets.cpu().numpy(), comp.offsets.cpu().numpy(), comp.out_idx.cpu(), comp.out_k.cpu(), comp.out_v.cpu())
    comp.close()
    return out


def _check_against_per_stage(cfg, res, ref):
    budgets, offsets, idx, ok, ov = ref
    np.testing.assert_array_equal(res.budgets.numpy(), budgets)
    np.testing.assert_array_equal(res.offsets.numpy(), offsets)
    rows = 0
    for l in range(cfg.num_layers):
        assert int(res.layer_rows[l]) == rows
        r = int(offsets[l, -1])
        rows += r
        k, v, i = res.layer(l)
        assert tuple(i.shape) == (cfg.num_heads, r)
        assert torch.equal(i, idx[l, :, :r])
        assert torch.equal(k.view(torch.uint8), ok[l, :r].contiguous().view(torch.uint8))
        assert torch.equal(v.view(torch.uint8), ov[l, :r].contiguous().view(torch.uint8))
    assert int(res.layer_rows[cfg.num_layers]) == rows


def test_host_pipeline_matches_per_stage_calls_and_oracle(fc):
    base = S.paper_configs()["cfg5"]
    cfg = S.scaled(base, "host_small", num_layers=5, seqlens=(300, 0, 1024, 17, 2048))
    Ks, Vs = _layers(cfg)
    ref = _per_stage(fc, cfg, Ks, Vs)
    hc = fc.HostCompressor(cfg.num_layers, cfg.num_heads, cfg.head_dim, cfg.cu_seqlens, cfg.torch_dtype, cfg.rho,
                           cfg.gamma, cfg.min_keep)
    assert hc.rows == int(ref[0].sum())                     # the budgets add up to B_tot per sequence
    res = hc.new_result()
    hc.compress(Ks, Vs, res)
    torch.cuda.synchronize()
    hc.check_device_status()
    _check_against_per_stage(cfg, res, ref)

    # the oracle's rule on the oracle's scores: kept sets agree except next to the threshold, rows are copies
    cu, tol = cfg.cu_seqlens, TOL[cfg.torch_dtype]
    for l in range(cfg.num_layers):
        o, _ = O.score_layer(Ks[l].double().numpy(), Vs[l].double().numpy(), cu, cfg.gamma, "fft")
        k, v, idx = res.layer(l)
        for h in range(cfg.num_heads):
            for b, n in enumerate(cfg.seqlens):
                kb, off = int(res.budgets[l, b]), int(res.offsets[l, b])
                got = idx[h, off:off + kb].numpy()
                osc = o[h, cu[b]:cu[b + 1]]
                diff = np.setxor1d(got, O.select_topk(osc, kb))
                if len(diff) and kb > 0:
                    tau = np.sort(osc)[::-1][kb - 1]
                    assert np.all(np.abs(osc[diff] - tau) <= tol * tau)
                assert torch.equal(k[off:off + kb, h].contiguous().view(torch.uint8),
                                   Ks[l][cu[b] + got, h].contiguous().view(torch.uint8))
    hc.close()


def test_back_to_back_jobs_share_the_arena(fc):
    # three jobs in a row without a host synchronisation in between, alternating two result sets and two
    # different inputs: every job must see its own inputs although the next one's copies are already queued
    base = S.paper_configs()["cfg3"]
    cfg_a = S.scaled(base, "host_a", num_layers=4, seqlens=(4096,))
    cfg_b = S.scaled(base, "host_b", num_layers=4, seqlens=(4096,), seed=base.seed + 17)
    Ka, Va = _layers(cfg_a)
    Kb, Vb = _layers(cfg_b)
    ref_a = _per_stage(fc, cfg_a, Ka, Va)
    ref_b = _per_stage(fc, cfg_b, Kb, Vb)
    assert not np.array_equal(ref_a[2].numpy(), ref_b[2].numpy())
    hc = fc.HostCompressor(cfg_a.num_layers, cfg_a.num_heads, cfg_a.head_dim, cfg_a.cu_seqlens, cfg_a.torch_dtype,
                           cfg_a.rho, cfg_a.gamma, cfg_a.min_keep)
    r0, r1 = hc.new_result(), hc.new_result()
    hc.compress(Ka, Va, r0)
    hc.compress(Kb, Vb, r1)
    torch.cuda.synchronize()
    _check_against_per_stage(cfg_a, r0, ref_a)
    _check_against_per_stage(cfg_b, r1, ref_b)
    hc.compress(Ka, Va, r1)
    torch.cuda.synchronize()
    hc.check_device_status()
    _check_against_per_stage(cfg_a, r1, ref_a)
    hc.close()


def test_pageable_inputs_and_bad_arguments(fc):
    base = S.paper_configs()["cfg3"]
    cfg = S.scaled(base, "host_pageable", num_layers=2, seqlens=(1000, 2048))
    Ks, Vs = _layers(cfg, pin=False)
    ref = _per_stage(fc, cfg, Ks, Vs)
    hc = fc.HostCompressor(cfg.num_layers, cfg.num_heads, cfg.head_dim, cfg.cu_seqlens, cfg.torch_dtype, cfg.rho,
                           cfg.gamma, cfg.min_keep)
    res = hc.new_result()
    hc.compress(Ks, Vs, res)
    torch.cuda.synchronize()
    _check_against_per_stage(cfg, res, ref)
    # fewer output rows than the budgets need: refused before anything is copied back
    small = fc.HostResult(cfg.num_layers, cfg.num_heads, cfg.head_dim, len(cfg.seqlens), hc.rows - 1, cfg.torch_dtype)
    with pytest.raises(fc.FlashCacheError) as e:
        hc.compress(Ks, Vs, small)
    assert e.value.code == 3
    # an arena that is too small
    hc._job.arena_bytes = hc._job.arena_bytes - 256
    with pytest.raises(fc.FlashCacheError) as e:
        hc.compress(Ks, Vs, res)
    assert e.value.code == 3
    hc.close()


def test_host_pipeline_with_selection_options(fc):
    base = S.paper_configs()["cfg2"]
    cfg = S.scaled(base, "host_options", num_layers=3, seqlens=(1024, 600), min_keep=24)
    Ks, Vs = _layers(cfg)
    cu = cfg.cu_seqlens
    protect = torch.zeros(cu[-1], dtype=torch.uint8)
    for b in range(2):
        protect[cu[b]:cu[b] + 4] = 1
        protect[cu[b + 1] - 16:cu[b + 1]] = 1
    protect = protect.pin_memory()
    ref = _per_stage(fc, cfg, Ks, Vs, per_layer=True, protect=protect)
    hc = fc.HostCompressor(cfg.num_layers, cfg.num_heads, cfg.head_dim, cu, cfg.torch_dtype, cfg.rho, cfg.gamma,
                           cfg.min_keep, per_layer=True, protect=protect)
    res = hc.new_result()
    hc.compress(Ks, Vs, res)
    torch.cuda.synchronize()
    hc.check_device_status()
    _check_against_per_stage(cfg, res, ref)
    k, v, idx = res.layer(0)
    assert torch.equal(idx[0], idx[1])                                   # one index set per layer
    got = set(idx[0, :int(res.budgets[0, 0])].tolist())
    assert set(range(4)) <= got and set(range(1024 - 16, 1024)) <= got   # the marked tokens of sequence 0 survive
    hc.close()
