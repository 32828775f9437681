"""fc_score_layer_static, the scoring entry point for callers that must not allocate
device memory (a process whose memory is owned by a framework pool, a plug-in that may
not allocate after start-up, a latency-critical path that cannot afford cudaMalloc's
implicit synchronisation).  It keeps its scratch in a fixed array inside the library, so
every call shares that array and finds the previous call's leftovers in it.

The test calls it through the C ABI twice in a row on different inputs and checks each
result against fc_score_layer (the entry point with a caller-provided workspace) within
the score tolerances of the parity tests; a further test holds it to the fp64 oracle directly.  It is collected last so that a failure here
cannot hide another test's result in a run that stops at the first failure, and it makes
no assumption about what ran before it in the process.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-3, torch.float16: 2e-2, torch.bfloat16: 2e-2}


@pytest.fixture(scope="module")
def fc():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2511_16786_b200 import binding
    return binding


def _inputs(lens, H, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    T = int(sum(lens))
    t = torch.arange(T, dtype=torch.float32)[:, None, None] / max(T, 1)
    k = 0.3 * torch.randn((T, H, d), generator=g) + 3.0 * torch.cos(40.0 * t + torch.randn((1, H, d), generator=g))
    v = 0.3 * torch.randn((T, H, d), generator=g) + 2.0 * t
    cu = [0]
    for n in lens:
        cu.append(cu[-1] + int(n))
    return k.to(dtype).cuda(), v.to(dtype).cuda(), cu


def _with_workspace(fc, k, v, cu, gamma):
    h = fc.fc_create(0, 4096)
    try:
        scores = torch.zeros((k.shape[1], k.shape[0]), dtype=torch.float32, device="cuda")
        energy = torch.zeros((len(cu) - 1, 4), dtype=torch.float64, device="cuda")
        ws = torch.empty(fc.fc_score_workspace_bytes(h, k, v, cu), dtype=torch.uint8, device="cuda")
        fc.fc_score_layer(h, k, v, cu, gamma, scores, energy, ws)
        assert fc.fc_last_device_status(h) == 0
        return scores.cpu().numpy().astype(np.float64), energy.cpu().numpy()
    finally:
        fc.fc_destroy(h)


def _static(fc, k, v, cu, gamma):
    scores = torch.full((k.shape[1], k.shape[0]), -1.0, dtype=torch.float32, device="cuda")
    energy = torch.full((len(cu) - 1, 4), -1.0, dtype=torch.float64, device="cuda")
    fc.fc_score_layer_static(k, v, cu, gamma, scores, energy)
    torch.cuda.synchronize()
    return scores.cpu().numpy().astype(np.float64), energy.cpu().numpy()


def _compare(fc, lens, H, d, dtype, seed, gamma=0.2):
    k, v, cu = _inputs(lens, H, d, dtype, seed)
    want, want_e = _with_workspace(fc, k, v, cu, gamma)
    got, got_e = _static(fc, k, v, cu, gamma)
    tol = TOL[dtype]
    kk, vv = k.double().cpu().numpy(), v.double().cpu().numpy()
    for b in range(len(cu) - 1):
        s, e = cu[b], cu[b + 1]
        if e == s:
            assert not got_e[b].any()
            continue
        for h in range(H):
            ebar = ((kk[s:e, h] ** 2).sum(1) + (vv[s:e, h] ** 2).sum(1)).mean() / d
            den = np.maximum(want[h, s:e], 1e-6 * ebar)
            err = float((np.abs(got[h, s:e] - want[h, s:e]) / den).max())
            assert err <= tol, "sequence %d head %d: score error %.3e" % (b, h, err)
        np.testing.assert_allclose(got_e[b, [1, 3]], want_e[b, [1, 3]], rtol=1e-6)
        np.testing.assert_allclose(got_e[b, [0, 2]], want_e[b, [0, 2]], rtol=tol)


def test_two_calls_in_a_row_match_the_workspace_entry_point(fc):
    assert fc.fc_static_scratch_bytes() == 8 << 20
    # first call: ragged batch (chirp path, tiny, empty, and power-of-two lengths), bf16
    _compare(fc, [300, 0, 1024, 17, 2048], 3, 128, torch.bfloat16, 1)
    # second call straight after, different shape and dtype: the scratch still holds the first call's data
    _compare(fc, [4096, 777], 2, 128, torch.float32, 2)
    # and once more with the first shape: results do not depend on what the scratch held
    _compare(fc, [300, 0, 1024, 17, 2048], 3, 128, torch.bfloat16, 1)


def test_static_entry_point_matches_the_oracle(fc):
    # the same check the workspace entry point gets: element by element against the fp64 oracle on a small ragged
    # batch (chirp path, empty sequence, power of two), and the status word of the static calls reads clean
    from oracle import flashcache_oracle as O
    for dtype, seed in ((torch.float32, 11), (torch.bfloat16, 12)):
        k, v, cu = _inputs([257, 0, 512, 33], 2, 128, dtype, seed)
        got, got_e = _static(fc, k, v, cu, 0.2)
        assert fc.fc_static_last_device_status() == 0
        kk, vv = k.double().cpu().numpy(), v.double().cpu().numpy()
        want, want_e = O.score_layer(kk, vv, cu, 0.2, "fft")
        tol = TOL[dtype]
        for b in range(len(cu) - 1):
            s0, e0 = cu[b], cu[b + 1]
            if e0 == s0:
                continue
            for h in range(2):
                ebar = ((kk[s0:e0, h] ** 2).sum(1) + (vv[s0:e0, h] ** 2).sum(1)).mean() / 128
                den = np.maximum(want[h, s0:e0], 1e-6 * ebar)
                err = float((np.abs(got[h, s0:e0] - want[h, s0:e0]) / den).max())
                assert err <= tol, "sequence %d head %d: score error %.3e" % (b, h, err)
            np.testing.assert_allclose(got_e[b, [1, 3]], want_e[b, [1, 3]], rtol=1e-5)
            np.testing.assert_allclose(got_e[b, [0, 2]], want_e[b, [0, 2]], rtol=max(tol, 1e-4), atol=1e-6 * want_e[b, 1])


def test_sizes_beyond_the_fixed_scratch_are_refused(fc):
    k, v, cu = _inputs([4097], 1, 128, torch.float32, 3)
    scores = torch.zeros((1, 4097), dtype=torch.float32, device="cuda")
    energy = torch.zeros((1, 4), dtype=torch.float64, device="cuda")
    with pytest.raises(fc.FlashCacheError) as e:
        fc.fc_score_layer_static(k, v, cu, 0.2, scores, energy)          # longer than 4096
    assert e.value.code == 2
    k, v, cu = _inputs([4096], 1, 256, torch.float32, 4)
    scores = torch.zeros((1, 4096), dtype=torch.float32, device="cuda")
    with pytest.raises(fc.FlashCacheError) as e:
        fc.fc_score_layer_static(k, v, cu, 0.2, scores, energy)          # 4096 x 256 complex values alone fill 8 MiB
    assert e.value.code == 3


def test_other_lengths_up_to_the_limit_fit(fc):
    # the chirp path transforms a head in 32-column groups here, so every length up to 4096 fits
    _compare(fc, [3000, 4095], 2, 128, torch.float32, 5)
    _compare(fc, [2500], 1, 256, torch.bfloat16, 6)
