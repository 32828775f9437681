"""fc_decode_attention (the decoding step of Eq. 3-4 on the compacted cache) against the fp64 oracle.
Inputs are fp16/bf16 values; the kernel keeps fp32 sums and rounds the probabilities to the storage
type before the second product, so the bar is 2e-2 of the largest output magnitude of the head
(the 16-bit tolerance of the other parity tests), checked element by element."""
import numpy as np
import pytest
import torch

from oracle import flashcache_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fc():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2511_16786_b200 import binding
    return binding


def _run(fc, q, ck, cv, offsets, tail=None, max_rows=None):
    B = q.shape[0]
    h = fc.fc_create(0, 1024)
    try:
        qd, kd, vd = q.cuda(), ck.cuda(), cv.cuda()
        od = torch.tensor(offsets, dtype=torch.int64, device="cuda")
        tk = tv = tl = None
        n_tail = 0
        if tail is not None:
            tk, tv, tl = tail[0].cuda(), tail[1].cuda(), torch.tensor(tail[2], dtype=torch.int32, device="cuda")
            n_tail = max(tail[2])
        if max_rows is None:
            max_rows = max(offsets[b + 1] - offsets[b] for b in range(B)) + n_tail
        args = fc.make_decode_args(qd, kd, vd, od, max_rows, tk, tv, tl)
        need = fc.fc_decode_workspace_bytes(h, args)
        assert need > 0
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        out = torch.full(q.shape, float("nan"), dtype=q.dtype, device="cuda")
        fc.fc_decode_attention(h, args, out, ws)
        assert fc.fc_last_device_status(h) == 0
        return out.float().cpu().numpy().astype(np.float64)
    finally:
        fc.fc_destroy(h)


def _check(got, want, tol=2e-2):
    scale = np.abs(want).max(axis=-1, keepdims=True)
    scale = np.maximum(scale, 1e-6)
    err = np.abs(got - want) / scale
    assert err.max() <= tol, "attention error %.3e" % err.max()


def _inputs(rows, B, H, G, dtype, seed, peaked=False):
    g = torch.Generator().manual_seed(seed)
    d = 128
    ck = torch.randn((rows, H, d), generator=g).to(dtype)
    cv = torch.randn((rows, H, d), generator=g).to(dtype)
    q = torch.randn((B, H * G, d), generator=g)
    if peaked:
        q = q * 4.0                                   # a few rows carry most of the weight
    return q.to(dtype), ck, cv


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("lens,H,G", [([1], 1, 1), ([63, 64, 65], 2, 7), ([0, 300, 1, 4097], 4, 7),
                                      ([20000], 2, 16), ([777, 0], 3, 4)])
def test_decode_matches_oracle(fc, lens, H, G, dtype):
    offsets = [0] + [int(x) for x in np.cumsum(lens)]
    q, ck, cv = _inputs(max(offsets[-1], 1) + 5, len(lens), H, G, dtype, 31 + sum(lens))
    got = _run(fc, q, ck, cv, offsets)
    want = O.decode_attention(q.double().numpy(), ck.double().numpy(), cv.double().numpy(), offsets)
    _check(got, want)
    for b, n in enumerate(lens):
        if n == 0:
            assert not got[b].any()


def test_decode_with_uncompressed_tail_and_peaked_scores(fc):
    lens = [500, 0, 64, 3000]
    tail_len = [3, 17, 0, 100]
    offsets = [0] + [int(x) for x in np.cumsum(lens)]
    B, H, G, d = 4, 2, 7, 128
    q, ck, cv = _inputs(offsets[-1], B, H, G, torch.bfloat16, 5, peaked=True)
    g = torch.Generator().manual_seed(6)
    tk = torch.randn((B, 128, H, d), generator=g).to(torch.bfloat16)
    tv = torch.randn((B, 128, H, d), generator=g).to(torch.bfloat16)
    got = _run(fc, q, ck, cv, offsets, tail=(tk, tv, tail_len))
    want = O.decode_attention(q.double().numpy(), ck.double().numpy(), cv.double().numpy(), offsets,
                              tk.double().numpy(), tv.double().numpy(), tail_len)
    _check(got, want)
    # a generous bound on the rows changes the launch shape, not the result
    got2 = _run(fc, q, ck, cv, offsets, tail=(tk, tv, tail_len), max_rows=50000)
    _check(got2, want)


def test_decode_ignores_what_lies_past_the_valid_rows(fc):
    # rows after a sequence's last kept row (the next sequence's rows, rows after offsets[B]) and tail rows at or past
    # tail_len may hold anything, NaN and Inf bit patterns included: they have no weight and must not reach the output
    lens = [70, 1, 130]
    tail_len = [5, 0, 33]
    offsets = [0] + [int(x) for x in np.cumsum(lens)]
    B, H, G, d = 3, 2, 4, 128
    for dtype in (torch.bfloat16, torch.float16):
        q, ck, cv = _inputs(offsets[-1] + 100, B, H, G, dtype, 77)
        g = torch.Generator().manual_seed(78)
        tk = torch.randn((B, 64, H, d), generator=g).to(dtype)
        tv = torch.randn((B, 64, H, d), generator=g).to(dtype)
        want = O.decode_attention(q.double().numpy(), ck.double().numpy(), cv.double().numpy(), offsets,
                                  tk.double().numpy(), tv.double().numpy(), tail_len)
        poison = torch.tensor([float("nan"), float("inf"), -float("inf"), 1e30], dtype=torch.float32).to(dtype)
        ck[offsets[-1]:] = poison[0]
        cv[offsets[-1]:] = poison[torch.arange(cv[offsets[-1]:].numel()) % 4].view_as(cv[offsets[-1]:])
        for b in range(B):
            tk[b, tail_len[b]:] = poison[1]
            tv[b, tail_len[b]:] = poison[torch.arange(tv[b, tail_len[b]:].numel()) % 4].view_as(tv[b, tail_len[b]:])
        got = _run(fc, q, ck, cv, offsets, tail=(tk, tv, tail_len))
        assert np.isfinite(got).all()
        _check(got, want)
    # the last sequence's neighbour inside the cache: sequence 0's last tile also holds rows of sequence 1 and 2;
    # make those non-finite for a run that only looks at sequence 0
    q, ck, cv = _inputs(200, 1, 1, 2, torch.bfloat16, 79)
    want = O.decode_attention(q.double().numpy(), ck[:70].double().numpy(), cv[:70].double().numpy(), [0, 70])
    ck[70:] = float("nan")
    cv[70:] = float("inf")
    _check(_run(fc, q, ck, cv, [0, 70]), want)


def test_decode_closed_forms_on_the_device(fc):
    # zero query: the mean of the value rows; one row: that row
    g = torch.Generator().manual_seed(9)
    ck = torch.randn((200, 1, 128), generator=g).to(torch.float16)
    cv = torch.randn((200, 1, 128), generator=g).to(torch.float16)
    q = torch.zeros((2, 4, 128), dtype=torch.float16)
    got = _run(fc, q, ck, cv, [0, 199, 200])
    np.testing.assert_allclose(got[0, 2], cv[:199, 0].double().mean(dim=0).numpy(), atol=2e-3)
    np.testing.assert_allclose(got[1, 0], cv[199, 0].double().numpy(), atol=1e-3)


def test_decode_rejects_bad_arguments(fc):
    q, ck, cv = _inputs(10, 1, 2, 3, torch.bfloat16, 1)
    h = fc.fc_create(0, 64)
    try:
        od = torch.tensor([0, 10], dtype=torch.int64, device="cuda")
        args = fc.make_decode_args(q.cuda(), ck.cuda(), cv.cuda(), od, 10)
        args.head_dim = 64
        assert fc.fc_decode_workspace_bytes(h, args) == 0
        args.head_dim = 128
        args.num_q_heads = 5                                  # not a multiple of the KV heads
        assert fc.fc_decode_workspace_bytes(h, args) == 0
        args.num_q_heads = 6
        out = torch.empty((1, 6, 128), dtype=torch.bfloat16, device="cuda")
        ws = torch.empty(256, dtype=torch.uint8, device="cuda")
        with pytest.raises(fc.FlashCacheError) as e:
            fc.fc_decode_attention(h, args, out, ws[:16])
        assert e.value.code == 3
    finally:
        fc.fc_destroy(h)
