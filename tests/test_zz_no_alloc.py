"""tri_score_static: the scoring entry point for callers that cannot allocate device memory when they
call (a server whose KV page pool already owns all of HBM, a plug-in that must stay out of its host
application's allocator).  Its scratch is a 16 MiB array built into the library, so the checks here
are: same results as tri_score (and as the CPU oracle) on calls in a row that share that array, with the
raw scores kept inside the array as well as handed to the caller, so that anything left over from the
previous call would show; no device memory taken by the calls (the driver's own free-memory figure, not a
framework's allocator counter); shapes right at the array's limit accepted and one step beyond it refused
before anything is launched.  Collected last on purpose: it is an add-on to the round."""
import ctypes

import pytest
import torch

from paper_2604_04921_b200 import binding as tb
from paper_2604_04921_b200 import workloads as W

from parity import REL, check_scores, make_ctx, oracle_unit, src_view

pytestmark = pytest.mark.gpu
DEV = "cuda"
LIMIT = 16 * 1024 * 1024


def _close(a, b):
    return bool(torch.all((a - b).abs() <= REL * torch.clamp(b.abs(), min=1.0)))


def _both(w):
    """tri_score, then tri_score_static twice: once with the raw scores going to the caller, once with them
    staying in the built-in array.  Returns the reference and both results."""
    sp = w.spec
    ctx = make_ctx(w)
    src = src_view(w)
    S, U, N, G = sp.n_seqs, w.k.shape[0] * sp.n_seqs * sp.n_kv_heads, src.c_view().n_max, sp.group_size
    ws = ctx.workspace(S, N, sp.budget)
    want_s = torch.zeros(U, N, dtype=torch.float32, device=DEV)
    want_r = torch.zeros(U, N, G, dtype=torch.float32, device=DEV)
    ctx.score(src, w.cur_pos, want_s, ws, raw=want_r)
    got_s, got_r, got_s2 = torch.zeros_like(want_s), torch.zeros_like(want_r), torch.zeros_like(want_s)
    ctx.score_static(src, w.cur_pos, got_s2)               # first use on this device: looks the array up
    got_s2.zero_()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]             # cudaMemGetInfo: sees any cudaMalloc, whoever makes it
    ctx.score_static(src, w.cur_pos, got_s, raw=got_r)
    ctx.score_static(src, w.cur_pos, got_s2)               # raw scores live in the shared array this time
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before     # the calls took no device memory
    return ctx, (want_s, want_r), (got_s, got_r, got_s2)


def test_static_scratch_scoring_matches_tri_score_twice_in_a_row():
    base = W.SPECS["qwen3_8b_oneshot_32k"]
    # first shape: 2 layers x 2 heads x 5,000 keys, three scoring blocks per unit
    w1 = W.make_workload(base.scaled(name="noalloc1", n_layers=2, n_kv_heads=2, n_keys=5000, budget=300), DEV)
    _, want1, got1 = _both(w1)
    assert _close(got1[0], want1[0]) and _close(got1[1], want1[1]) and _close(got1[2], want1[0])
    ref = oracle_unit(w1, 1, 0, 1, 300)                    # and against the CPU oracle, one unit
    u = 3
    check_scores(got1[1][u].cpu().numpy(), got1[2][u].cpu().numpy(), ref)
    # second shape, straight after, a smaller ragged batch: the array still holds the first shape's data
    sp2 = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="noalloc2", n_layers=1, n_kv_heads=2, n_seqs=3, n_keys=1200,
                                                   n_keys_min=100, budget=128)
    w2 = W.make_workload(sp2, DEV)
    _, want2, got2 = _both(w2)
    n_max = got2[0].shape[1]
    valid = (torch.arange(n_max, device=DEV)[None, :] < w2.seq_lens.repeat_interleave(sp2.n_kv_heads)[:, None])
    assert _close(got2[0][valid], want2[0][valid]) and _close(got2[1][valid], want2[1][valid])
    assert _close(got2[2][valid], want2[0][valid])
    assert float(got2[0][valid].abs().max()) > 0.1          # real scores, not the zero fill


def _scratch_need(ctx, S, U, n_max):
    """Bytes of the built-in array a shape uses, as the library states them; checked here against the header's
    account of what goes there (1 KiB of phasors per sequence, 4 G bytes of raw scores per key, 16 G bytes of partial
    sums per scoring block of at least 1,024 keys, each area rounded up to 256 bytes; G = 4 here)."""
    need = ctx.score_static_bytes(S, n_max)
    raw = U * n_max * 16
    assert raw + 1024 * S <= need <= raw + 1024 * S + U * (n_max // 1024 + 1) * 64 + 3 * 256
    return need


def test_static_scratch_limit_is_exact():
    """One head, G = 4: the largest row capacity whose scratch fits the array is accepted and scores like
    tri_score; 16 rows more is refused."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="noalloc4", n_layers=1, n_kv_heads=1, n_keys=3000, budget=32)
    w = W.make_workload(sp, DEV)
    ctx = make_ctx(w)
    n_fit = 1040000
    while _scratch_need(ctx, 1, 1, n_fit + 16) <= LIMIT:
        n_fit += 16
    assert _scratch_need(ctx, 1, 1, n_fit) <= LIMIT < _scratch_need(ctx, 1, 1, n_fit + 16)
    assert 1040000 < n_fit < 1048576                        # 16 B of raw scores per key, plus phasors and partial sums
    # the cache holds 3,000 keys; the view claims capacity for n_fit rows (only seq_lens rows are ever read)
    k = torch.zeros(1, 1, 1, n_fit + 16, 128, dtype=torch.bfloat16, device=DEV)
    k[..., :3000, :] = w.k
    scores = torch.zeros(1, n_fit, dtype=torch.float32, device=DEV)
    ctx.score_static(tb.CacheView(k[..., :n_fit, :], None, seq_lens=w.seq_lens), w.cur_pos, scores)
    want = torch.zeros(1, 3000, dtype=torch.float32, device=DEV)
    ctx.score(src_view(w), w.cur_pos, want, ctx.workspace(1, 3000, 32))
    torch.cuda.synchronize()
    assert _close(scores[:, :3000], want) and bool((scores[:, 3000:] == 0).all())
    over = torch.zeros(1, n_fit + 16, dtype=torch.float32, device=DEV)
    with pytest.raises(tb.TriError) as e:
        ctx.score_static(tb.CacheView(k, None, seq_lens=w.seq_lens), w.cur_pos, over)
    assert e.value.code == 3 and f"needs {_scratch_need(ctx, 1, 1, n_fit + 16)} bytes" in str(e.value)
    torch.cuda.synchronize()
    assert bool((over == 0).all())


def test_static_scratch_rejects_shapes_beyond_its_array():
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="noalloc3", n_layers=1, n_kv_heads=1, n_keys=256, budget=32)
    w = W.make_workload(sp, DEV)
    ctx = make_ctx(w)
    # a view that claims 8 M rows per unit needs 128 MiB of raw scores: refused on the host before any
    # launch, so none of the pointers is followed
    cv = tb.CacheView(w.k, w.v, seq_lens=w.seq_lens, n_max=8 * 1024 * 1024).c_view()
    scores = torch.zeros(16, dtype=torch.float32, device=DEV)
    code = tb.lib().tri_score_static(ctx._h, ctypes.byref(cv), 1, w.cur_pos.data_ptr(), scores.data_ptr(), None, None)
    assert code == 3
    msg = tb.lib().tri_last_cuda_error().decode()
    assert "needs 134" in msg and "built-in array holds 16777216" in msg
    torch.cuda.synchronize()
    assert torch.all(scores == 0)
