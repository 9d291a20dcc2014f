"""tri_score_static: the scoring entry point for callers that cannot allocate device memory when they
call (a server whose KV page pool already owns all of HBM, a plug-in that must stay out of its host
application's allocator).  Its scratch is a 16 MiB array built into the library, so the checks here
are: same results as tri_score on two calls in a row that share that array (the second on another
shape, so anything left over from the first would show), no device allocation by the calls, and a
clean refusal of shapes that do not fit.  Collected last on purpose: it is an add-on to the round."""
import pytest
import torch

from paper_2604_04921_b200 import binding as tb
from paper_2604_04921_b200 import workloads as W

from parity import REL, make_ctx, src_view

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _close(a, b):
    return bool(torch.all((a - b).abs() <= REL * torch.clamp(b.abs(), min=1.0)))


def _both(w):
    sp = w.spec
    ctx = make_ctx(w)
    src = src_view(w)
    S, U, N, G = sp.n_seqs, w.k.shape[0] * sp.n_seqs * sp.n_kv_heads, src.c_view().n_max, sp.group_size
    ws = ctx.workspace(S, N, sp.budget)
    want_s = torch.zeros(U, N, dtype=torch.float32, device=DEV)
    want_r = torch.zeros(U, N, G, dtype=torch.float32, device=DEV)
    ctx.score(src, w.cur_pos, want_s, ws, raw=want_r)
    got_s, got_r = torch.zeros_like(want_s), torch.zeros_like(want_r)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    ctx.score_static(src, w.cur_pos, got_s, raw=got_r)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before          # the call took nothing from torch's allocator
    return ctx, (want_s, want_r), (got_s, got_r)


def test_static_scratch_scoring_matches_tri_score_twice_in_a_row():
    base = W.SPECS["qwen3_8b_oneshot_32k"]
    # first call: 2 layers x 2 heads x 5,000 keys, three scoring blocks per unit
    w1 = W.make_workload(base.scaled(name="noalloc1", n_layers=2, n_kv_heads=2, n_keys=5000, budget=300), DEV)
    _, want1, got1 = _both(w1)
    assert _close(got1[0], want1[0]) and _close(got1[1], want1[1])
    # second call, straight after, on a smaller ragged batch: the array still holds the first call's data
    sp2 = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="noalloc2", n_layers=1, n_kv_heads=2, n_seqs=3, n_keys=1200,
                                                   n_keys_min=100, budget=128)
    w2 = W.make_workload(sp2, DEV)
    _, want2, got2 = _both(w2)
    n_max = got2[0].shape[1]
    valid = (torch.arange(n_max, device=DEV)[None, :] < w2.seq_lens.repeat_interleave(sp2.n_kv_heads)[:, None])
    assert _close(got2[0][valid], want2[0][valid]) and _close(got2[1][valid], want2[1][valid])
    assert float(got2[0][valid].abs().max()) > 0.1          # real scores, not the zero fill


def test_static_scratch_rejects_shapes_beyond_its_array():
    import ctypes
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
