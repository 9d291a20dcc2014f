"""GPU parity: the CUDA library, called through its C ABI, against the float64 CPU oracle on the same
seeded inputs.  Sizes are chosen so that the oracle finishes in seconds while every unit still spans
several scoring blocks and a ragged tail."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_04921_b200 import binding as tb
from paper_2604_04921_b200 import workloads as W

from parity import (check_compacted, check_kept, check_scores, check_unit, make_ctx, oracle_unit, out_rows, run_compress,
                    src_view, unit_index)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _all_units(w):
    return [(l, s, h) for l in range(w.k.shape[0]) for s in range(w.spec.n_seqs) for h in range(w.spec.n_kv_heads)]


def test_config0_tiny_bf16_post_rope():
    w = W.make_workload(W.SPECS["tiny"], DEV)
    B = w.spec.budget
    ref = oracle_unit(w, 0, 0, 0, B)
    res = run_compress(w, B)
    st = check_unit(w, res, ref, 0, 0, 0, B)
    assert int(res["status"].item()) == 0
    assert int(res["new_seq_lens"][0].item()) == B
    assert st["raw_err"] < 0.1      # far inside the tolerance: errors are ~1e-5 relative


def test_config0_tiny_fp32_pre_rope():
    """The configuration's own input format: fp32 pre-RoPE keys, position = slot."""
    w = W.make_workload(W.SPECS["tiny"], DEV)
    sp, B = w.spec, w.spec.budget
    kpre = w.k_pre_fp32
    N = sp.n_keys
    qc = w.q_center[0].double().numpy()
    qn = w.q_mean_norm[0].double().numpy()
    raw_o = oracle.score_raw(kpre[0, 0, 0].double().cpu().numpy(), np.arange(N), N, qc, qn, theta=sp.theta)
    _, s_o = oracle.normalize(raw_o)
    idx_o = oracle.select(s_o, B)
    ctx = make_ctx(w)
    src = tb.CacheView(kpre, None, seq_lens=w.seq_lens)
    ws = ctx.workspace(1, N, B)
    scores = torch.empty(1, N, dtype=torch.float32, device=DEV)
    raw = torch.empty(1, N, 1, dtype=torch.float32, device=DEV)
    ctx.score(src, w.cur_pos, scores, ws, raw=raw)
    ref = dict(raw=raw_o, s_final=s_o, idx=idx_o)
    check_scores(raw[0].cpu().numpy(), scores[0].cpu().numpy(), ref)
    kout = torch.zeros(1, 1, 1, B, 128, dtype=torch.float32, device=DEV)
    kept_idx = torch.empty(1, B, dtype=torch.int32, device=DEV)
    kept_cnt = torch.empty(1, dtype=torch.int32, device=DEV)
    ctx.compress(src, w.cur_pos, B, tb.CacheView(kout, None), ws, kept_idx=kept_idx, kept_cnt=kept_cnt)
    torch.cuda.synchronize()
    check_kept(kept_idx[0].cpu().numpy(), int(kept_cnt[0]), ref, B)
    sel = kept_idx[0].long()
    assert torch.equal(kout[0, 0, 0], kpre[0, 0, 0][sel])


@pytest.mark.parametrize("G,layout", [(4, 0), (8, 0), (3, 1)])
def test_bf16_pre_rope_keys(G, layout):
    """k_kind 2: the cache holds the pre-RoPE vectors k_f of Section 4.1 in bf16, each slot with its position (here
    scattered, ascending, up to 60,000 below the query).  Scored in fp32 with tabulated distance phasors; against the
    oracle's pre-RoPE reading on the same bf16 values, then selection and compaction as for any cache."""
    N, B, H = 2500, 300, 2
    sp = W.SPECS["tiny"].scaled(name=f"pre{G}{layout}", n_kv_heads=H, group_size=G, n_keys=N, budget=B)
    w = W.make_workload(sp, DEV)
    kpre = w.k_pre_fp32.to(torch.bfloat16)                                   # [1, 1, H, N, 128], interleaved pairs
    g = torch.Generator().manual_seed(9)
    pos = torch.stack([torch.sort(torch.randperm(50000, generator=g)[:N]).values for _ in range(H)]).to(torch.int32)
    p_q = 60000
    qc, qn = w.q_center, w.q_mean_norm
    k_dev, qc_dev = kpre, qc
    if layout == 1:
        perm = torch.cat([torch.arange(0, 128, 2), torch.arange(1, 128, 2)])
        k_dev, qc_dev = kpre[..., perm.to(DEV)].contiguous(), qc[..., perm].contiguous()
    ctx = tb.TriContext(1, H, G, qc_dev, qn, rope_theta=sp.theta, pair_layout=layout)
    positions = pos.view(1, 1, H, N).to(DEV)
    cur = torch.tensor([p_q], dtype=torch.int64, device=DEV)
    src = tb.CacheView(k_dev, w.v, seq_lens=w.seq_lens, positions=positions, pre_rope=True)
    ws = ctx.workspace(1, N, B)
    scores = torch.empty(H, N, dtype=torch.float32, device=DEV)
    raw = torch.empty(H, N, G, dtype=torch.float32, device=DEV)
    ctx.score(src, cur, scores, ws, raw=raw)
    k2 = torch.zeros(1, 1, H, B, 128, dtype=torch.bfloat16, device=DEV); v2 = torch.zeros_like(k2)
    p2 = torch.zeros(1, 1, H, B, dtype=torch.int32, device=DEV)
    idx = torch.empty(H, B, dtype=torch.int32, device=DEV); cnt = torch.empty(H, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ctx.compress(src, cur, B, tb.CacheView(k2, v2, positions=p2, pre_rope=True), ws, kept_idx=idx, kept_cnt=cnt, device_status=status)
    torch.cuda.synchronize()
    assert int(status) == 0
    for h in range(H):
        raw_o = oracle.score_raw(kpre[0, 0, h].double().cpu().numpy(), pos[h].numpy(), p_q, qc[0, h * G:(h + 1) * G].double().numpy(),
                                 qn[0, h * G:(h + 1) * G].double().numpy(), theta=sp.theta)
        _, s_o = oracle.normalize(raw_o)
        ref = dict(raw=raw_o, s_final=s_o, idx=oracle.select(s_o, B), k=k_dev[0, 0, h].cpu(), v=w.v[0, 0, h].cpu(), pos=pos[h].long())
        check_scores(raw[h].cpu().numpy(), scores[h].cpu().numpy(), ref)
        got = idx[h].cpu().numpy()
        check_kept(got, int(cnt[h]), ref, B)
        check_compacted(k2[0, 0, h], v2[0, 0, h], p2[0, 0, h], got, ref)
    # a distance outside the phasor tables is reported, not mis-scored silently
    far = torch.tensor([p_q + (1 << 21)], dtype=torch.int64, device=DEV)
    ctx.compress(src, far, B, tb.CacheView(k2, v2, positions=p2, pre_rope=True), ws, kept_idx=idx, kept_cnt=cnt, device_status=status)
    torch.cuda.synchronize()
    assert int(status) == 5


def test_config1_shape_scaled():
    """Qwen3-8B head geometry (G = 4), 2 layers x 2 KV heads, 5,000 keys: 3 scoring blocks + ragged tail."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(n_layers=2, n_kv_heads=2, n_keys=5000, budget=300)
    w = W.make_workload(sp, DEV)
    res = run_compress(w, sp.budget)
    assert int(res["status"].item()) == 0
    for (l, s, h) in _all_units(w):
        check_unit(w, res, oracle_unit(w, l, s, h, sp.budget), l, s, h, sp.budget)


def test_config2_shape_steady_state():
    """Batch of sequences holding budget + 128 keys at scattered original positions."""
    sp = W.SPECS["qwen3_8b_steady_b64"].scaled(n_layers=1, n_kv_heads=2, n_seqs=3)
    w = W.make_workload(sp, DEV)
    res = run_compress(w, sp.budget)
    assert res["new_seq_lens"].tolist() == [sp.budget] * 3
    for (l, s, h) in _all_units(w):
        check_unit(w, res, oracle_unit(w, l, s, h, sp.budget), l, s, h, sp.budget)


def test_config3_shape_mixed_noise():
    """Per-head noise std in [0.2, 1.0]: concentrated and diffuse heads in one launch."""
    sp = W.SPECS["qwen3_8b_long_128k"].scaled(n_layers=1, n_kv_heads=3, n_keys=12345, budget=1000)
    w = W.make_workload(sp, DEV)
    res = run_compress(w, sp.budget)
    for (l, s, h) in _all_units(w):
        check_unit(w, res, oracle_unit(w, l, s, h, sp.budget), l, s, h, sp.budget)


@pytest.mark.parametrize("in_place", [False, True])
def test_config4_shape_ragged_paged(in_place):
    """G = 8, ragged lengths, 16-token pages in a shuffled table; compacted rows go back into pages."""
    sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(n_layers=2, n_kv_heads=2, n_seqs=3, n_keys=2500, n_keys_min=300,
                                                  budget=512)
    w = W.make_workload(sp, DEV)
    refs = {u: oracle_unit(w, *u, sp.budget) for u in _all_units(w)}      # before any in-place write
    res = run_compress(w, sp.budget, in_place=in_place)
    assert int(res["status"].item()) == 0
    lens = w.seq_lens.tolist()
    assert res["new_seq_lens"].tolist() == [min(n, sp.budget) for n in lens]
    for u, ref in refs.items():
        check_unit(w, res, ref, *u, sp.budget)


@pytest.mark.parametrize("page_size,G", [(64, 4), (32, 8), (128, 8)])
def test_other_page_sizes(page_size, G):
    """Pages of 32, 64 and 128 tokens (any multiple of 16 is accepted), both scoring kernels' copy loops, in place."""
    sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(name=f"pg{page_size}", n_layers=1, n_kv_heads=2, n_seqs=3, n_keys=3000,
                                                  n_keys_min=500, budget=400, page_size=page_size, group_size=G)
    w = W.make_workload(sp, DEV)
    refs = {u: oracle_unit(w, *u, sp.budget) for u in _all_units(w)}
    res = run_compress(w, sp.budget, in_place=True)
    assert int(res["status"].item()) == 0
    for u, ref in refs.items():
        check_unit(w, res, ref, *u, sp.budget)


def test_token_major_page_layout():
    """Pages stored [layer][page][slot][head][128] (head stride 128, slot stride H * 128): the view's strides
    describe it, nothing else changes."""
    sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="tokmajor", n_layers=2, n_kv_heads=2, n_seqs=2, n_keys=1800,
                                                  n_keys_min=400, budget=256)
    w = W.make_workload(sp, DEV)
    ref = run_compress(w, sp.budget)
    # same pool, token-major in memory, exposed through a permuted (strided) view of the usual index order
    w2 = W.Workload(sp, w.q_center, w.q_mean_norm, w.k.permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4),
                    w.v.permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4), w.seq_lens, w.cur_pos, None, w.page_table)
    assert w2.k.stride()[2:4] == (128, sp.n_kv_heads * 128)
    res = run_compress(w2, sp.budget, in_place=True)
    assert int(res["status"].item()) == 0
    assert torch.equal(res["kept_idx"], ref["kept_idx"])
    assert torch.equal(torch.nan_to_num(res["raw"]), torch.nan_to_num(ref["raw"]))      # unwritten entries stay NaN
    for (l, s, h) in _all_units(w):
        cnt = int(ref["kept_cnt"][unit_index(w, l, s, h)])
        k_a, v_a, _ = out_rows(w, ref, l, s, h, cnt)
        k_b, v_b, _ = out_rows(w2, res, l, s, h, cnt)
        assert torch.equal(k_a.view(torch.int16), k_b.view(torch.int16)) and torch.equal(v_a.view(torch.int16), v_b.view(torch.int16))


def test_in_place_contiguous_matches_out_of_place():
    sp = W.SPECS["qwen3_8b_steady_b64"].scaled(n_layers=1, n_kv_heads=2, n_seqs=2)
    w = W.make_workload(sp, DEV)
    a = run_compress(w, sp.budget, want_scores=False)
    k0, v0, p0 = w.k.clone(), w.v.clone(), w.positions.clone()
    b = run_compress(w, sp.budget, in_place=True, want_scores=False)
    assert torch.equal(a["kept_idx"], b["kept_idx"])
    B = sp.budget
    assert torch.equal(a["k_out"].view(torch.int16), w.k[:, :, :, :B].view(torch.int16))
    assert torch.equal(a["v_out"].view(torch.int16), w.v[:, :, :, :B].view(torch.int16))
    assert torch.equal(a["pos_out"], w.positions[:, :, :, :B])
    # rows beyond the budget are untouched
    assert torch.equal(k0[:, :, :, B:].view(torch.int16), w.k[:, :, :, B:].view(torch.int16))
    assert torch.equal(p0[:, :, :, B:], w.positions[:, :, :, B:])


@pytest.mark.parametrize("G", [1, 2, 3, 5, 8, 16])
def test_group_sizes(G):
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name=f"g{G}", n_layers=1, n_kv_heads=2, group_size=G, n_keys=1111,
                                                budget=100)
    w = W.make_workload(sp, DEV)
    res = run_compress(w, sp.budget)
    for (l, s, h) in _all_units(w):
        check_unit(w, res, oracle_unit(w, l, s, h, sp.budget), l, s, h, sp.budget)


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("shape", ["g4", "g8_paged", "g16", "g3_half_split"])
def test_both_score_kernels(kernel, shape):
    """The tcgen05 kernel (0) and the mma.sync kernel (1) on the same inputs, each against the oracle, whatever the
    default for the group size is: several 128-key tiles per block, a ragged last tile, paged keys, 32 accumulator
    columns (G = 16) and the half-split band layout."""
    base = W.SPECS["qwen3_8b_oneshot_32k"]
    layout = 0
    if shape == "g4":
        sp = base.scaled(name="k_g4", n_layers=1, n_kv_heads=2, n_keys=9001, budget=700)
    elif shape == "g8_paged":
        sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="k_g8", n_layers=2, n_kv_heads=2, n_seqs=2, n_keys=5000,
                                                      n_keys_min=1000, budget=512)
    elif shape == "g16":
        sp = base.scaled(name="k_g16", n_layers=1, n_kv_heads=1, group_size=16, n_keys=4500, budget=300)
    else:
        sp = base.scaled(name="k_g3", n_layers=1, n_kv_heads=2, group_size=3, n_keys=3333, budget=200)
        layout = 1
    w = W.make_workload(sp, DEV)
    if layout == 1:
        perm = torch.cat([torch.arange(0, 128, 2), torch.arange(1, 128, 2)])
        w = W.Workload(sp, w.q_center[..., perm].contiguous(), w.q_mean_norm, w.k[..., perm.to(DEV)].contiguous(),
                       w.v, w.seq_lens, w.cur_pos, None, None)
    ctx = make_ctx(w, pair_layout=layout)
    ctx.set_score_kernel(kernel)
    res = run_compress(w, sp.budget, ctx=ctx)
    assert int(res["status"].item()) == 0
    for (l, s, h) in _all_units(w):
        check_unit(w, res, oracle_unit(w, l, s, h, sp.budget, layout=layout), l, s, h, sp.budget)


@pytest.mark.parametrize("norm_variant", [1, 2])
def test_norm_variants(norm_variant):
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="nv", n_layers=1, n_kv_heads=1, n_keys=2000, budget=128)
    w = W.make_workload(sp, DEV)
    ctx = make_ctx(w, norm_variant=norm_variant)
    res = run_compress(w, sp.budget, ctx=ctx)
    check_unit(w, res, oracle_unit(w, 0, 0, 0, sp.budget, norm_variant=norm_variant), 0, 0, 0, sp.budget)


def test_other_offset_sets():
    """The offset ablation's sets are runtime parameters (Appendix on future offsets)."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="off", n_layers=1, n_kv_heads=1, n_keys=1500, budget=64)
    w = W.make_workload(sp, DEV)
    for offs in ([1], [1, 2, 4, 8, 16, 32, 64, 128], list(range(1, 65537, 4096)) + [65536]):
        ctx = make_ctx(w, offsets=offs)
        res = run_compress(w, sp.budget, ctx=ctx)
        check_unit(w, res, oracle_unit(w, 0, 0, 0, sp.budget, offsets=offs), 0, 0, 0, sp.budget)


def test_half_split_layout():
    """pair_layout 1: band f = (x[f], x[f+64]).  Same data permuted must give the same result."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="hs", n_layers=1, n_kv_heads=2, n_keys=1800, budget=200)
    w = W.make_workload(sp, DEV)
    perm = torch.cat([torch.arange(0, 128, 2), torch.arange(1, 128, 2)])
    res0 = run_compress(w, sp.budget)
    w2 = W.Workload(sp, w.q_center[..., perm].contiguous(), w.q_mean_norm, w.k[..., perm.to(DEV)].contiguous(),
                    w.v, w.seq_lens, w.cur_pos, None, None)
    ctx = make_ctx(w2, pair_layout=1)
    res1 = run_compress(w2, sp.budget, ctx=ctx)
    assert torch.equal(res0["kept_idx"], res1["kept_idx"])
    assert torch.allclose(res0["raw"], res1["raw"], rtol=0, atol=2e-4)
    for (l, s, h) in _all_units(w2):
        kk, vv, pos = w2.unit_rows(l, s, h)
        G = sp.group_size
        raw, sfin, idx = oracle.unit_bf16(W.bf16_bits(kk), pos.numpy(), int(w2.cur_pos[s]),
                                          w2.q_center[l, h * G:(h + 1) * G].double().numpy(),
                                          w2.q_mean_norm[l, h * G:(h + 1) * G].double().numpy(), sp.budget, layout=1)
        check_unit(w2, res1, dict(raw=raw, s_final=sfin, idx=idx, k=kk, v=vv, pos=pos), l, s, h, sp.budget)


def test_degenerate_sizes():
    """N <= B keeps everything in order; N = 1; B = 1; a sequence of length 0 beside a full one."""
    base = W.SPECS["qwen3_8b_oneshot_32k"]
    for n, B in [(100, 512), (512, 512), (1, 4), (700, 1), (17, 16)]:
        sp = base.scaled(name=f"deg{n}_{B}", n_layers=1, n_kv_heads=2, n_keys=n, budget=B)
        w = W.make_workload(sp, DEV)
        res = run_compress(w, B)
        for (l, s, h) in _all_units(w):
            check_unit(w, res, oracle_unit(w, l, s, h, B), l, s, h, B)
        if n <= B:
            u = res["kept_idx"][:, :n].cpu()
            assert torch.equal(u, torch.arange(n, dtype=torch.int32).expand_as(u))
    # ragged batch with an empty sequence
    sp = base.scaled(name="empty", n_layers=1, n_kv_heads=1, n_seqs=3, n_keys=600, budget=64)
    w = W.make_workload(sp, DEV)
    w.seq_lens = torch.tensor([600, 0, 37], dtype=torch.int32, device=DEV)
    w.cur_pos = torch.tensor([600, 0, 37], dtype=torch.int64, device=DEV)
    res = run_compress(w, 64)
    assert res["kept_cnt"].tolist() == [64, 0, 37]
    assert res["new_seq_lens"].tolist() == [64, 0, 37]
    for s in (0, 2):
        check_unit(w, res, oracle_unit(w, 0, s, 0, 64), 0, s, 0, 64)
    assert torch.all(res["k_out"][0, 1] == 0)


def test_random_shapes_against_oracle():
    """Twenty seeded random shapes (layers, heads, group size, batch, lengths, budget; contiguous, steady-state
    positions or paged; in place or not) -- every unit against the oracle."""
    import random
    rnd = random.Random(20260404)
    for case in range(20):
        kind = rnd.choice(["oneshot", "steady", "ragged_paged"])
        L, H, G, S = rnd.randint(1, 2), rnd.randint(1, 3), rnd.choice([1, 2, 3, 4, 6, 8]), rnd.randint(1, 3)
        N = rnd.choice([17, 100, 333, 1024, 1999, 3100])
        B = max(1, min(N + 50, int(N * rnd.choice([0.05, 0.3, 0.9, 1.2]))))
        base = {"oneshot": "qwen3_8b_oneshot_32k", "steady": "qwen3_8b_steady_b64", "ragged_paged": "qwen3_32b_ragged_paged"}[kind]
        extra = {}
        if kind == "steady":
            N = max(N, 200)
            extra = dict(n_new=min(128, N // 2), pos_lo=N, pos_hi=N + 5000)
        if kind == "ragged_paged":
            extra = dict(n_keys_min=max(1, N // 4))
        sp = W.SPECS[base].scaled(name=f"rand{case}", n_layers=L, n_kv_heads=H, group_size=G, n_seqs=S, n_keys=N,
                                  budget=B, **extra)
        w = W.make_workload(sp, DEV)
        in_place = kind != "oneshot" and rnd.random() < 0.5
        refs = {u: oracle_unit(w, *u, B) for u in _all_units(w)}       # before any in-place write
        res = run_compress(w, B, in_place=in_place)
        assert int(res["status"].item()) == 0, (case, kind)
        for u, ref in refs.items():
            check_unit(w, res, ref, *u, B)


def test_decode_windows_in_place_over_several_rounds():
    """The deployed loop (Section 4.3): every 128 decoded tokens the cache, budget + 128 rows, is compressed in
    place back to the budget; survivors keep their original positions.  Four rounds on the device against the
    oracle applied to the same evolving cache on the host."""
    B, beta, rounds = 384, 128, 4
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="loop", n_layers=1, n_kv_heads=2, n_keys=B + beta * rounds, budget=B)
    full = W.make_workload(sp, DEV)                     # the whole decode: slot i = position i
    L, S, H, G, cap = 1, 1, 2, sp.group_size, B + beta
    k = torch.zeros(L, S, H, cap, 128, dtype=torch.bfloat16, device=DEV); v = torch.zeros_like(k)
    pos = torch.zeros(L, S, H, cap, dtype=torch.int32, device=DEV)
    k[..., :B, :], v[..., :B, :] = full.k[..., :B, :], full.v[..., :B, :]
    pos[..., :B] = torch.arange(B, dtype=torch.int32, device=DEV)
    lens = torch.tensor([B], dtype=torch.int32, device=DEV)
    ctx = make_ctx(full)
    ws = ctx.workspace(S, cap, B)
    view = tb.CacheView(k, v, seq_lens=lens, positions=pos)
    host = [dict(k=full.k[0, 0, h, :B].cpu(), v=full.v[0, 0, h, :B].cpu(), pos=torch.arange(B)) for h in range(H)]
    for r in range(rounds):
        t0 = B + beta * r                               # the window's tokens: positions t0 .. t0 + beta - 1
        k[..., B:, :], v[..., B:, :] = full.k[..., t0:t0 + beta, :], full.v[..., t0:t0 + beta, :]
        pos[..., B:] = torch.arange(t0, t0 + beta, dtype=torch.int32, device=DEV)
        lens.fill_(cap)
        cur = torch.tensor([t0 + beta], dtype=torch.int64, device=DEV)
        ctx.compress(view, cur, B, view, ws, new_seq_lens=lens)
        torch.cuda.synchronize()
        assert lens.tolist() == [B]
        for h in range(H):
            st = host[h]
            kk = torch.cat([st["k"], full.k[0, 0, h, t0:t0 + beta].cpu()])
            vv = torch.cat([st["v"], full.v[0, 0, h, t0:t0 + beta].cpu()])
            pp = torch.cat([st["pos"], torch.arange(t0, t0 + beta)])
            _, s_o, idx_o = oracle.unit_bf16(W.bf16_bits(kk), pp.numpy(), t0 + beta, full.q_center[0, h * G:(h + 1) * G].double().numpy(),
                                             full.q_mean_norm[0, h * G:(h + 1) * G].double().numpy(), B, theta=sp.theta)
            got_pos = pos[0, 0, h, :B].cpu().long()
            want_pos = pp[torch.from_numpy(idx_o.astype(np.int64))]
            assert torch.all(got_pos[1:] > got_pos[:-1])
            if not torch.equal(got_pos, want_pos):     # only keys in the tie band may differ
                diff = np.setxor1d(got_pos.numpy(), want_pos.numpy())
                s_b = np.sort(s_o)[::-1][B - 1]
                where = np.isin(pp.numpy(), diff)
                assert np.all(np.abs(s_o[where] - s_b) <= 1e-3 * max(1.0, abs(s_b)))
            # the rows on the device are bit copies of the rows its kept positions name; the host copy of the cache
            # follows the DEVICE's choice, so a tie-band swap does not make later rounds incomparable
            sel = torch.from_numpy(np.searchsorted(pp.numpy(), got_pos.numpy()))
            assert torch.equal(pp[sel], got_pos)
            assert torch.equal(k[0, 0, h, :B].cpu().view(torch.int16), kk[sel].view(torch.int16))
            assert torch.equal(v[0, 0, h, :B].cpu().view(torch.int16), vv[sel].view(torch.int16))
            host[h] = dict(k=kk[sel], v=vv[sel], pos=got_pos)


def test_lengths_updated_in_place_with_many_units():
    """new_seq_lens may be the array the round reads its lengths from (a decode loop updating them in place).
    With far more units than one wave of thread blocks, every unit must still see the old length: a length
    stored early by one block would make the later blocks of that sequence keep rows 0..B-1 instead of the top B."""
    sp = W.SPECS["qwen3_8b_steady_b64"].scaled(name="alias", n_layers=8, n_kv_heads=8, n_seqs=64, n_keys=400, budget=256,
                                               n_new=144, pos_lo=400, pos_hi=4000)
    w = W.make_workload(sp, DEV)
    B, S, H, L = sp.budget, sp.n_seqs, sp.n_kv_heads, sp.n_layers
    lens0 = torch.randint(300, 401, (S,), dtype=torch.int32, device=DEV, generator=torch.Generator(DEV).manual_seed(7))
    w.seq_lens = lens0.clone()
    ctx = make_ctx(w)
    src = src_view(w)
    U = L * S * H
    ws = ctx.workspace(S, sp.n_keys, B)
    ref_idx = torch.full((U, B), -1, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(U, dtype=torch.int32, device=DEV)
    k2 = torch.zeros(L, S, H, B, 128, dtype=torch.bfloat16, device=DEV); v2 = torch.zeros_like(k2)
    p2 = torch.zeros(L, S, H, B, dtype=torch.int32, device=DEV)
    dst = tb.CacheView(k2, v2, positions=p2)
    separate = torch.zeros(S, dtype=torch.int32, device=DEV)
    ctx.compress(src, w.cur_pos, B, dst, ws, kept_idx=ref_idx, kept_cnt=cnt, new_seq_lens=separate)
    torch.cuda.synchronize()
    assert separate.tolist() == [B] * S and w.seq_lens.tolist() == lens0.tolist()
    for rep in range(3):                                   # aliased: three times, the race was timing dependent
        w.seq_lens.copy_(lens0)
        idx = torch.full((U, B), -1, dtype=torch.int32, device=DEV)
        ctx.compress(src, w.cur_pos, B, dst, ws, kept_idx=idx, kept_cnt=cnt, new_seq_lens=w.seq_lens)
        torch.cuda.synchronize()
        assert w.seq_lens.tolist() == [B] * S
        assert torch.equal(idx, ref_idx), rep
    keep_all = torch.arange(B, dtype=torch.int32, device=DEV)
    assert not bool((ref_idx == keep_all).all(dim=1).any())      # no unit took the keep-everything path
    w.seq_lens.copy_(lens0)
    res = dict(kept_idx=ref_idx, kept_cnt=cnt, k_out=k2, v_out=v2, pos_out=p2)
    for (l, s, h) in [(0, 0, 0), (3, 17, 5), (7, 63, 7), (5, 40, 2)]:
        check_unit(w, res, oracle_unit(w, l, s, h, B), l, s, h, B)


@pytest.mark.parametrize("kind", ["contiguous", "paged_in_place"])
def test_budget_per_unit(kind):
    """Head-specific budgets (the future work of Appendix A): every (layer, sequence, head) keeps its own number of
    rows, drawn in [B/4, B], with a few units at 0, at 1 and above their length.  Every unit against the oracle run
    with that unit's budget; tri_select_budgets on the exported scores gives the same indices."""
    if kind == "contiguous":
        sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="ub", n_layers=2, n_kv_heads=3, n_seqs=2, n_keys=3000, budget=512)
    else:
        sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="ub_p", n_layers=2, n_kv_heads=2, n_seqs=3, n_keys=2500,
                                                      n_keys_min=600, budget=512)
    w = W.make_workload(sp, DEV)
    B, L, S, H = sp.budget, sp.n_layers, sp.n_seqs, sp.n_kv_heads
    U = L * S * H
    g = torch.Generator().manual_seed(3)
    ub = torch.randint(B // 4, B + 1, (U,), generator=g, dtype=torch.int32)
    ub[1], ub[2], ub[U - 1], ub[U - 2] = 0, 1, 10 ** 6, -5          # nothing, one row, clamped to B, negative = nothing
    ub_d = ub.to(DEV)
    refs = {}
    for (l, s_, h) in _all_units(w):
        b_u = int(min(max(int(ub[unit_index(w, l, s_, h)]), 0), B))
        refs[(l, s_, h)] = (b_u, oracle_unit(w, l, s_, h, max(b_u, 1)))
    res = run_compress(w, B, in_place=(kind != "contiguous"), unit_budgets=ub_d)
    assert int(res["status"].item()) == 0
    lens = w.seq_lens.tolist()
    per_seq = [0] * S
    for (l, s_, h), (b_u, ref) in refs.items():
        u = unit_index(w, l, s_, h)
        cnt = int(res["kept_cnt"][u])
        assert cnt == min(b_u, lens[s_])
        per_seq[s_] = max(per_seq[s_], cnt)
        if b_u == 0:
            continue
        check_unit(w, res, ref, l, s_, h, b_u)
    assert res["new_seq_lens"].tolist() == per_seq
    # selection alone, from the scores the round exported
    idx = torch.full((U, B), -1, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(U, dtype=torch.int32, device=DEV)
    n_max = res["scores"].shape[1]
    res["ctx"].select(res["scores"], w.seq_lens, n_max, B, idx, cnt, unit_budgets=ub_d)
    torch.cuda.synchronize()
    assert torch.equal(cnt, res["kept_cnt"])
    valid = torch.arange(B, device=DEV)[None, :] < cnt[:, None]
    assert torch.equal(idx[valid], res["kept_idx"][valid])


def test_only_overflowing_sequences_are_touched():
    """A batch in which one sequence exceeds the budget and two do not: the short ones are kept whole, in order,
    and the round gives the same kept rows for the long one as a batch holding it alone."""
    base = W.SPECS["qwen3_8b_oneshot_32k"]
    sp = base.scaled(name="due", n_layers=1, n_kv_heads=2, n_seqs=3, n_keys=900, budget=256)
    w = W.make_workload(sp, DEV)
    w.seq_lens = torch.tensor([200, 900, 256], dtype=torch.int32, device=DEV)
    w.cur_pos = torch.tensor([200, 900, 256], dtype=torch.int64, device=DEV)
    res = run_compress(w, 256, want_scores=False)
    assert res["kept_cnt"].tolist() == [200, 200, 256, 256, 256, 256]
    assert res["new_seq_lens"].tolist() == [200, 256, 256]
    for s_, n_ in ((0, 200), (2, 256)):
        for h in range(2):
            u = unit_index(w, 0, s_, h)
            assert res["kept_idx"][u, :n_].tolist() == list(range(n_))
            assert torch.equal(res["k_out"][0, s_, h, :n_].view(torch.int16), w.k[0, s_, h, :n_].view(torch.int16))
    for h in range(2):
        check_unit(w, res, oracle_unit(w, 0, 1, h, 256), 0, 1, h, 256)


def test_constant_head_contributes_zero():
    """A query head with zero centre and E|q_f| = 0 scores every key 0: sigma = 0, z = 0 for that head."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="const", n_layers=1, n_kv_heads=1, group_size=2, n_keys=900,
                                                budget=90)
    w = W.make_workload(sp, DEV)
    w.q_center[0, 1] = 0
    w.q_mean_norm[0, 1] = 0
    res = run_compress(w, sp.budget)
    ref = oracle_unit(w, 0, 0, 0, sp.budget)
    assert np.all(ref["raw"][1] == 0)
    check_unit(w, res, ref, 0, 0, 0, sp.budget)
    assert float(res["scores"][0, :900].min()) >= 0.0


def test_head_with_spread_of_a_few_ulps_counts_as_constant():
    """Reading of Section 4.3 for sigma_g = 0, at its boundary.  A head whose raw scores differ only by a few units in
    the last place of fp32 (relative spread ~1e-7) is below what fp32 scoring can resolve: the library treats it as
    constant (z = 0 for every key: var <= 1e-12 mu^2), while the float64 oracle, exact on the bf16 inputs, still sees a
    spread and z-scores it.  Both behaviours are pinned here: the device's final scores equal the oracle's with that
    head's raw scores made exactly constant, and differ from the oracle's on the raw scores as they are."""
    N, B, G = 2000, 150, 2
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="ulps", n_layers=1, n_kv_heads=1, group_size=G, n_keys=N, budget=B)
    w = W.make_workload(sp, DEV)
    # head 1: zero centre, E|q_f| = 1 on bands 0 and 1 only  ->  raw_1(k) = |k_0| + |k_1|
    w.q_center[0, 1] = 0
    w.q_mean_norm[0, 1] = 0
    w.q_mean_norm[0, 1, :2] = 1.0
    # band 0 = (64, 0) for every key, band 1 = (j * 2^-17, 0) with j in 1..4: raw_1 = 64 + j ulps (ulp(64) = 2^-17)
    j = (torch.arange(N) % 4 + 1).to(torch.float32)
    w.k[0, 0, 0, :, 0] = 64.0
    w.k[0, 0, 0, :, 1] = 0.0
    w.k[0, 0, 0, :, 2] = (j * 2.0 ** -17).to(torch.bfloat16).to(DEV)
    w.k[0, 0, 0, :, 3] = 0.0
    res = run_compress(w, B)
    ref = oracle_unit(w, 0, 0, 0, B)
    raw_o = ref["raw"]
    assert 0 < raw_o[1].max() - raw_o[1].min() <= 4 * 2.0 ** -17           # the oracle sees 1..4 ulps of spread
    _, s_plain = oracle.normalize(raw_o)
    flat = raw_o.copy()
    flat[1] = 64.0
    _, s_flat = oracle.normalize(flat)
    got = res["scores"][0, :N].cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - s_flat) <= 1e-3 * np.maximum(np.abs(s_flat), 1.0))      # device: head 1 contributes 0
    assert float(got.min()) >= 0.0
    assert np.max(np.abs(s_plain - s_flat)) > 0.5                                      # oracle as is: head 1 z-scored
    check_kept(res["kept_idx"][0].cpu().numpy(), int(res["kept_cnt"][0]), dict(s_final=s_flat, idx=oracle.select(s_flat, B)), B)


def test_select_bit_exact_with_ties():
    """tri_select alone on fp32 scores full of ties: indices must equal the oracle's exactly."""
    g = torch.Generator().manual_seed(5)
    cases = [(1, 5000, 777, 50), (3, 131072, 4096, 0), (4, 9999, 9998, 7), (2, 4096, 1, 3), (2, 70000, 35000, 1000),
             (1, 32768, 100, 20), (2, 32769, 30000, 0), (1, 500000, 4096, 5000),
             # very few distinct values: the threshold's value bin overflows the candidate list
             (1, 50000, 20000, 3), (2, 200000, 4096, 2), (1, 3000, 1500, 1)]
    for U, n, B, levels in cases:
        x = torch.randn(U, n, generator=g)
        if levels:
            x = torch.round(x * levels / 6) / levels          # many exactly equal values
        x[0, : min(n, 10)] = 0.0
        sc = x.to(DEV)
        lens = torch.tensor([n], dtype=torch.int32, device=DEV)
        ctx = tb.TriContext(U, 1, 1, torch.zeros(U, 1, 128), torch.zeros(U, 1, 64))
        idx = torch.full((U, B), -1, dtype=torch.int32, device=DEV)
        cnt = torch.zeros(U, dtype=torch.int32, device=DEV)
        ctx.select(sc, lens, n, B, idx, cnt)
        torch.cuda.synchronize()
        assert cnt.tolist() == [min(B, n)] * U
        for u in range(U):
            want = oracle.select(x[u].double().numpy(), B)
            assert np.array_equal(idx[u].cpu().numpy(), want), (U, n, B, levels, u)
    # scores far outside the histogram's [-8, 8) range all land in its end bins; the result stays exact
    x = torch.randn(2, 20000, generator=g) * 1000.0
    ctx = tb.TriContext(2, 1, 1, torch.zeros(2, 1, 128), torch.zeros(2, 1, 64))
    idx = torch.full((2, 5000), -1, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int32, device=DEV)
    ctx.select(x.to(DEV), torch.tensor([20000], dtype=torch.int32, device=DEV), 20000, 5000, idx, cnt)
    for u in range(2):
        assert np.array_equal(idx[u].cpu().numpy(), oracle.select(x[u].double().numpy(), 5000))
    # negative values, -0.0 vs +0.0 and infinities keep the float order
    x = torch.tensor([[0.0, -0.0, -1.0, float("inf"), 1e-40, -1e-40, 3.0, float("-inf")]])
    ctx = tb.TriContext(1, 1, 1, torch.zeros(1, 1, 128), torch.zeros(1, 1, 64))
    idx = torch.full((1, 3), -1, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    ctx.select(x.to(DEV), torch.tensor([8], dtype=torch.int32, device=DEV), 8, 3, idx, cnt)
    assert sorted(idx[0].tolist()) == [3, 4, 6]


def test_compact_standalone_and_rerun_determinism():
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="det", n_layers=2, n_kv_heads=2, n_keys=4000, budget=256)
    w = W.make_workload(sp, DEV)
    a = run_compress(w, sp.budget)
    b = run_compress(w, sp.budget)
    for key in ("scores", "raw", "kept_idx", "kept_cnt"):
        assert torch.equal(a[key], b[key]), key
    assert torch.equal(a["k_out"].view(torch.int16), b["k_out"].view(torch.int16))
    # tri_compact on its own from the kept indices reproduces the fused call's rows
    ctx = a["ctx"]
    k2, v2 = torch.zeros_like(a["k_out"]), torch.zeros_like(a["v_out"])
    p2 = torch.zeros_like(a["pos_out"])
    lens = torch.zeros(1, dtype=torch.int32, device=DEV)
    ctx.compact(src_view(w), a["kept_idx"], a["kept_cnt"], 1, sp.budget, tb.CacheView(k2, v2, positions=p2), lens)
    torch.cuda.synchronize()
    assert torch.equal(k2.view(torch.int16), a["k_out"].view(torch.int16))
    assert torch.equal(v2.view(torch.int16), a["v_out"].view(torch.int16))
    assert torch.equal(p2, a["pos_out"]) and lens.tolist() == [sp.budget]


@pytest.mark.parametrize("pinned,budget,G", [(True, 700, 4), (False, 700, 4), (True, 2048, 4), (True, 700, 8)])
def test_host_resident_cache_round(pinned, budget, G):
    """tri_compress_host: K/V/positions in host memory in, compacted rows in host memory out; with pinned
    arrays and at most half of the rows kept, V and positions are never copied in bulk (the gather reads the
    kept rows from host memory)."""
    sp = W.SPECS["qwen3_8b_steady_b64"].scaled(name="hostpath", n_layers=2, n_kv_heads=2, n_seqs=3, budget=budget, group_size=G)
    w = W.make_workload(sp, DEV)
    ref = run_compress(w, sp.budget, want_scores=False)
    L, S, H, B, N = 2, 3, 2, sp.budget, sp.n_keys
    host = lambda t: (t.cpu().pin_memory() if pinned else t.cpu())
    hk, hv, hpos = host(w.k), host(w.v), host(w.positions)
    hlens, hcur = host(w.seq_lens), host(w.cur_pos)
    hk2 = host(torch.zeros(L, S, H, B, 128, dtype=torch.bfloat16)); hv2 = host(torch.zeros_like(hk2))
    hp2 = host(torch.zeros(L, S, H, B, dtype=torch.int32)); hcnt = host(torch.zeros(L * S * H, dtype=torch.int32))
    dk = torch.empty_like(w.k); dv = torch.full_like(w.v, float("nan")); dpos = torch.full_like(w.positions, -7)
    dlens, dcur = torch.empty_like(w.seq_lens), torch.empty_like(w.cur_pos)
    k2 = torch.empty(L, S, H, B, 128, dtype=torch.bfloat16, device=DEV); v2 = torch.empty_like(k2)
    p2 = torch.empty(L, S, H, B, dtype=torch.int32, device=DEV); cnt = torch.empty(L * S * H, dtype=torch.int32, device=DEV)
    ctx = ref["ctx"]
    ws = ctx.workspace(S, N, B)
    ctx.compress_host(tb.CacheView(hk, hv, seq_lens=hlens, positions=hpos), tb.CacheView(dk, dv, seq_lens=dlens, positions=dpos),
                      hcur, dcur, B, tb.CacheView(hk2, hv2, positions=hp2), tb.CacheView(k2, v2, positions=p2), hcnt, cnt, ws)
    torch.cuda.synchronize()
    assert torch.equal(hcnt, ref["kept_cnt"].cpu())
    assert torch.equal(hk2.view(torch.int16), ref["k_out"].cpu().view(torch.int16))
    assert torch.equal(hv2.view(torch.int16), ref["v_out"].cpu().view(torch.int16))
    assert torch.equal(hp2, ref["pos_out"].cpu())
    if pinned and 2 * B <= N:      # the staging copies of V and positions were never written
        assert bool(torch.isnan(dv.float()).all()) and bool((dpos == -7).all())


@pytest.mark.parametrize("kind", ["oneshot", "paged_in_place"])
def test_pipelined_round_is_bit_identical(kind):
    """tri_set_pipeline: the round issued over 1, 2, 5 and 16 unit ranges (selection and compaction on the context's
    side stream under the scoring of the next range) gives the same bits as the single-stream round, and the
    caller's stream sees the finished round."""
    if kind == "oneshot":
        sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="pipe", n_layers=3, n_kv_heads=3, n_keys=4000, budget=300)
    else:
        sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="pipe_p", n_layers=3, n_kv_heads=2, n_seqs=3, n_keys=3000,
                                                      n_keys_min=200, budget=512)
    w = W.make_workload(sp, DEV)
    k0, v0 = w.k.clone(), w.v.clone()
    u = (2, sp.n_seqs - 1, 1)
    oref = oracle_unit(w, *u, sp.budget)                     # before any in-place write
    ctx = make_ctx(w)
    ref = None
    for ranges in (1, 2, 5, 16, 0):
        w.k.copy_(k0); w.v.copy_(v0)
        ctx.set_pipeline(ranges)
        res = run_compress(w, sp.budget, ctx=ctx, in_place=(kind != "oneshot"), want_scores=False)
        assert int(res["status"].item()) == 0
        check_unit(w, res, oref, *u, sp.budget)
        got = dict(idx=res["kept_idx"].clone(), cnt=res["kept_cnt"].clone(), lens=res["new_seq_lens"].clone(),
                   k=res["k_out"].clone().view(torch.int16), v=res["v_out"].clone().view(torch.int16))
        if ref is None:
            ref = got
        for key in ref:
            assert torch.equal(ref[key], got[key]), (ranges, key)


@pytest.mark.parametrize("G", [4, 8])
def test_round_replays_from_a_cuda_graph(G):
    """tri_compress only enqueues kernels on the given stream (no allocation, no synchronisation), so a decode
    loop can capture one round in a CUDA graph and replay it; the replay reads cur_pos from device memory."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="graph", n_layers=2, n_kv_heads=2, n_keys=6000, budget=500, group_size=G)
    w = W.make_workload(sp, DEV)
    direct = run_compress(w, sp.budget, want_scores=False)           # also the first call: one-time kernel set-up
    ctx = direct["ctx"]
    src = src_view(w)
    U = 4
    k2, v2 = torch.zeros_like(direct["k_out"]), torch.zeros_like(direct["v_out"])
    p2 = torch.zeros_like(direct["pos_out"])
    idx = torch.zeros(U, sp.budget, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(U, dtype=torch.int32, device=DEV)
    ws = ctx.workspace(1, sp.n_keys, sp.budget)
    cur = w.cur_pos.clone()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.compress(src, cur, sp.budget, tb.CacheView(k2, v2, positions=p2), ws, kept_idx=idx, kept_cnt=cnt)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(idx, direct["kept_idx"]) and torch.equal(cnt, direct["kept_cnt"])
    assert torch.equal(k2.view(torch.int16), direct["k_out"].view(torch.int16)) and torch.equal(p2, direct["pos_out"])
    # a later query position, written into the captured buffer, changes the scores of the replay
    cur += 4096
    w.cur_pos = cur.clone()
    later = run_compress(w, sp.budget, ctx=ctx, want_scores=False)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(idx, later["kept_idx"]) and not torch.equal(idx, direct["kept_idx"])
    assert torch.equal(v2.view(torch.int16), later["v_out"].view(torch.int16))


def test_windowed_round_in_a_decode_loop_from_a_graph():
    """tri_compress_windowed captured once and replayed after every decoded token (Section 4.3's trigger on the device):
    nothing moves until a sequence's window counter reaches beta with its cache above the budget; then that sequence
    alone is compressed in place.  Two sequences out of phase (one starts at the budget, one far below it), 40 steps,
    against a host model that applies the oracle at the same moments."""
    B, beta, steps, S, H = 64, 8, 40, 2, 2
    cap = B + beta
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="win", n_layers=1, n_kv_heads=H, n_seqs=S, n_keys=B + steps, budget=B)
    full = W.make_workload(sp, DEV)                     # every token either sequence will ever hold: slot i = position i
    G = sp.group_size
    start = [B, 30]
    k = torch.zeros(1, S, H, cap, 128, dtype=torch.bfloat16, device=DEV); v = torch.zeros_like(k)
    pos = torch.zeros(1, S, H, cap, dtype=torch.int32, device=DEV)
    lens = torch.tensor(start, dtype=torch.int32, device=DEV)
    cur = torch.tensor(start, dtype=torch.int64, device=DEV)
    decoded = torch.zeros(S, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(S * H, dtype=torch.int32, device=DEV)
    host = {}
    for s_ in range(S):
        n0 = start[s_]
        k[0, s_, :, :n0], v[0, s_, :, :n0] = full.k[0, s_, :, :n0], full.v[0, s_, :, :n0]
        pos[0, s_, :, :n0] = torch.arange(n0, dtype=torch.int32, device=DEV)
        for h in range(H):
            host[(s_, h)] = dict(k=full.k[0, s_, h, :n0].cpu(), v=full.v[0, s_, h, :n0].cpu(), pos=torch.arange(n0))
    ctx = make_ctx(full)
    ws = ctx.workspace(S, cap, B)
    view = tb.CacheView(k, v, seq_lens=lens, positions=pos)
    ctx.compress_windowed(view, cur, B, decoded, 0, beta, view, ws, kept_cnt=cnt, new_seq_lens=lens)   # set-up call, nothing due
    torch.cuda.synchronize()
    assert lens.tolist() == start and decoded.tolist() == [0, 0]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.compress_windowed(view, cur, B, decoded, 1, beta, view, ws, kept_cnt=cnt, new_seq_lens=lens)
    h_len, h_dec, rounds = list(start), [0, 0], 0
    for step in range(steps):
        for s_ in range(S):                            # the model appends one token per sequence
            t = start[s_] + step
            n = h_len[s_]
            k[0, s_, :, n], v[0, s_, :, n] = full.k[0, s_, :, t], full.v[0, s_, :, t]
            pos[0, s_, :, n] = t
            for h in range(H):
                st = host[(s_, h)]
                host[(s_, h)] = dict(k=torch.cat([st["k"], full.k[0, s_, h, t:t + 1].cpu()]),
                                     v=torch.cat([st["v"], full.v[0, s_, h, t:t + 1].cpu()]), pos=torch.cat([st["pos"], torch.tensor([t])]))
            h_len[s_] += 1
        lens.copy_(torch.tensor(h_len, dtype=torch.int32))
        cur.copy_(torch.tensor([start[s_] + step + 1 for s_ in range(S)], dtype=torch.int64))
        graph.replay()
        torch.cuda.synchronize()
        for s_ in range(S):
            h_dec[s_] += 1
            due = False
            if h_dec[s_] >= beta:
                h_dec[s_] = 0
                due = h_len[s_] > B
            for h in range(H):
                st = host[(s_, h)]
                if due:
                    _, s_o, idx_o = oracle.unit_bf16(W.bf16_bits(st["k"]), st["pos"].numpy(), start[s_] + step + 1,
                                                     full.q_center[0, h * G:(h + 1) * G].double().numpy(),
                                                     full.q_mean_norm[0, h * G:(h + 1) * G].double().numpy(), B, theta=sp.theta)
                    got_pos = pos[0, s_, h, :B].cpu().long()
                    want_pos = st["pos"][torch.from_numpy(idx_o.astype(np.int64))]
                    if not torch.equal(got_pos, want_pos):
                        diff = np.setxor1d(got_pos.numpy(), want_pos.numpy())
                        s_b = np.sort(s_o)[::-1][B - 1]
                        assert np.all(np.abs(s_o[np.isin(st["pos"].numpy(), diff)] - s_b) <= 1e-3 * max(1.0, abs(s_b)))
                    sel = torch.from_numpy(np.searchsorted(st["pos"].numpy(), got_pos.numpy()))
                    assert torch.equal(st["pos"][sel], got_pos)
                    host[(s_, h)] = dict(k=st["k"][sel], v=st["v"][sel], pos=got_pos)
                    assert int(cnt[s_ * H + h]) == B
                    rounds += 1
                else:
                    assert int(cnt[s_ * H + h]) == 0
                st = host[(s_, h)]
                n = st["pos"].shape[0]
                assert torch.equal(pos[0, s_, h, :n].cpu().long(), st["pos"])
                assert torch.equal(k[0, s_, h, :n].cpu().view(torch.int16), st["k"].view(torch.int16))
                assert torch.equal(v[0, s_, h, :n].cpu().view(torch.int16), st["v"].view(torch.int16))
            if due:
                h_len[s_] = B
        assert lens.tolist() == h_len and decoded.tolist() == h_dec, step
    assert rounds >= 2 * H * 3                         # both sequences were compressed several times


def test_bad_page_id_sets_status_not_fault():
    """A page id outside the pool is reported through device_status; its rows are skipped."""
    sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="badpage", n_layers=1, n_kv_heads=1, n_seqs=2, n_keys=400,
                                                  n_keys_min=200, budget=64)
    w = W.make_workload(sp, DEV)
    w.page_table[0, 3] = 10 ** 6
    res = run_compress(w, sp.budget, want_scores=False)
    assert int(res["status"].item()) == 5


@pytest.mark.parametrize("fp32_keys", [True, False])
def test_out_of_range_kept_index_is_skipped_in_place(fp32_keys):
    """tri_compact in place with a kept index beyond the unit's capacity: that row is left as it was (not
    overwritten, not dereferenced); every other row moves.  fp32 keys without a value cache take the staged
    in-place kernel, bf16 K + V the tiled one."""
    n, cnt = 96, 40
    g = torch.Generator().manual_seed(11)
    k = torch.randn(1, 1, 1, n, 128, generator=g).to(DEV)
    if not fp32_keys:
        k = k.to(torch.bfloat16)
    v = None if fp32_keys else torch.randn(1, 1, 1, n, 128, generator=g).to(DEV).to(torch.bfloat16)
    pos = torch.arange(100, 100 + n, dtype=torch.int32, device=DEV).view(1, 1, 1, n)
    k0, pos0 = k.clone(), pos.clone()
    idx = torch.arange(cnt, dtype=torch.int32) * 2 + 1           # 1, 3, 5, ...: ascending, idx[j] > j
    idx[-1] = 10 ** 6
    idx_d = idx.view(1, cnt).to(DEV)
    cnt_d = torch.tensor([cnt], dtype=torch.int32, device=DEV)
    ctx = tb.TriContext(1, 1, 1, torch.zeros(1, 1, 128), torch.zeros(1, 1, 64))
    view = tb.CacheView(k, v, positions=pos)
    ctx.compact(view, idx_d, cnt_d, 1, cnt, view)
    torch.cuda.synchronize()
    good = idx[:-1].long().to(DEV)
    assert torch.equal(k[0, 0, 0, :cnt - 1], k0[0, 0, 0][good])
    assert torch.equal(pos[0, 0, 0, :cnt - 1], pos0[0, 0, 0][good])
    assert torch.equal(k[0, 0, 0, cnt - 1:], k0[0, 0, 0, cnt - 1:])          # the bad row and everything behind it
    assert torch.equal(pos[0, 0, 0, cnt - 1:], pos0[0, 0, 0, cnt - 1:])


def test_bounded_wait_runs_out_and_reports():
    """The wait the scoring kernel uses for its copy barriers gives up after its poll limit: a barrier that
    nothing completes yields status 6 (TRI_ERR_TIMEOUT), the kernel returns, and the device keeps working."""
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert tb.lib().tri_selftest_bounded_wait(status.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 6
    w = W.make_workload(W.SPECS["tiny"].scaled(name="afterwait", n_keys=500, budget=50), DEV)
    res = run_compress(w, 50)
    check_unit(w, res, oracle_unit(w, 0, 0, 0, 50), 0, 0, 0, 50)


def test_host_errors_launch_nothing():
    w = W.make_workload(W.SPECS["tiny"].scaled(n_keys=256, budget=32), DEV)
    ctx = make_ctx(w)
    src = src_view(w)
    ws = ctx.workspace(1, 256, 32)
    dst = tb.CacheView(torch.zeros(1, 1, 1, 32, 128, dtype=torch.bfloat16, device=DEV), None)
    with pytest.raises(tb.TriError) as e:
        ctx.compress(src, w.cur_pos, 32, dst, ws[:1024])
    assert e.value.code == 3
    with pytest.raises(tb.TriError) as e:
        ctx.compress(src, w.cur_pos, 0, dst, ws)
    assert e.value.code == 1
    small = tb.CacheView(torch.zeros(1, 1, 1, 8, 128, dtype=torch.bfloat16, device=DEV), None)
    with pytest.raises(tb.TriError) as e:
        ctx.compress(src, w.cur_pos, 32, small, ws)
    assert e.value.code == 1
    torch.cuda.synchronize()


def _sample(units, L, S, H, extra=()):
    """Eight or more (layer, sequence, head) picks: first and last unit, the extras, then a fixed stride through the rest."""
    out = [(0, 0, 0), (L - 1, S - 1, H - 1)] + list(extra)
    i = 1
    while len(out) < units:
        u = (i * 7919) % (L * S * H)
        pick = (u // (S * H), (u // H) % S, u % H)
        if pick not in out:
            out.append(pick)
        i += 1
    return out


def test_full_size_config1_sampled_units():
    """The benchmark's own workload and launch configuration (36 x 8 units of 32,768 keys, B = 2,048): whole-job
    invariants plus raw scores, final scores, kept set and copied rows of eight sampled units against the oracle."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"]
    w = W.make_workload(sp, DEV)
    res = run_compress(w, sp.budget)
    assert int(res["status"].item()) == 0
    assert torch.all(res["kept_cnt"] == sp.budget)
    idx = res["kept_idx"]
    assert torch.all(idx[:, 1:] > idx[:, :-1]) and int(idx.min()) >= 0 and int(idx.max()) < sp.n_keys
    # every compacted row is a bit copy of the row its index names
    L, H = sp.n_layers, sp.n_kv_heads
    gi = idx.view(L, 1, H, sp.budget, 1).long().expand(L, 1, H, sp.budget, 128)
    assert torch.equal(torch.gather(w.k, 3, gi).view(torch.int16), res["k_out"].view(torch.int16))
    assert torch.equal(torch.gather(w.v, 3, gi).view(torch.int16), res["v_out"].view(torch.int16))
    assert torch.equal(res["pos_out"].view(-1, sp.budget), idx)
    for (l, s_, h) in _sample(8, L, 1, H):
        ref = oracle_unit(w, l, s_, h, sp.budget)
        st = check_unit(w, res, ref, l, s_, h, sp.budget)
        assert "raw_err" in st


def _whole_job_invariants(w, res, budget):
    """Properties that hold at any size: counts, strictly ascending in-range indices."""
    sp = w.spec
    assert int(res["status"].item()) == 0
    lens = w.seq_lens.repeat_interleave(sp.n_kv_heads).repeat(w.k.shape[0])
    want = torch.clamp(lens, max=budget)
    assert torch.equal(res["kept_cnt"], want)
    idx = res["kept_idx"]
    col = torch.arange(budget, device=idx.device)[None, :]
    valid = col < want[:, None]
    assert torch.all((idx >= 0) | ~valid) and torch.all((idx < lens[:, None]) | ~valid)
    assert torch.all((idx[:, 1:] > idx[:, :-1]) | ~valid[:, 1:])


def test_full_size_config2_sampled_units():
    """The steady-state batch at full size (36 x 64 x 8 units of 2,176 keys at scattered positions): scores, kept
    set and rows of ten sampled units."""
    sp = W.SPECS["qwen3_8b_steady_b64"]
    w = W.make_workload(sp, DEV)
    res = run_compress(w, sp.budget)
    _whole_job_invariants(w, res, sp.budget)
    assert res["new_seq_lens"].tolist() == [sp.budget] * sp.n_seqs
    for (l, s_, h) in _sample(10, sp.n_layers, sp.n_seqs, sp.n_kv_heads, extra=[(17, 33, 5)]):
        st = check_unit(w, res, oracle_unit(w, l, s_, h, sp.budget), l, s_, h, sp.budget)
        assert "raw_err" in st


def test_full_size_config3_sampled_units():
    """The 131,072-token sequence at full size (36 x 8 units), mixed per-head noise: eight units including the most
    concentrated and the most diffuse head (the two ends of Section 3.1's spectrum)."""
    sp = W.SPECS["qwen3_8b_long_128k"]
    w = W.make_workload(sp, DEV)
    res = run_compress(w, sp.budget)
    _whole_job_invariants(w, res, sp.budget)
    noise = W._head_noise(sp, "cpu")
    lo, hi = int(noise.argmin()), int(noise.argmax())
    extra = [(lo // sp.n_kv_heads, 0, lo % sp.n_kv_heads), (hi // sp.n_kv_heads, 0, hi % sp.n_kv_heads)]
    assert float(noise.flatten()[lo]) < 0.25 and float(noise.flatten()[hi]) > 0.95
    for (l, s_, h) in _sample(8, sp.n_layers, 1, sp.n_kv_heads, extra=extra):
        st = check_unit(w, res, oracle_unit(w, l, 0, h, sp.budget), l, 0, h, sp.budget)
        assert "raw_err" in st


def test_full_size_config4_slab_sampled_units():
    """The ragged paged batch at full size per layer (16 sequences of 8K-64K keys, G = 8), a slab of 4 of
    its 64 layers as the benchmark runs it, compacted in place into the sequences' own pages: eight units including
    the shortest and the longest sequence."""
    sp = W.SPECS["qwen3_32b_ragged_paged"]
    w = W.make_workload(sp, DEV, layer0=0, n_layers=4)
    lens = w.seq_lens.tolist()
    picks = _sample(8, 4, sp.n_seqs, sp.n_kv_heads, extra=[(0, lens.index(min(lens)), 0), (3, lens.index(max(lens)), 7)])
    refs = {u: oracle_unit(w, *u, sp.budget) for u in picks}      # before the in-place write
    res = run_compress(w, sp.budget, in_place=True)
    _whole_job_invariants(w, res, sp.budget)
    assert res["new_seq_lens"].tolist() == [min(n, sp.budget) for n in lens]
    for u, ref in refs.items():
        st = check_unit(w, res, ref, *u, sp.budget)
        assert "raw_err" in st


@pytest.mark.parametrize("G,ties", [(4, False), (8, False), (3, False), (4, True)])
def test_fused_selection_of_long_units_equals_the_two_step_path(G, ties):
    """Units of at least 65,536 keys that keep at most an eighth take the one-sweep selection inside the fused round
    (sampled lower bound of the threshold, listed keys, exact selection on the list, bitmap emit).  Its kept slots
    must be the very ones tri_select finds in the final scores tri_score writes (the general three-sweep path, itself
    bit-exact against the oracle), and the oracle's.  With ties = True every key row is a copy of one of 40 rows, so
    a unit's scores take 40 values: the threshold falls inside a group of ~1,750 equal scores, the lowest slots of
    the group must win, and the group's value bin overflows the in-kernel list, which sends the unit down the
    general path from inside the one-sweep one."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name=f"long{G}{int(ties)}", n_layers=1, n_kv_heads=2, n_keys=70001, budget=1500,
                                                group_size=G)
    w = W.make_workload(sp, DEV)
    if ties:
        pick = torch.randint(0, 40, (sp.n_keys,), generator=torch.Generator().manual_seed(11)).to(DEV)
        w.k.copy_(w.k[..., pick, :].clone())
    res = run_compress(w, sp.budget)                       # fused round, then tri_score for the scores
    assert int(res["status"].item()) == 0
    ctx = res["ctx"]
    U = 2
    idx2 = torch.full((U, sp.budget), -1, dtype=torch.int32, device=DEV)
    cnt2 = torch.zeros(U, dtype=torch.int32, device=DEV)
    ctx.select(res["scores"], w.seq_lens, sp.n_keys, sp.budget, idx2, cnt2)
    torch.cuda.synchronize()
    assert torch.equal(cnt2, res["kept_cnt"].view(-1)) and torch.equal(idx2, res["kept_idx"].view(U, -1))
    if ties:
        sc = res["scores"].view(U, -1)
        assert all(len(torch.unique(sc[u])) <= 40 for u in range(U))
        kept = torch.gather(sc[0], 0, idx2[0].long())
        t = kept.min()                                   # the threshold: some keys equal to it are kept, some are not
        assert int((sc[0] == t).sum()) > int((kept == t).sum()) > 0
        eq = torch.nonzero(sc[0] == t).view(-1)
        assert torch.equal(idx2[0][kept == t].long(), eq[: int((kept == t).sum())])     # the lowest slots of the group
    else:
        check_unit(w, res, oracle_unit(w, 0, 0, 1, sp.budget), 0, 0, 1, sp.budget)


def _as_e4m3(w):
    """The same workload with K and V rounded to e4m3 (k_kind 3)."""
    return W.Workload(w.spec, w.q_center, w.q_mean_norm, w.k.float().to(torch.float8_e4m3fn), w.v.float().to(torch.float8_e4m3fn),
                      w.seq_lens, w.cur_pos, w.positions, w.page_table)


@pytest.mark.parametrize("shape", ["g4", "g8_paged_in_place", "g16", "g3_half_split", "g1_long"])
def test_e4m3_keys(shape):
    """8-bit caches (k_kind 3): raw and final scores, kept slots and the copied 128-byte K and V rows of every unit
    against the oracle's reading of the same bytes: 16-key tiles with a ragged tail, one, two and four MMA column
    tiles (G = 1..16), both band layouts, paged keys compacted in place, and a unit long enough for the one-sweep
    selection."""
    base = W.SPECS["qwen3_8b_oneshot_32k"]
    layout, in_place = 0, False
    if shape == "g4":
        sp = base.scaled(name="e4_g4", n_layers=2, n_kv_heads=2, n_keys=5003, budget=400)
    elif shape == "g8_paged_in_place":
        sp = W.SPECS["qwen3_32b_ragged_paged"].scaled(name="e4_g8", n_layers=2, n_kv_heads=2, n_seqs=3, n_keys=4000,
                                                      n_keys_min=300, budget=512)
        in_place = True
    elif shape == "g16":
        sp = base.scaled(name="e4_g16", n_layers=1, n_kv_heads=1, group_size=16, n_keys=3000, budget=300)
    elif shape == "g3_half_split":
        sp = base.scaled(name="e4_g3", n_layers=1, n_kv_heads=2, group_size=3, n_keys=3333, budget=200)
        layout = 1
    else:
        sp = base.scaled(name="e4_g1", n_layers=1, n_kv_heads=1, group_size=1, n_keys=70001, budget=1000)
    w = W.make_workload(sp, DEV)
    if layout == 1:
        perm = torch.cat([torch.arange(0, 128, 2), torch.arange(1, 128, 2)])
        w = W.Workload(sp, w.q_center[..., perm].contiguous(), w.q_mean_norm, w.k[..., perm.to(DEV)].contiguous(),
                       w.v, w.seq_lens, w.cur_pos, None, None)
    w = _as_e4m3(w)
    units = _all_units(w)
    refs = {u: oracle_unit(w, *u, sp.budget, layout=layout) for u in units}      # before any in-place write
    ctx = make_ctx(w, pair_layout=layout)
    res = run_compress(w, sp.budget, ctx=ctx, in_place=in_place)
    assert int(res["status"].item()) == 0
    for u in units:
        check_unit(w, res, refs[u], *u, sp.budget)
