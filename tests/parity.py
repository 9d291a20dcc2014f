"""Shared helpers of the GPU parity tests: run the CUDA library on a workload, run the CPU oracle on
chosen units of the same arrays, and compare under the stated tolerances.

Tolerances (from the benchmark spec of the bar):
  * raw per-head scores within 1e-3 relative error, |gpu - oracle| <= 1e-3 * max(|oracle|, sigma_g)
    (sigma_g, the spread of that head's scores, stands in when a score is near zero);
  * final scores |gpu - oracle| <= 1e-3 * max(|oracle|, 1)  (z-scores have unit spread);
  * kept set identical except for keys whose oracle score lies within 1e-3 * max(1, |S_B|) of the
    B-th largest oracle score S_B;
  * indices ascending, count exact, compacted K / V / positions bit-exact given the kept set.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2604_04921_b200 import binding as tb
from paper_2604_04921_b200 import workloads as W

REL = 1e-3


def make_ctx(w: W.Workload, **kw) -> tb.TriContext:
    sp = w.spec
    return tb.TriContext(w.k.shape[0], sp.n_kv_heads, sp.group_size, w.q_center, w.q_mean_norm,
                         rope_theta=sp.theta, **kw)


def src_view(w: W.Workload) -> tb.CacheView:
    return tb.CacheView(w.k, w.v, seq_lens=w.seq_lens, positions=w.positions, page_table=w.page_table)


def unit_index(w: W.Workload, l: int, s: int, h: int) -> int:
    return (l * w.spec.n_seqs + s) * w.spec.n_kv_heads + h


def oracle_unit(w: W.Workload, l: int, s: int, h: int, budget: int, offsets=oracle.DEFAULT_OFFSETS,
                layout: int = 0, norm_variant: int = 0):
    kk, vv, pos = w.unit_rows(l, s, h)
    G = w.spec.group_size
    qc = w.q_center[l, h * G:(h + 1) * G].double().numpy()
    qn = w.q_mean_norm[l, h * G:(h + 1) * G].double().numpy()
    if kk.dtype == torch.float8_e4m3fn:
        raw, sfin, idx = oracle.unit_e4m3(kk.contiguous().view(torch.uint8).numpy(), pos.numpy(), int(w.cur_pos[s].item()), qc, qn,
                                          budget, offsets=offsets, theta=w.spec.theta, layout=layout, norm_variant=norm_variant)
    else:
        raw, sfin, idx = oracle.unit_bf16(W.bf16_bits(kk), pos.numpy(), int(w.cur_pos[s].item()), qc, qn, budget,
                                          offsets=offsets, theta=w.spec.theta, layout=layout,
                                          norm_variant=norm_variant)
    return dict(raw=raw, s_final=sfin, idx=idx, k=kk, v=vv, pos=pos)


def check_scores(raw_gpu: np.ndarray, s_gpu: np.ndarray, ref: dict):
    """raw_gpu [N, G], s_gpu [N] against the oracle's raw [G, N], s_final [N]."""
    raw_o = ref["raw"]
    sig = raw_o.std(axis=1)
    tol = REL * np.maximum(np.abs(raw_o), sig[:, None])
    err = np.abs(raw_gpu.T.astype(np.float64) - raw_o)
    assert np.all(err <= tol), f"raw score error {np.max(err / np.maximum(tol, 1e-300)):.3g} x tolerance"
    s_o = ref["s_final"]
    tol_s = REL * np.maximum(np.abs(s_o), 1.0)
    err_s = np.abs(s_gpu.astype(np.float64) - s_o)
    assert np.all(err_s <= tol_s), f"final score error {np.max(err_s / tol_s):.3g} x tolerance"
    return float(np.max(err / np.maximum(tol, 1e-300))), float(np.max(err_s / tol_s))


def check_kept(idx_gpu: np.ndarray, cnt_gpu: int, ref: dict, budget: int):
    s_o, idx_o = ref["s_final"], ref["idx"]
    n = s_o.shape[0]
    assert cnt_gpu == min(budget, n) == idx_o.size
    idx_gpu = idx_gpu[:cnt_gpu]
    assert np.all(np.diff(idx_gpu) > 0), "kept indices not strictly ascending"
    assert idx_gpu.size == 0 or (idx_gpu[0] >= 0 and idx_gpu[-1] < n)
    diff = np.setxor1d(idx_gpu, idx_o)
    if diff.size:
        s_b = np.sort(s_o)[::-1][budget - 1]
        band = REL * max(1.0, abs(s_b))
        off = np.abs(s_o[diff] - s_b)
        assert np.all(off <= band), f"kept sets differ outside the tie band: {diff[off > band][:8]}"
    return int(diff.size)


def check_compacted(k_out, v_out, pos_out, idx_gpu: np.ndarray, ref: dict):
    """Rows [0, cnt) of the destination must be bit copies of the source rows at idx_gpu."""
    cnt = idx_gpu.size
    sel = torch.from_numpy(idx_gpu.astype(np.int64))
    bits = torch.uint8 if ref["k"].dtype == torch.float8_e4m3fn else torch.int16
    assert torch.equal(k_out[:cnt].cpu().view(bits), ref["k"].view(bits)[sel])
    if v_out is not None:
        assert torch.equal(v_out[:cnt].cpu().view(bits), ref["v"].view(bits)[sel])
    if pos_out is not None:
        assert torch.equal(pos_out[:cnt].cpu().long(), ref["pos"][sel])
        assert torch.all(pos_out[1:cnt] > pos_out[:cnt - 1])


def run_compress(w: W.Workload, budget: int, ctx: tb.TriContext = None, in_place: bool = False,
                 want_scores: bool = True, unit_budgets=None):
    """tri_score (+raw) and tri_compress on the whole workload.  Returns a dict of device tensors."""
    sp = w.spec
    own = ctx is None
    ctx = ctx or make_ctx(w)
    dev = w.k.device
    L, S, H, G = w.k.shape[0], sp.n_seqs, sp.n_kv_heads, sp.group_size
    src = src_view(w)
    n_max = src.c_view().n_max
    U = L * S * H
    ws = ctx.workspace(S, n_max, budget, dev)
    out = {}
    if want_scores:
        out["scores"] = torch.full((U, n_max), float("nan"), dtype=torch.float32, device=dev)
        out["raw"] = torch.full((U, n_max, G), float("nan"), dtype=torch.float32, device=dev)
        ctx.score(src, w.cur_pos, out["scores"], ws, raw=out["raw"])
    kept_idx = torch.full((U, budget), -1, dtype=torch.int32, device=dev)
    kept_cnt = torch.full((U,), -1, dtype=torch.int32, device=dev)
    new_lens = torch.full((S,), -1, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if in_place:
        dst = tb.CacheView(w.k, w.v, positions=w.positions, page_table=w.page_table, n_max=n_max)
        out["k_out"], out["v_out"], out["pos_out"] = w.k, w.v, w.positions
    elif w.paged:
        k2, v2 = torch.zeros_like(w.k), torch.zeros_like(w.v)
        dst = tb.CacheView(k2, v2, page_table=w.page_table, n_max=n_max)
        out["k_out"], out["v_out"], out["pos_out"] = k2, v2, None
    else:
        k2 = torch.zeros(L, S, H, budget, 128, dtype=w.k.dtype, device=dev)
        v2 = torch.zeros_like(k2)
        p2 = torch.full((L, S, H, budget), -1, dtype=torch.int32, device=dev)
        dst = tb.CacheView(k2, v2, positions=p2)
        out["k_out"], out["v_out"], out["pos_out"] = k2, v2, p2
    ctx.compress(src, w.cur_pos, budget, dst, ws, kept_idx=kept_idx, kept_cnt=kept_cnt, new_seq_lens=new_lens,
                 device_status=status, unit_budgets=unit_budgets)
    torch.cuda.synchronize()
    out.update(kept_idx=kept_idx, kept_cnt=kept_cnt, new_seq_lens=new_lens, status=status, ctx=ctx)
    if own:
        out["_own_ctx"] = ctx
    return out


def out_rows(w: W.Workload, res: dict, l: int, s: int, h: int, cnt: int):
    """Destination rows of one unit (K, V, positions) as host tensors."""
    if w.paged:
        ps = w.spec.page_size
        npg = (cnt + ps - 1) // ps
        pages = w.page_table[s, :npg].long()
        k = res["k_out"][l, pages, h].reshape(npg * ps, 128)[:cnt]
        v = res["v_out"][l, pages, h].reshape(npg * ps, 128)[:cnt]
        return k, v, None
    k = res["k_out"][l, s, h, :cnt]
    v = res["v_out"][l, s, h, :cnt]
    p = res["pos_out"][l, s, h, :cnt].cpu() if res["pos_out"] is not None else None
    return k, v, p


def check_unit(w: W.Workload, res: dict, ref: dict, l: int, s: int, h: int, budget: int):
    u = unit_index(w, l, s, h)
    n = ref["s_final"].shape[0]
    stats = {}
    if "raw" in res:
        raw_gpu = res["raw"][u, :n].cpu().numpy()
        s_gpu = res["scores"][u, :n].cpu().numpy()
        stats["raw_err"], stats["final_err"] = check_scores(raw_gpu, s_gpu, ref)
    cnt = int(res["kept_cnt"][u].item())
    idx_gpu = res["kept_idx"][u].cpu().numpy()
    stats["swaps"] = check_kept(idx_gpu, cnt, ref, budget)
    k, v, p = out_rows(w, res, l, s, h, cnt)
    check_compacted(k, v, p, idx_gpu[:cnt], ref)
    return stats
