"""Seeded synthetic inputs for the KV-compression round.

This module only *makes inputs*: model-shaped caches as a decoder would have left them
(pre-RoPE keys drawn around a per-head centre, rotated forward by RoPE, rounded to bf16),
calibration statistics as sample means over seeded query draws, positions, page tables.
It holds none of the compression method's arithmetic (no scoring, no inverse rotation, no
selection, no gather) and imports neither the CUDA binding nor the CPU oracle; both sides
consume the arrays it returns.

The five named workloads mirror the benchmark configurations (shapes of Qwen3-8B /
Qwen3-32B attention: head_dim 128, RoPE theta 1e6, GQA 4 or 8).  They stand in for the
paper's decoding traces (Section 5 measures on reasoning benchmarks with trained weights,
neither of which is available offline); the centre+noise model follows Observation 3.1
(pre-RoPE Q/K concentrated around non-zero centres).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

MASTER_SEED = 20260404
HEAD_DIM = 128
N_CALIB = 1024  # seeded query draws per query head behind E[q_f] and E|q_f|


@dataclasses.dataclass(frozen=True)
class Spec:
    """Shape of one workload.  Sizes follow the benchmark configurations."""
    name: str
    n_layers: int
    n_kv_heads: int
    group_size: int           # G query heads per KV head
    n_seqs: int               # S
    n_keys: int               # cached keys per head (max over sequences when ragged)
    budget: int               # B
    kind: str                 # "oneshot" | "steady" | "ragged_paged"
    noise_lo: float = 0.5     # per-head noise std drawn uniformly in [noise_lo, noise_hi]
    noise_hi: float = 0.5
    n_keys_min: int = 0       # ragged: lengths uniform in [n_keys_min, n_keys]
    page_size: int = 16
    n_new: int = 128          # steady: newly decoded tokens on top of the budget
    pos_lo: int = 2048        # steady: current position uniform in [max(pos_lo, n_keys), pos_hi]
    pos_hi: int = 32768
    theta: float = 1e6
    fp32_pre_rope: bool = False   # also return the fp32 pre-RoPE keys (tiny config)

    def scaled(self, **kw) -> "Spec":
        return dataclasses.replace(self, **kw)


SPECS = {
    # config 0: 1 layer, 1 KV head, 1 query head, 4,096 keys, B = 512
    "tiny": Spec("tiny", 1, 1, 1, 1, 4096, 512, "oneshot", fp32_pre_rope=True),
    # config 1: Qwen3-8B shape, one-shot 32,768 -> 2,048
    "qwen3_8b_oneshot_32k": Spec("qwen3_8b_oneshot_32k", 36, 8, 4, 1, 32768, 2048, "oneshot"),
    # config 2: Qwen3-8B shape, batch 64, 2,048 kept + 128 new -> 2,048
    "qwen3_8b_steady_b64": Spec("qwen3_8b_steady_b64", 36, 8, 4, 64, 2048 + 128, 2048, "steady"),
    # config 3: Qwen3-8B shape, one sequence of 131,072 -> 4,096, noise std per head in [0.2, 1.0]
    "qwen3_8b_long_128k": Spec("qwen3_8b_long_128k", 36, 8, 4, 1, 131072, 4096, "oneshot",
                               noise_lo=0.2, noise_hi=1.0),
    # config 4: Qwen3-32B shape, batch 16, lengths U[8K, 64K], 16-token pages, B = 4,096
    "qwen3_32b_ragged_paged": Spec("qwen3_32b_ragged_paged", 64, 8, 8, 16, 65536, 4096,
                                   "ragged_paged", n_keys_min=8192),
}


@dataclasses.dataclass
class Workload:
    spec: Spec
    q_center: torch.Tensor        # [L, Hq, 128] fp32 (host)   E[q_f], interleaved (re, im) pairs
    q_mean_norm: torch.Tensor     # [L, Hq, 64]  fp32 (host)   E|q_f|
    k: torch.Tensor               # bf16; contiguous [L, S, H, N, 128] or pool [L, P, H, page, 128]
    v: torch.Tensor               # same layout as k
    seq_lens: torch.Tensor        # [S] int32 (device)
    cur_pos: torch.Tensor         # [S] int64 (device)  p_q of each sequence
    positions: Optional[torch.Tensor]   # [L, S, H, N] int32 (device) or None (= slot index)
    page_table: Optional[torch.Tensor]  # [S, max_pages] int32 (device) or None
    k_pre_fp32: Optional[torch.Tensor] = None   # [L, S, H, N, 128] fp32 pre-RoPE (tiny only)
    layer0: int = 0               # first layer of this slab (statistics are sliced to match)

    @property
    def paged(self) -> bool:
        return self.page_table is not None

    def total_keys(self) -> int:
        sp = self.spec
        return int(self.seq_lens.sum().item()) * self.k.shape[0] * sp.n_kv_heads

    def unit_rows(self, layer: int, seq: int, head: int):
        """K rows, V rows (bf16 [n, 128]) and positions (int64 [n]) of one unit, on the host."""
        n = int(self.seq_lens[seq].item())
        if self.paged:
            ps = self.spec.page_size
            npg = (n + ps - 1) // ps
            pages = self.page_table[seq, :npg].long()
            kk = self.k[layer, pages, head].reshape(npg * ps, HEAD_DIM)[:n]
            vv = self.v[layer, pages, head].reshape(npg * ps, HEAD_DIM)[:n]
        else:
            kk = self.k[layer, seq, head, :n]
            vv = self.v[layer, seq, head, :n]
        if self.positions is None:
            pos = torch.arange(n, dtype=torch.int64)
        else:
            pos = self.positions[layer, seq, head, :n].long().cpu()
        return kk.cpu(), vv.cpu(), pos


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    import numpy as np
    return t.contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def _gen(device, *key) -> torch.Generator:
    """One independent seeded stream per (workload, purpose, layer, ...) tuple."""
    h = MASTER_SEED
    for x in key:
        if isinstance(x, str):
            x = sum((i + 1) * b for i, b in enumerate(x.encode()))
        h = (h * 1000003 + int(x) + 0x9E3779B9) % (1 << 62)
    g = torch.Generator(device=device)
    g.manual_seed(h)
    return g


def rope_forward(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """What the model does before caching a key: rotate band f (components 2f, 2f+1) by the
    angle omega_f * p, omega_f = theta^(-2f/d) (Section 2.1), in float64.
    x [..., N, d] float64, pos [..., N] integer."""
    d = x.shape[-1]
    f = torch.arange(d // 2, dtype=torch.float64, device=x.device)
    omega = torch.exp(-(2.0 * f / d) * math.log(theta))
    ang = pos.to(torch.float64).unsqueeze(-1) * omega
    c, s = torch.cos(ang), torch.sin(ang)
    xr, xi = x[..., 0::2], x[..., 1::2]
    out = torch.empty_like(x)
    out[..., 0::2] = c * xr - s * xi
    out[..., 1::2] = s * xr + c * xi
    return out


def _head_noise(spec: Spec, device) -> torch.Tensor:
    """Noise std per (layer, KV head), uniform in [noise_lo, noise_hi]; [L, H] float64 on host."""
    g = _gen("cpu", spec.name, "noise")
    u = torch.rand(spec.n_layers, spec.n_kv_heads, generator=g, dtype=torch.float64)
    return spec.noise_lo + (spec.noise_hi - spec.noise_lo) * u


def make_queries(spec: Spec, layer: int, n_tokens: int, device="cpu", dtype=torch.float64) -> torch.Tensor:
    """Pre-RoPE calibration queries of one layer: q = c_q + s * eps per query head, [n_tokens, Hq, 128].
    The draws come in blocks of N_CALIB tokens, so the first N_CALIB tokens do not depend on n_tokens."""
    H, G = spec.n_kv_heads, spec.group_size
    noise = _head_noise(spec, "cpu")
    g = _gen(device, spec.name, "q", layer)
    centre = torch.randn(H * G, 1, HEAD_DIM, generator=g, dtype=torch.float64, device=device)
    std = noise[layer].repeat_interleave(G).view(H * G, 1, 1).to(device)
    out = torch.empty(n_tokens, H * G, HEAD_DIM, dtype=dtype, device=device)
    for t0 in range(0, n_tokens, N_CALIB):
        eps = torch.randn(H * G, N_CALIB, HEAD_DIM, generator=g, dtype=torch.float64, device=device)
        n = min(N_CALIB, n_tokens - t0)
        out[t0:t0 + n] = (centre + std * eps)[:, :n].transpose(0, 1).to(dtype)
    return out


def make_stats(spec: Spec):
    """Calibration statistics per query head as sample means over N_CALIB seeded draws
    q = c_q + eps (Section 3.3 / 4.1: E[q_f] and E|q_f| come from calibration data).
    Returns q_center [L, Hq, 128] fp32 and q_mean_norm [L, Hq, 64] fp32 on the host."""
    L, H, G = spec.n_layers, spec.n_kv_heads, spec.group_size
    qc = torch.empty(L, H * G, HEAD_DIM, dtype=torch.float32)
    qn = torch.empty(L, H * G, HEAD_DIM // 2, dtype=torch.float32)
    for l in range(L):
        q = make_queries(spec, l, N_CALIB, "cpu").transpose(0, 1)          # [Hq, N_CALIB, 128] float64
        qc[l] = q.mean(dim=1).to(torch.float32)
        qn[l] = torch.sqrt(q[..., 0::2] ** 2 + q[..., 1::2] ** 2).mean(dim=1).to(torch.float32)
    return qc, qn


def _layer_keys(spec: Spec, layer: int, n_seqs: int, n: int, pos: torch.Tensor, noise_l: torch.Tensor,
                device, want_pre: bool):
    """Keys and values of one layer: k = c_k + eps per KV head, rotated to its position, -> bf16.
    pos broadcastable to [S, H, n]."""
    H = spec.n_kv_heads
    g = _gen(device, spec.name, "kv", layer)
    centre = torch.randn(1, H, 1, HEAD_DIM, generator=g, dtype=torch.float64, device=device)
    eps = torch.randn(n_seqs, H, n, HEAD_DIM, generator=g, dtype=torch.float64, device=device)
    std = noise_l.to(device).view(1, H, 1, 1)
    k_pre = centre + std * eps
    del eps
    k_post = rope_forward(k_pre, pos.expand(n_seqs, H, n), spec.theta).to(torch.bfloat16)
    v = torch.randn(n_seqs, H, n, HEAD_DIM, generator=g, dtype=torch.float32, device=device).to(torch.bfloat16)
    return k_post, v, (k_pre.to(torch.float32) if want_pre else None)


def make_workload(spec: Spec, device="cpu", layer0: int = 0, n_layers: Optional[int] = None) -> Workload:
    """Build layers [layer0, layer0 + n_layers) of a workload on `device`.

    The statistics returned are sliced to the same layers, so a slab is a self-contained
    model of n_layers layers."""
    device = torch.device(device)
    L = spec.n_layers - layer0 if n_layers is None else n_layers
    H, S, N = spec.n_kv_heads, spec.n_seqs, spec.n_keys
    qc, qn = make_stats(spec)
    qc, qn = qc[layer0:layer0 + L].contiguous(), qn[layer0:layer0 + L].contiguous()
    noise = _head_noise(spec, device)

    if spec.kind == "oneshot":
        # slot i holds position i; the next query sits at position N
        seq_lens = torch.full((S,), N, dtype=torch.int32, device=device)
        cur_pos = torch.full((S,), N, dtype=torch.int64, device=device)
        pos = torch.arange(N, device=device).view(1, 1, N)
        k = torch.empty(L, S, H, N, HEAD_DIM, dtype=torch.bfloat16, device=device)
        v = torch.empty_like(k)
        kpre = torch.empty(L, S, H, N, HEAD_DIM, dtype=torch.float32, device=device) if spec.fp32_pre_rope else None
        for l in range(L):
            k[l], v[l], p = _layer_keys(spec, layer0 + l, S, N, pos, noise[layer0 + l], device, spec.fp32_pre_rope)
            if kpre is not None:
                kpre[l] = p
        return Workload(spec, qc, qn, k, v, seq_lens, cur_pos, None, None, kpre, layer0)

    if spec.kind == "steady":
        # each sequence is at position T ~ U[max(pos_lo, N), pos_hi]; the newest n_new slots hold
        # T-n_new..T-1, the older B slots a sorted sample without replacement of [0, T-n_new),
        # drawn independently per (layer, head) since each head kept different keys earlier.
        B, n_new = N - spec.n_new, spec.n_new
        g = _gen("cpu", spec.name, "T")
        lo = max(spec.pos_lo, N)
        T = torch.randint(lo, spec.pos_hi + 1, (S,), generator=g, dtype=torch.int64)
        seq_lens = torch.full((S,), N, dtype=torch.int32, device=device)
        cur_pos = T.to(device)
        positions = torch.empty(L, S, H, N, dtype=torch.int32, device=device)
        k = torch.empty(L, S, H, N, HEAD_DIM, dtype=torch.bfloat16, device=device)
        v = torch.empty_like(k)
        M = int(T.max().item()) - n_new
        limit = (cur_pos - n_new).view(S, 1, 1)
        col = torch.arange(M, device=device).view(1, 1, M)
        for l in range(L):
            gp = _gen(device, spec.name, "pos", layer0 + l)
            u = torch.rand(S, H, M, generator=gp, device=device)
            u = torch.where(col < limit, u, torch.full_like(u, -1.0))
            old = torch.topk(u, B, dim=-1).indices.sort(dim=-1).values        # [S, H, B] distinct, ascending
            new = (cur_pos.view(S, 1, 1) - n_new + torch.arange(n_new, device=device).view(1, 1, n_new))
            pos_l = torch.cat([old, new.expand(S, H, n_new)], dim=-1)
            positions[l] = pos_l.to(torch.int32)
            k[l], v[l], _ = _layer_keys(spec, layer0 + l, S, N, pos_l, noise[layer0 + l], device, False)
        return Workload(spec, qc, qn, k, v, seq_lens, cur_pos, positions, None, None, layer0)

    if spec.kind == "ragged_paged":
        ps = spec.page_size
        g = _gen("cpu", spec.name, "len")
        lens = torch.randint(spec.n_keys_min, N + 1, (S,), generator=g, dtype=torch.int64)
        npages = (lens + ps - 1) // ps
        total_pages = int(npages.sum().item())
        max_pages = int(npages.max().item())
        perm = torch.randperm(total_pages, generator=g)
        table = torch.full((S, max_pages), -1, dtype=torch.int32)
        off = 0
        for s in range(S):
            table[s, :npages[s]] = perm[off:off + npages[s]].to(torch.int32)
            off += int(npages[s])
        k = torch.zeros(L, total_pages, H, ps, HEAD_DIM, dtype=torch.bfloat16, device=device)
        v = torch.zeros_like(k)
        table_d = table.to(device)
        for l in range(L):
            for s in range(S):
                n = int(lens[s]); npg = int(npages[s]); npad = npg * ps
                sub = spec.scaled(name=f"{spec.name}/s{s}")
                pos = torch.arange(npad, device=device).view(1, 1, npad)
                kk, vv, _ = _layer_keys(sub, layer0 + l, 1, npad, pos, noise[layer0 + l], device, False)
                kk[:, :, n:] = 0
                vv[:, :, n:] = 0
                pages = table_d[s, :npg].long()
                k[l, pages] = kk[0].view(H, npg, ps, HEAD_DIM).permute(1, 0, 2, 3)
                v[l, pages] = vv[0].view(H, npg, ps, HEAD_DIM).permute(1, 0, 2, 3)
        seq_lens = lens.to(torch.int32).to(device)
        cur_pos = lens.to(device)
        return Workload(spec, qc, qn, k, v, seq_lens, cur_pos, None, table_d, None, layer0)

    raise ValueError(spec.kind)
