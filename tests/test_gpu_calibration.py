"""GPU parity of the calibration-statistics kernels (E[q_f], E|q_f|, R_f) against the float64 oracle, through
the C ABI.  Tolerance: the kernel adds 32 tokens in fp32 before moving to fp64 and writes fp32 results, so
|gpu - oracle| <= 1e-5 * max(1, |oracle|) holds with a wide margin (the error budget is ~2e-6 relative)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_04921_b200 import binding as tb
from paper_2604_04921_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = 1e-5


def _check(got, want):
    got, want = got.double().cpu().numpy(), np.asarray(want)
    assert np.all(np.abs(got - want) <= TOL * np.maximum(1.0, np.abs(want))), float(np.max(np.abs(got - want)))


def _oracle_all(q, layout):
    res = [oracle.calibrate(q[:, h].double().cpu().numpy(), layout=layout) for h in range(q.shape[1])]
    return [np.stack([r[i] for r in res]) for i in range(3)]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("layout", [0, 1])
def test_calibration_matches_oracle(dtype, layout):
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="calib", n_layers=1, n_kv_heads=2, group_size=3)
    q = W.make_queries(sp, 0, 5003, DEV, dtype=dtype)              # ragged: not a multiple of any tile
    cal = tb.Calibrator(q.shape[1], pair_layout=layout)
    cal.add(q)
    qc, qn, r = cal.result()
    torch.cuda.synchronize()
    c_o, n_o, r_o = _oracle_all(q, layout)
    _check(qc, c_o); _check(qn, n_o); _check(r, r_o)
    assert float(r.min()) >= 0.0 and float(r.max()) <= 1.0 + 1e-6


@pytest.mark.parametrize("dtype,pitch,lead,tma", [(torch.bfloat16, 128, 0, True), (torch.bfloat16, 136, 8, True),
                                                  (torch.bfloat16, 132, 4, False), (torch.float32, 132, 4, True)])
def test_calibration_on_both_load_paths(dtype, pitch, lead, tma):
    """Rows whose base and strides are multiples of 16 bytes are staged by the TMA unit (every fp32 layout the entry
    point accepts is one); a bf16 view that starts 8 bytes into a wider buffer with a row pitch of 132 elements has
    neither and takes the kernel on plain loads.  Both against the oracle, on enough tokens for several blocks per
    head with a ragged last tile, and with a token stride that is not the head count times the row pitch."""
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="calib3", n_layers=1, n_kv_heads=1, group_size=3)
    T, H = 40000 + 7, 3
    q = W.make_queries(sp, 0, T, DEV, dtype=dtype)
    wide = torch.zeros(T, H + 1, pitch, dtype=dtype, device=DEV)      # one spare head
    view = wide[:, :H, lead:lead + 128]
    view.copy_(q)
    es = 2 if dtype == torch.bfloat16 else 4
    assert (view.data_ptr() % 16 == 0 and view.stride(1) * es % 16 == 0 and view.stride(0) * es % 16 == 0) == tma
    cal = tb.Calibrator(H)
    cal.add(view)
    qc, qn, r = cal.result()
    torch.cuda.synchronize()
    c_o, n_o, r_o = _oracle_all(q, 0)
    _check(qc, c_o); _check(qn, n_o); _check(r, r_o)


def test_calibration_streams_in_chunks_and_feeds_the_round():
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="calib2", n_layers=1, n_kv_heads=2, n_keys=1500, budget=100)
    q = W.make_queries(sp, 0, 3 * W.N_CALIB + 17, DEV, dtype=torch.float32)
    whole = tb.Calibrator(q.shape[1]); whole.add(q)
    parts = tb.Calibrator(q.shape[1])
    for a, b in [(0, 1), (1, 1000), (1000, 1024), (1024, q.shape[0])]:
        parts.add(q[a:b])
    (c1, n1, r1), (c2, n2, r2) = whole.result(), parts.result()
    c_o, n_o, r_o = _oracle_all(q, 0)
    for got in ((c1, n1, r1), (c2, n2, r2)):
        _check(got[0], c_o); _check(got[1], n_o); _check(got[2], r_o)
    # reset starts over; a strided view (every other token) is accepted as it is
    parts.reset(); parts.add(q[::2])
    c3, n3, _ = parts.result()
    c_h, n_h, _ = _oracle_all(q[::2], 0)
    _check(c3, c_h); _check(n3, n_h)
    # the statistics drive a compression round exactly like the generator's own
    w = W.make_workload(sp, DEV)
    q_host = W.make_queries(sp, 0, W.N_CALIB, "cpu", dtype=torch.float32)      # the generator's own draws (CPU stream)
    first = tb.Calibrator(q.shape[1]); first.add(q_host.to(DEV))
    c4, n4, _ = first.result()
    assert torch.allclose(c4.cpu(), w.q_center[0], atol=2e-6) and torch.allclose(n4.cpu(), w.q_mean_norm[0], atol=2e-6)


def test_calibration_rejects_bad_arguments():
    L = tb.lib()
    st = torch.zeros(L.tri_calib_state_bytes(4) // 8, dtype=torch.float64, device=DEV)
    q = torch.zeros(16, 4, 128, dtype=torch.float32, device=DEV)
    ws = torch.zeros(1, dtype=torch.float64, device=DEV)
    assert L.tri_calib_accumulate(q.data_ptr(), 1, 16, 4, 512, 128, 0, st.data_ptr(), ws.data_ptr(), 8, None) == 3
    assert L.tri_calib_accumulate(q.data_ptr(), 1, 16, 4, 510, 128, 0, st.data_ptr(), ws.data_ptr(), 1 << 20, None) == 1
    assert L.tri_calib_accumulate(None, 1, 16, 4, 512, 128, 0, st.data_ptr(), ws.data_ptr(), 1 << 20, None) == 1
    assert L.tri_calib_reset(None, 4, None) == 1
    assert L.tri_calib_finalize(st.data_ptr(), 4, 2, q.data_ptr(), q.data_ptr(), None, None) == 1
    torch.cuda.synchronize()


def test_calibration_at_rotary_width_64():
    """Heads with a 64-wide rotary part (the MLA-style models of the paper's cross-architecture appendix): with
    interleaved pairs two adjacent heads of 64 components are one row of 128 whose 64 bands are the two heads' 32 + 32,
    so the statistics of `n_heads` narrow heads come out of a pass over `n_heads / 2` wide ones, read as [n_heads][64]
    centres and [n_heads][32] norms and mean resultant lengths.  Against the oracle run on every narrow head alone."""
    T, H = 9001, 6
    g = torch.Generator().manual_seed(64)
    q = (torch.randn(H, 64, generator=g)[None] + 0.5 * torch.randn(T, H, 64, generator=g)).to(torch.bfloat16).to(DEV)
    cal = tb.Calibrator(H // 2)
    cal.add(q.view(T, H // 2, 128))
    qc, qn, r = cal.result()
    torch.cuda.synchronize()
    res = [oracle.calibrate(q[:, h].double().cpu().numpy()) for h in range(H)]
    _check(qc.view(H, 64), np.stack([x[0] for x in res]))
    _check(qn.view(H, 32), np.stack([x[1] for x in res]))
    _check(r.view(H, 32), np.stack([x[2] for x in res]))
