"""Pins for the CPU oracle: each check uses something other than the oracle's own formula
(explicit 2x2 rotations and dot products, closed forms, invariants, exhaustive search), so a
dropped term, a wrong sign or index, or a transposed operand in ``oracle/tri_oracle.c`` fails
at least one of them.  No GPU needed."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle

THETA = 1e6
D = 128
F = D // 2


def rot2x2(x, p, theta=THETA):
    """RoPE exactly as the rotation matrix of Section 2.1 prints it, one band at a time."""
    y = np.empty_like(x, dtype=np.float64)
    d = x.shape[-1]
    for f in range(d // 2):
        a = theta ** (-2.0 * f / d) * p
        R = np.array([[math.cos(a), -math.sin(a)], [math.sin(a), math.cos(a)]])
        y[2 * f:2 * f + 2] = R @ x[2 * f:2 * f + 2]
    return y


def band_abs(x):
    return np.hypot(x[..., 0::2], x[..., 1::2])


@pytest.fixture(scope="module")
def rng():
    return np.random.default_rng(12345)


def test_offsets_match_paper_fixture():
    path = os.path.join(os.path.dirname(__file__), "golden", "future_offsets.txt")
    vals = [int(l) for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(vals) == 17
    assert vals == [2 ** j for j in range(17)]
    assert list(oracle.DEFAULT_OFFSETS) == vals


def test_omega_closed_form():
    w = oracle.omega(THETA, D)
    assert w.shape == (F,)
    assert w[0] == 1.0
    assert w[F - 1] == pytest.approx(THETA ** (-126.0 / 128.0), rel=1e-14)
    ratio = w[1:] / w[:-1]
    assert np.allclose(ratio, THETA ** (-2.0 / D), rtol=1e-13)
    w4 = oracle.omega(1e4, 64)
    assert w4[1] == pytest.approx(1e4 ** (-2.0 / 64), rel=1e-14)


def test_bf16_widening_exact():
    import torch
    x = torch.randn(1000, dtype=torch.float32).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.bf16_to_f64(bits), x.to(torch.float64).numpy())


def test_unrotate_inverts_explicit_rotation(rng):
    N = 7
    k = rng.standard_normal((N, D))
    pos = np.array([0, 1, 5, 100, 4095, 65536, 131071])
    k_post = np.stack([rot2x2(k[n], pos[n]) for n in range(N)])
    back = oracle.unrotate(k_post, pos, THETA, layout=0)
    assert np.max(np.abs(back - k)) < 1e-9
    # position 0 is the identity
    assert np.array_equal(oracle.unrotate(k[:1], np.array([0]), THETA), k[:1])


def test_unrotate_inverts_workload_rope():
    import torch
    from paper_2604_04921_b200.workloads import rope_forward
    g = torch.Generator().manual_seed(3)
    k = torch.randn(5, D, generator=g, dtype=torch.float64)
    pos = torch.tensor([3, 77, 2048, 30000, 131071])
    post = rope_forward(k, pos, THETA).numpy()
    # the generator's forward rotation equals the explicit 2x2 rotation ...
    want = np.stack([rot2x2(k[n].numpy(), int(pos[n])) for n in range(5)])
    assert np.max(np.abs(post - want)) < 1e-10
    # ... and the oracle undoes it
    assert np.max(np.abs(oracle.unrotate(post, pos.numpy(), THETA) - k.numpy())) < 1e-9


@pytest.mark.parametrize("offsets", [[0], [1], [1, 2, 4], list(oracle.DEFAULT_OFFSETS)])
def test_s_trig_equals_mean_of_explicitly_rotated_dot_products(rng, offsets):
    """Brute force: rotate the query centre to p_q + delta and the key to p_k with the 2x2
    matrices and take plain dot products; their mean over D must equal the oracle's
    offset-averaged S_trig (norm term switched off)."""
    N, G = 6, 2
    c = rng.standard_normal((G, D))
    k = rng.standard_normal((N, D)) * 0.7 + rng.standard_normal(D)
    pos = np.array([0, 3, 17, 200, 1000, 4000])
    p_q = 4096
    n_mean = band_abs(c) + 0.3
    raw = oracle.score_raw(k, pos, p_q, c, n_mean, offsets=offsets, theta=THETA, norm_variant=2)
    for g in range(G):
        for n in range(N):
            kp = rot2x2(k[n], pos[n])
            bf = np.mean([np.dot(rot2x2(c[g], p_q + dl), kp) for dl in offsets])
            assert raw[g, n] == pytest.approx(bf, abs=2e-9)


def test_offset_zero_is_rope_attention_logit(rng):
    """D = {0}: the score is the ordinary RoPE logit <RoPE(q,p_q), RoPE(k,p_k)>."""
    q = rng.standard_normal(D)
    k = rng.standard_normal(D)
    for p_q, p_k in [(10, 3), (5000, 4999), (70000, 1)]:
        want = float(np.dot(rot2x2(q, p_q), rot2x2(k, p_k)))
        got = oracle.s_trig(k, q, THETA, p_q - p_k)
        assert got == pytest.approx(want, abs=1e-9)


def test_shift_invariance(rng):
    """The score depends on positions only through p_q - p_k (Section 3.2)."""
    N = 9
    c = rng.standard_normal((1, D))
    n_mean = band_abs(c) * 1.2
    k = rng.standard_normal((N, D))
    pos = np.sort(rng.choice(3000, N, replace=False))
    a = oracle.score_raw(k, pos, 3000, c, n_mean)
    b = oracle.score_raw(k, pos + 12345, 3000 + 12345, c, n_mean)
    assert np.max(np.abs(a - b)) < 1e-9
    # post-RoPE flavour: the same pre-RoPE keys cached at shifted positions
    post = np.stack([rot2x2(k[n], pos[n] + 777) for n in range(N)])
    kpre = oracle.unrotate(post, pos + 777, THETA)
    cshift = oracle.score_raw(kpre, pos + 777, 3000 + 777, c, n_mean)
    assert np.max(np.abs(a - cshift)) < 1e-8


def test_single_band_closed_form():
    """Only band f non-zero and k_f = c_f: S_trig = |c_f|^2 cos(omega_f Delta)."""
    for f in [0, 1, 17, 63]:
        c = np.zeros(D)
        c[2 * f], c[2 * f + 1] = 0.6, -1.3
        w = THETA ** (-2.0 * f / D)
        for Delta in [0.0, 1.0, 2.5, 1000.0, 65537.0]:
            want = (0.6 ** 2 + 1.3 ** 2) * math.cos(w * Delta)
            assert oracle.s_trig(c, c, THETA, Delta) == pytest.approx(want, abs=1e-9)


def test_phase_sign_convention():
    """phi_f = arg q_f - arg k_f: with k_f = q_f e^{i alpha} the term is |q|^2 cos(omega Delta - alpha),
    which peaks where omega Delta = alpha (a key *ahead* in phase is matched at positive distance)."""
    f, alpha = 5, 0.4
    w = THETA ** (-2.0 * f / D)
    q = np.zeros(D); q[2 * f] = 1.0
    k = np.zeros(D); k[2 * f], k[2 * f + 1] = math.cos(alpha), math.sin(alpha)
    assert oracle.s_trig(k, q, THETA, alpha / w) == pytest.approx(1.0, abs=1e-12)
    assert oracle.s_trig(k, q, THETA, 0.0) == pytest.approx(math.cos(alpha), abs=1e-12)
    assert oracle.s_trig(k, q, THETA, 1.0) == pytest.approx(math.cos(w - alpha), abs=1e-12)


def test_a_b_coefficient_form(rng):
    """sum_f [a_f cos(omega_f Delta) + b_f sin(omega_f Delta)], a_f = |q||k| cos(phi),
    b_f = -|q||k| sin(phi) (Appendix B.3) equals the phase form."""
    q, k = rng.standard_normal(D), rng.standard_normal(D)
    w = oracle.omega(THETA, D)
    amp = band_abs(q) * band_abs(k)
    phi = np.arctan2(q[1::2], q[0::2]) - np.arctan2(k[1::2], k[0::2])
    a, b = amp * np.cos(phi), -amp * np.sin(phi)
    for Delta in [1.0, 7.0, 333.0, 40000.0]:
        want = float(np.sum(a * np.cos(w * Delta) + b * np.sin(w * Delta)))
        assert oracle.s_trig(k, q, THETA, Delta) == pytest.approx(want, abs=1e-9)


def test_norm_term_forms_and_special_cases(rng):
    c = rng.standard_normal(D)
    k = rng.standard_normal(D)
    n_mean = band_abs(c) + rng.random(F)
    want = float(np.sum((n_mean - band_abs(c)) * band_abs(k)))
    v0 = oracle.s_norm(k, c, n_mean, variant=0)
    assert v0 == pytest.approx(want, rel=1e-13)
    # (1 - R_f) E|q_f| form of Section 4.2 agrees with the rewritten difference form
    assert oracle.s_norm(k, c, n_mean, variant=3) == pytest.approx(v0, rel=1e-12)
    # "w/o R" variant
    assert oracle.s_norm(k, c, n_mean, variant=1) == pytest.approx(float(np.sum(n_mean * band_abs(k))), rel=1e-13)
    # R_f = 1 everywhere -> no norm contribution;  0 <= R <= 1 -> S_norm >= 0
    assert oracle.s_norm(k, c, band_abs(c), variant=0) == pytest.approx(0.0, abs=1e-13)
    assert v0 >= 0.0
    # a key with zero norm scores zero in both terms
    z = np.zeros(D)
    assert oracle.s_norm(z, c, n_mean) == 0.0
    assert oracle.s_trig(z, c, THETA, 5.0) == 0.0


def test_combined_score_adds_norm_once(rng):
    """S~ = mean_delta S_trig + S_norm: the norm term does not depend on delta."""
    N = 5
    c = rng.standard_normal((1, D))
    n_mean = band_abs(c) + 0.25
    k = rng.standard_normal((N, D))
    pos = np.arange(N)
    full = oracle.score_raw(k, pos, N, c, n_mean)
    trig = oracle.score_raw(k, pos, N, c, n_mean, norm_variant=2)
    for n in range(N):
        assert full[0, n] - trig[0, n] == pytest.approx(oracle.s_norm(k[n], c[0], n_mean[0]), rel=1e-11)
    # zero centre: only the norm part with weights E|q_f| survives (the "without S_trig" ablation)
    zc = np.zeros((1, D))
    only = oracle.score_raw(k, pos, N, zc, n_mean)
    assert np.allclose(only[0], band_abs(k) @ n_mean[0], rtol=1e-12)


def test_half_split_layout_is_a_permutation(rng):
    N, G = 6, 2
    c = rng.standard_normal((G, D))
    k = rng.standard_normal((N, D))
    n_mean = band_abs(c) + 0.1
    pos = np.arange(N) * 3
    perm = np.concatenate([np.arange(0, D, 2), np.arange(1, D, 2)])  # interleaved -> half split
    a = oracle.score_raw(k, pos, 100, c, n_mean, layout=0)
    b = oracle.score_raw(k[:, perm], pos, 100, c[:, perm], n_mean, layout=1)
    assert np.max(np.abs(a - b)) < 1e-10


def test_normalize_invariants(rng):
    G, N = 4, 257
    raw = rng.standard_normal((G, N)) * rng.random((G, 1)) * 10 + rng.standard_normal((G, 1)) * 5
    z, s = oracle.normalize(raw)
    assert np.allclose(z.mean(axis=1), 0.0, atol=1e-12)
    assert np.allclose((z ** 2).mean(axis=1), 1.0, rtol=1e-12)          # population variance
    assert np.allclose(z, (raw - raw.mean(1, keepdims=True)) / raw.std(1, keepdims=True), atol=1e-12)
    assert np.array_equal(s, z.max(axis=0))
    # z-scoring removes any per-head affine rescaling
    z2, s2 = oracle.normalize(raw * np.array([[2.0], [0.5], [7.0], [1.0]]) + 3.0)
    assert np.allclose(s, s2, atol=1e-10)
    # constant head -> all zeros for that head
    raw[1] = 4.2
    z3, _ = oracle.normalize(raw)
    assert np.all(z3[1] == 0.0)
    # N = 1
    z4, s4 = oracle.normalize(np.array([[3.0], [9.0]]))
    assert np.all(z4 == 0.0) and s4[0] == 0.0


def test_g1_selection_equals_raw_topb(rng):
    N, B = 200, 37
    raw = rng.standard_normal((1, N))
    _, s = oracle.normalize(raw)
    assert set(oracle.select(s, B)) == set(np.argsort(-raw[0], kind="stable")[:B])


def test_select_exhaustive_small():
    """For tiny N the kept set must be the size-B subset with the largest score sum."""
    rng = np.random.default_rng(7)
    for N in range(1, 11):
        s = rng.standard_normal(N)
        for B in range(1, N + 2):
            idx = oracle.select(s, B)
            assert len(idx) == min(B, N)
            assert np.all(np.diff(idx) > 0)
            if B < N:
                best = max(itertools.combinations(range(N), B), key=lambda c: s[list(c)].sum())
                assert tuple(idx) == best


def test_select_ties_prefer_lower_slot():
    s = np.array([1.0, 5.0, 1.0, 1.0, 0.0, 5.0, 1.0])
    assert list(oracle.select(s, 2)) == [1, 5]
    assert list(oracle.select(s, 3)) == [0, 1, 5]
    assert list(oracle.select(s, 4)) == [0, 1, 2, 5]
    assert list(oracle.select(s, 6)) == [0, 1, 2, 3, 5, 6]
    assert list(oracle.select(s, 7)) == list(range(7))
    assert list(oracle.select(s, 100)) == list(range(7))
    assert list(oracle.select(np.zeros(5), 2)) == [0, 1]
    assert len(oracle.select(s, 0)) == 0


def test_select_matches_numpy_partition(rng):
    for N, B in [(1000, 1), (1000, 999), (4096, 512), (5000, 2048)]:
        s = rng.standard_normal(N)
        idx = oracle.select(s, B)
        want = np.sort(np.argpartition(-s, B - 1)[:B])
        assert np.array_equal(idx, want)
        assert s[idx].min() >= np.delete(s, idx).max()


def test_compact_is_a_stable_bit_copy(rng):
    rows = rng.integers(0, 2 ** 16, size=(50, 128), dtype=np.uint16)
    pos = np.sort(rng.choice(10000, 50, replace=False)).astype(np.int32)
    idx = np.array([0, 3, 4, 17, 49], dtype=np.int32)
    assert np.array_equal(oracle.compact(rows, idx), rows[idx])
    p = oracle.compact(pos, idx)
    assert np.array_equal(p, pos[idx]) and np.all(np.diff(p) > 0)
    assert oracle.compact(rows, np.zeros(0, np.int32)).shape == (0, 128)


def test_unit_bf16_chains_the_steps(rng):
    """The whole-unit entry point equals its steps applied one after another."""
    import torch
    from paper_2604_04921_b200.workloads import rope_forward, bf16_bits
    N, G, B = 300, 2, 40
    g = torch.Generator().manual_seed(11)
    k = torch.randn(N, D, generator=g, dtype=torch.float64) * 0.5 + torch.randn(D, generator=g, dtype=torch.float64)
    pos = torch.arange(N)
    bits = bf16_bits(rope_forward(k, pos, THETA).to(torch.bfloat16))
    c = rng.standard_normal((G, D))
    n_mean = band_abs(c) + 0.2
    raw, s, idx = oracle.unit_bf16(bits, pos.numpy(), N, c, n_mean, B)
    kpre = oracle.unrotate(oracle.bf16_to_f64(bits), pos.numpy(), THETA)
    assert np.max(np.abs(kpre - k.numpy())) < 0.05          # bf16 rounding only
    raw2 = oracle.score_raw(kpre, pos.numpy(), N, c, n_mean)
    assert np.array_equal(raw, raw2)
    _, s2 = oracle.normalize(raw2)
    assert np.array_equal(s, s2)
    assert np.array_equal(idx, oracle.select(s2, B))


def test_e4m3_values_and_the_unit_entry_point(rng):
    """8-bit keys: the decoder against the format's definition (1.0, the largest finite value 448, the smallest
    subnormal 2^-9, the smallest normal 2^-6, signs, both zeros, the two not-a-number codes), against torch's own
    conversion of all 256 codes, and monotone over the positive codes; the whole-unit entry point equals the steps
    on the decoded values, and equals the bf16 entry point on keys both formats hold exactly."""
    import torch
    from paper_2604_04921_b200.workloads import rope_forward, bf16_bits
    codes = np.arange(256, dtype=np.uint8)
    val = oracle.e4m3_to_f64(codes)
    want = {0x38: 1.0, 0x7E: 448.0, 0x01: 2.0 ** -9, 0x08: 2.0 ** -6, 0xB8: -1.0, 0x40: 2.0, 0x3C: 1.5, 0x00: 0.0, 0x07: 7 * 2.0 ** -9}
    for code, v in want.items():
        assert val[code] == v, (hex(code), val[code])
    assert np.signbit(val[0x80]) and val[0x80] == 0.0 and np.isnan(val[0x7F]) and np.isnan(val[0xFF])
    assert np.all(np.diff(val[:0x7F]) > 0) and np.array_equal(val[0x80:0xFF], -val[:0x7F])
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).double().numpy()
    assert np.array_equal(np.isnan(val), np.isnan(lib)) and np.array_equal(val[~np.isnan(val)], lib[~np.isnan(lib)])
    N, G, B = 200, 3, 30
    g = torch.Generator().manual_seed(3)
    k = torch.randn(N, D, generator=g, dtype=torch.float64) * 0.5 + torch.randn(D, generator=g, dtype=torch.float64)
    pos = torch.arange(N)
    k8 = rope_forward(k, pos, THETA).float().to(torch.float8_e4m3fn)
    bits8 = k8.view(torch.uint8).numpy()
    c = rng.standard_normal((G, D))
    n_mean = band_abs(c) + 0.2
    raw, s, idx = oracle.unit_e4m3(bits8, pos.numpy(), N, c, n_mean, B)
    kpre = oracle.unrotate(oracle.e4m3_to_f64(bits8), pos.numpy(), THETA)
    assert np.max(np.abs(kpre - k.numpy())) < 0.3            # e4m3 rounding only (3 mantissa bits)
    raw2 = oracle.score_raw(kpre, pos.numpy(), N, c, n_mean)
    assert np.array_equal(raw, raw2)
    assert np.array_equal(idx, oracle.select(oracle.normalize(raw2)[1], B))
    raw_b, s_b, idx_b = oracle.unit_bf16(bf16_bits(k8.to(torch.bfloat16)), pos.numpy(), N, c, n_mean, B)   # exact widening
    assert np.array_equal(raw, raw_b) and np.array_equal(s, s_b) and np.array_equal(idx, idx_b)


def test_calibration_statistics_pins(rng):
    """E[q_f], E|q_f| and R_f against closed forms and an independent computation."""
    T = 360
    # identical vectors: centre = the vector, mean norm = its band magnitudes, R = 1 in every band
    v = rng.standard_normal(D)
    c, n, r = oracle.calibrate(np.tile(v, (T, 1)))
    assert np.allclose(c, v, rtol=1e-13) and np.allclose(n, band_abs(v), rtol=1e-13) and np.allclose(r, 1.0, rtol=1e-12)
    # band f turning through whole circles at constant radius: centre 0, mean norm = radius, R = 0
    q = np.zeros((T, D))
    ang = 2 * math.pi * np.arange(T) / T
    for f in range(F):
        q[:, 2 * f], q[:, 2 * f + 1] = (f + 1) * np.cos((f % 5 + 1) * ang), (f + 1) * np.sin((f % 5 + 1) * ang)
    c, n, r = oracle.calibrate(q)
    assert np.max(np.abs(c)) < 1e-12 and np.allclose(n, np.arange(1, F + 1), rtol=1e-13) and np.max(r) < 1e-12
    # two opposite phases with weights 3:1 at unit radius: R = |3 - 1| / 4 = 1/2
    q = np.zeros((4, D)); q[:3, 10] = 1.0; q[3, 10] = -1.0
    c, n, r = oracle.calibrate(q)
    assert c[10] == pytest.approx(0.5) and n[5] == pytest.approx(1.0) and r[5] == pytest.approx(0.5)
    assert r[0] == 0.0                                   # an all-zero band: R defined as 0
    # random data: numpy on complex numbers, 0 <= R <= 1 (Appendix B.5), and the half-split layout as a permutation
    q = rng.standard_normal((T, D)) * 0.5 + rng.standard_normal(D)
    c, n, r = oracle.calibrate(q)
    z = q[:, 0::2] + 1j * q[:, 1::2]
    assert np.allclose(c[0::2] + 1j * c[1::2], z.mean(axis=0), rtol=1e-12)
    assert np.allclose(n, np.abs(z).mean(axis=0), rtol=1e-12)
    assert np.allclose(r, np.abs(z.mean(axis=0)) / np.abs(z).mean(axis=0), rtol=1e-12)
    assert np.all(r >= 0.0) and np.all(r <= 1.0 + 1e-15)
    perm = np.concatenate([np.arange(0, D, 2), np.arange(1, D, 2)])
    c2, n2, r2 = oracle.calibrate(q[:, perm], layout=1)
    assert np.allclose(c2, c[perm], rtol=1e-13) and np.allclose(n2, n, rtol=1e-13) and np.allclose(r2, r, rtol=1e-12)


def test_calibration_matches_the_workload_generator_statistics():
    """The input generator computes its per-head statistics with torch; the oracle must agree on the same draws."""
    import torch
    from paper_2604_04921_b200 import workloads as W
    sp = W.SPECS["qwen3_8b_oneshot_32k"].scaled(name="calibpin", n_layers=1, n_kv_heads=1, group_size=2)
    q = W.make_queries(sp, 0, W.N_CALIB, "cpu", dtype=torch.float64)          # [T, Hq, 128]
    qc, qn = W.make_stats(sp)
    for hq in range(2):
        c, n, r = oracle.calibrate(q[:, hq].numpy())
        assert np.allclose(c, qc[0, hq].double().numpy(), atol=1e-6)
        assert np.allclose(n, qn[0, hq].double().numpy(), atol=1e-6)


def test_oracle_reproduces_its_stored_config0_values():
    """Regression guard: the oracle on the tiny configuration against the values its committed script stored
    (tests/golden/make_config0_oracle.py, which calls only the oracle).  Floats to 1e-9 relative: libm's cos /
    atan2 may differ in the last bits between machines; the kept set must be identical."""
    import importlib.util
    here = os.path.join(os.path.dirname(__file__), "golden")
    spec = importlib.util.spec_from_file_location("make_config0_oracle", os.path.join(here, "make_config0_oracle.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.render(*mod.compute()).splitlines()
    stored = open(os.path.join(here, "config0_oracle.txt")).read().splitlines()
    assert len(now) == len(stored)
    for a, b in zip(now, stored):
        ta, tb_ = a.split(), b.split()
        if a.startswith("#") or ta[0].startswith("kept"):
            assert a == b
            continue
        assert ta[0] == tb_[0]
        for x, y in zip(ta[1:], tb_[1:]):
            assert float(x) == pytest.approx(float(y), rel=1e-9, abs=1e-9)
