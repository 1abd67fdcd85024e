"""Pins for the oracle's FP8 (E4M3) view functions: what the number format and the already-pinned bf16
functions fix, checked without re-using the oracle's own conversion formulas."""
import numpy as np
from conftest import from_bits, to_bits

from oracle import kvmem_oracle as orc

rng = np.random.default_rng(2024)


def _e4m3_value(code: int) -> float:
    """E4M3 (finite-only variant) written from the format definition: bias 7, subnormals at exponent field 0."""
    s, e, m = code >> 7, (code >> 3) & 15, code & 7
    if e == 15 and m == 7:
        return float("nan")
    v = m * 2.0 ** -9 if e == 0 else (1 + m / 8) * 2.0 ** (e - 7)
    return -v if s else v


def test_decode_matches_the_format_definition_for_all_codes():
    codes = np.arange(256, dtype=np.uint8)
    got = orc.dequantize_e4m3(codes)
    for c in range(256):
        want = _e4m3_value(c)
        assert (np.isnan(got[c]) and np.isnan(want)) or got[c] == want, c
    assert got[0x7e] == 448.0 and got[0x08] == 2.0 ** -6 and got[0x01] == 2.0 ** -9      # max, min normal, min subnormal


def test_every_finite_code_encodes_to_itself():
    finite = np.array([c for c in range(256) if (c & 0x7f) != 0x7f], np.uint8)
    vals = orc.dequantize_e4m3(finite)                       # all exactly representable in bf16 (3 mantissa bits)
    back = orc.quantize_e4m3(to_bits(vals.astype(np.float32)))
    assert np.array_equal(back, finite)


def test_rounding_is_to_nearest_with_ties_to_even_and_saturates():
    def enc(x):
        return int(orc.quantize_e4m3(to_bits(np.array([x], np.float32)))[0])
    assert enc(1.0) == 0x38 and enc(1.125) == 0x39
    assert enc(1.0625) == 0x38                               # halfway between 1.0 (even code) and 1.125: even wins
    assert enc(1.1875) == 0x3a                               # halfway between 1.125 (odd) and 1.25 (even)
    assert enc(1.09375) == 0x39                              # above the midpoint
    assert enc(448.0) == 0x7e and enc(1000.0) == 0x7e and enc(-1.0e6) == 0xfe and enc(464.0) == 0x7e
    assert enc(2.0 ** -10) == 0x00                           # half the smallest subnormal ties to zero (even)
    assert enc(1.5 * 2.0 ** -9) == 0x02                      # halfway between codes 1 and 2
    assert enc(0.0) == 0x00 and enc(-0.0) == 0x80


def test_brute_force_nearest_value_on_random_inputs_and_relative_error_bound():
    x = (rng.standard_normal(5000) * np.exp(rng.uniform(-6, 5, 5000))).astype(np.float32)
    xb = to_bits(x)
    xf = from_bits(xb).astype(np.float64)                    # the bf16 values actually quantised
    codes = orc.quantize_e4m3(xb)
    table = np.array([_e4m3_value(c) for c in range(0x7f)])  # non-negative finite values, ascending
    for v, c in zip(xf, codes):
        a = min(abs(v), 448.0)
        best = np.abs(table - a).min()
        assert abs(_e4m3_value(int(c) & 0x7f) - a) == best   # a nearest value (ties checked separately)
        assert (int(c) >> 7) == (1 if np.signbit(v) else 0)
    deq = orc.dequantize_e4m3(codes).astype(np.float64)
    normal = (np.abs(xf) >= 2.0 ** -6) & (np.abs(xf) <= 448)
    assert np.all(np.abs(deq[normal] - xf[normal]) <= np.abs(xf[normal]) * 2.0 ** -4)


def test_scale_is_applied_before_rounding():
    x = to_bits(np.array([3.0, -100.0, 0.3], np.float32))
    c = orc.quantize_e4m3(x, inv_scale=0.5)
    assert np.allclose(orc.dequantize_e4m3(c, scale=2.0), [3.0, -96.0, 0.3125], rtol=0, atol=0.02)
    assert orc.dequantize_e4m3(c)[1] == -48.0                # -100 * 0.5 = -50 -> nearest of 48 and 52 is 48 (tie -> even)


def _repo(B=16, L=1, G=2, d=16, NB=12, seed=3):
    r = np.random.default_rng(seed)
    K = to_bits(r.standard_normal((NB * B, L, G, d)).astype(np.float32))
    V = to_bits(r.standard_normal((NB * B, L, G, d)).astype(np.float32))
    table = r.permutation(NB).astype(np.int32)
    repo = orc.Repository.empty(NB, B, L, G, d)
    repo.place(K, V, table)
    return repo, table, K, V


def test_fp8_gather_is_the_quantised_gather_with_values_transposed_per_tile():
    repo, table, _, _ = _repo()
    sel = np.array([1, 4, 5, 7, 10], np.int32)               # 80 tokens: one full 64-token tile and a quarter
    cap = 128
    vK, vV = orc.gather(repo, table, sel, cap)
    k8, v8t = orc.gather_fp8(repo, table, sel, cap, k_inv_scale=0.5, v_inv_scale=2.0)
    T = len(sel) * 16
    assert np.array_equal(k8[:, :, :T], orc.quantize_e4m3(vK, 0.5)[:, :, :T])
    want_v = orc.quantize_e4m3(vV, 2.0)                      # [L][G][cap][d]
    L, G, _, d = want_v.shape
    want_vt = want_v.reshape(L, G, cap // 64, 64, d).transpose(0, 1, 2, 4, 3)
    tok = np.arange(cap).reshape(cap // 64, 64)
    live = np.broadcast_to((tok < T)[None, None, :, None, :], want_vt.shape)
    assert np.array_equal(v8t[live], want_vt[live])


def test_fp8_attention_equals_bf16_attention_over_the_dequantised_view():
    # every E4M3 value is exactly representable in bf16, so the pinned bf16 attention applies to the same numbers
    repo, table, _, _ = _repo(B=16, G=2, d=16, NB=12, seed=8)
    sel = np.array([0, 2, 3, 9, 11], np.int32)
    cap, T = 128, 80
    k8, v8t = orc.gather_fp8(repo, table, sel, cap)
    H, M, L, G, d = 4, 3, 1, 2, 16
    q = to_bits(rng.standard_normal((M, L, H, d)).astype(np.float32))
    kb = to_bits(orc.dequantize_e4m3(k8))
    vb = to_bits(orc.dequantize_e4m3(v8t).transpose(0, 1, 2, 4, 3).reshape(L, G, cap, d).copy())
    assert np.array_equal(from_bits(kb), orc.dequantize_e4m3(k8))                       # exact in bf16
    O1, lse1 = orc.attend_fp8(q, k8, v8t, T)
    O2, lse2 = orc.attend(q, np.ascontiguousarray(kb), np.ascontiguousarray(vb), T)
    assert np.array_equal(O1, O2) and np.array_equal(lse1, lse2)
    # scales: keys * 2 with scale / 2 is the same logit; values * 3 scales the output
    O3, lse3 = orc.attend_fp8(q, k8, v8t, T, k_scale=2.0, v_scale=3.0, scale=0.5 / np.sqrt(d))
    assert np.allclose(O3, 3.0 * O1, rtol=1e-6) and np.allclose(lse3, lse1, atol=1e-6)
    # and quantisation moves the result only a little relative to the bf16 view
    vK, vV = orc.gather(repo, table, sel, cap)
    O4, _ = orc.attend(q, vK, vV, T)
    assert np.abs(O4 - O1).max() < 0.1


def test_fp8_attention_with_the_query_rotated_back_reduces_to_the_known_cases():
    """attend_fp8_qrot (FP8 codes of in-block-rotated keys, query rotated back per block): at compact position 0 the
    rotation is the identity, so one tile must give attend_fp8 exactly; in general it must agree, within the rounding of
    the rotated query, with attention over keys rotated FORWARD in fp64 (the formulation it replaces); and the
    scales must act as in attend_fp8."""
    B, L, G, d, H, M, NB = 64, 1, 2, 16, 4, 3, 3
    r = np.random.default_rng(77)
    tab = orc.rope_table(1024, d, 1.0e4)
    K = to_bits(r.standard_normal((NB * B, L, G, d)).astype(np.float32))
    V = to_bits(r.standard_normal((NB * B, L, G, d)).astype(np.float32))
    q = to_bits(r.standard_normal((M, L, H, d)).astype(np.float32))
    table = np.arange(NB, dtype=np.int32)
    # repository of in-block-rotated keys, then its FP8 view
    t_in = (np.arange(NB * B) % B).astype(np.int32)
    Kp = orc.rope_rotate(np.ascontiguousarray(K.reshape(NB * B, L * G, d)), t_in, tab).reshape(K.shape)
    repo = orc.Repository.empty(NB, B, L, G, d)
    repo.place(Kp, V, table)
    sel = np.array([0, 2], np.int32)
    cap, T = 2 * B, 2 * B
    k8, v8t = orc.gather_fp8(repo, table, sel, cap, 0.5, 2.0)
    # one tile at position 0: R(0) = identity
    O1, l1 = orc.attend_fp8_qrot(q, k8, v8t, B, B, 0, tab, 2.0, 0.5)
    O2, l2 = orc.attend_fp8(q, k8, v8t, B, 2.0, 0.5)
    assert np.array_equal(O1, O2) and np.array_equal(l1, l2)
    # two tiles at first position 37: against forward rotation of the dequantised keys in fp64
    first = 37
    O3, l3 = orc.attend_fp8_qrot(q, k8, v8t, T, B, first, tab, 2.0, 0.5)
    kd = orc.dequantize_e4m3(k8, 2.0).astype(np.float64)                     # [L][G][cap][d]
    vd = orc.dequantize_e4m3(v8t, 0.5).astype(np.float64).transpose(0, 1, 2, 4, 3).reshape(L, G, cap, d)
    half = d // 2
    freq = 1.0e4 ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    qf = from_bits(q).astype(np.float64)
    for m in range(M):
        for h in range(H):
            g = h // (H // G)
            p0 = first + (np.arange(T) // B) * B                              # the block's compact position: t is already in the key
            ang = p0[:, None] * freq[None, :]
            c, s = np.cos(ang), np.sin(ang)
            kk = kd[0, g, :T]
            kr = np.concatenate([kk[:, :half] * c - kk[:, half:] * s, kk[:, half:] * c + kk[:, :half] * s], axis=1)
            logit = kr @ qf[m, 0, h] / np.sqrt(d)
            w = np.exp(logit - logit.max())
            o = (w / w.sum()) @ vd[0, g, :T]
            assert np.abs(O3[m, 0, h] - o).max() < 2e-2
            assert abs(l3[m, 0, h] - (logit.max() + np.log(w.sum()))) < 2e-2
    # a different first position changes the result (the rotation is really applied)
    O4, _ = orc.attend_fp8_qrot(q, k8, v8t, T, B, first + 300, tab, 2.0, 0.5)
    assert np.abs(O4 - O3).max() > 1e-3
