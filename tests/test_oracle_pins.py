"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here touches the CUDA library.  Each test is chosen so that a
plausible mistake in the oracle (a dropped term, a wrong sign or index, a
transposed operand, a wrong rounding mode) fails it.
"""
import os

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as xo
from paper_2601_01204_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


def _rng(seed):
    return np.random.default_rng(seed)


def _bf16(x):
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x.astype(F32)))


# ---------------------------------------------------------------- quantiser
def test_quantizer_worked_example_eq7_eq8():
    rows, params = [], None
    for line in open(os.path.join(GOLDEN, "quantizer_worked_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        if len(f) == 3:
            rows.append((float(f[0]), int(f[1]), float(f[2])))
        else:
            params = (float(f[0]), float(f[1]))
    x = np.array([r[0] for r in rows], dtype=F32)[:, None]
    codes, s, z = xo.quantize_groups(x, 4)
    assert codes[:, 0].tolist() == [r[1] for r in rows]
    assert s[0] == F32(params[0]) and z[0] == F32(params[1])
    deq = xo.dequantize(codes, s, z)[:, 0]
    np.testing.assert_allclose(deq, [r[2] for r in rows], rtol=0, atol=1e-6)
    # half-even: half-away-from-zero would give code 8 for x = 0.5
    assert codes[2, 0] == 7


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_quantizer_error_bound_and_code_range(bits):
    """|x - s(q - z)| <= s/2 (Eq. 7-8), codes within [0, 2^b - 1], minimum -> code 0."""
    rng = _rng(bits)
    x = (rng.standard_normal((64, 500)) * rng.uniform(0.01, 30, 500) + rng.uniform(-20, 20, 500)).astype(F32)
    codes, s, z = xo.quantize_groups(x, bits)
    deq = xo.dequantize(codes, s, z)
    qmax = (1 << bits) - 1
    assert codes.min() >= 0 and codes.max() <= qmax
    bound = s[None] * 0.5 * (1 + 2.0 ** -20) + np.abs(z)[None] * s[None] * 2.0 ** -22 + 1e-30
    assert np.all(np.abs(x.astype(np.float64) - deq) <= bound)
    # the group minimum gets code 0 and the maximum the top code
    assert np.all(codes[x.argmin(axis=0), np.arange(500)] == 0)
    assert np.all(codes[x.argmax(axis=0), np.arange(500)] == qmax)
    # scale is the range over the number of steps (Eq. 8)
    np.testing.assert_allclose(s, (x.max(0) - x.min(0)) / qmax, rtol=1e-6)


def test_quantizer_zero_exactly_representable():
    """Eq. 8's zero-point makes real 0 a grid point when the group straddles 0."""
    rng = _rng(5)
    x = rng.standard_normal((64, 200)).astype(F32)
    x[0, :] = 0.0
    codes, s, z = xo.quantize_groups(x, 4)
    deq = xo.dequantize(codes, s, z)
    assert np.all(deq[0] == 0.0)
    assert np.all(codes[0] == z)


def test_quantizer_degenerate_group_and_regrid():
    x = np.full((64, 3), 2.75, dtype=F32)
    codes, s, z = xo.quantize_groups(x, 4)
    assert np.all(s == 1.0)
    deq = xo.dequantize(codes, s, z)
    assert np.all(np.abs(deq - x) <= 0.5)
    # a group already on a 16-level grid (exactly representable) keeps its codes
    q0 = _rng(1).integers(0, 16, size=(64, 50)).astype(np.uint8)
    q0[0], q0[1] = 0, 15
    grid = (F32(0.25) * (q0.astype(F32) - F32(7.0))).astype(F32)
    codes2, s2, z2 = xo.quantize_groups(grid, 4)
    assert np.array_equal(codes2, q0) and np.all(s2 == 0.25) and np.all(z2 == 7.0)


def test_key_and_value_grouping_axes():
    """Keys: one (s, z) per (head, 64-position group, channel); values: per (head, token)."""
    rng = _rng(2)
    K = rng.standard_normal((2, 150, 8)).astype(F32)
    codes, s, z = xo.quantize_keys(K, 64, 4)
    assert s.shape == (2, 3, 8)
    # brute force on one group/channel
    for (h, gi, c) in [(0, 0, 3), (1, 1, 7), (1, 2, 0)]:
        seg = K[h, gi * 64:min(gi * 64 + 64, 150), c]
        cc, ss, zz = xo.quantize_groups(seg[:, None], 4)
        assert ss[0] == s[h, gi, c] and zz[0] == z[h, gi, c]
        assert np.array_equal(cc[:, 0], codes[h, gi * 64:gi * 64 + len(seg), c])
    # an outlier CHANNEL must not inflate the scale of other channels
    K2 = K.copy()
    K2[:, :, 5] *= 100
    _, s_out, _ = xo.quantize_keys(K2, 64, 4)
    assert np.array_equal(np.delete(s_out, 5, axis=2), np.delete(s, 5, axis=2))
    V = rng.standard_normal((2, 10, 8)).astype(F32)
    vc, vs, vz = xo.quantize_values(V, 4)
    assert vs.shape == (2, 10)
    cc, ss, zz = xo.quantize_groups(V[1, 4][:, None], 4)
    assert ss[0] == vs[1, 4] and np.array_equal(cc[:, 0], vc[1, 4])
    np.testing.assert_allclose(xo.dequantize_values(vc, vs, vz), V, atol=float(vs.max()) * 0.51)
    np.testing.assert_allclose(xo.dequantize_keys(codes, s, z, 64), K, atol=float(s.max()) * 0.51)


# ------------------------------------------------------------------ packing
def test_nibble_order_vectors_and_roundtrip():
    for line in open(os.path.join(GOLDEN, "nibble_order.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        codes = np.array([int(v) for v in f[:8]], dtype=np.uint8)
        want = bytes(int(v, 16) for v in f[8:12])
        assert xo.pack_nibbles(codes).tobytes() == want
    q = _rng(3).integers(0, 16, size=(3, 7, 64)).astype(np.uint8)
    p = xo.pack_nibbles(q)
    assert p.shape == (3, 7, 32) and p.dtype == np.uint8
    assert np.array_equal(xo.unpack_nibbles(p), q)


def test_byte_order_of_8_bit_codes():
    """4 channels per little-endian word c0 | c2<<8 | c1<<16 | c3<<24."""
    codes = np.array([0x11, 0x22, 0x33, 0x44, 1, 2, 3, 4], dtype=np.uint8)
    p = xo.pack_bytes8(codes)
    assert p.view("<u4").tolist() == [0x11 | 0x33 << 8 | 0x22 << 16 | 0x44 << 24, 1 | 3 << 8 | 2 << 16 | 4 << 24]
    w = int(p.view("<u4")[0])
    assert (w & 0x00FF00FF) == (0x11 | 0x22 << 16) and ((w >> 8) & 0x00FF00FF) == (0x33 | 0x44 << 16)
    q = _rng(33).integers(0, 256, size=(2, 5, 64)).astype(np.uint8)
    assert np.array_equal(xo.unpack_bytes8(xo.pack_bytes8(q)), q)


# ------------------------------------------------------------------- scores
def test_pooled_query_shapes_and_partial_group():
    rng = _rng(4)
    H, n, d, nsp, g = 3, 5 + 16 * 2 + 9, 4, 5, 16
    Q = rng.standard_normal((H, n, d)).astype(F32)
    Qbar = xo.pooled_query_literal(Q, nsp, g)
    assert Qbar.shape == (xo.n_pooled(n, nsp, g), d) == (5 + 3, d)
    np.testing.assert_allclose(Qbar[:5], Q[:, :5].astype(np.float64).mean(0))       # specials untouched
    np.testing.assert_allclose(Qbar[5], Q[:, 5:21].astype(np.float64).mean((0, 1)))
    np.testing.assert_allclose(Qbar[7], Q[:, 37:46].astype(np.float64).mean((0, 1)))  # 9-token tail
    np.testing.assert_allclose(xo.pooled_query_canonical(Q, nsp, g), Qbar, rtol=1e-5, atol=1e-6)


def test_pooled_query_of_a_frame_shorter_than_the_special_tokens():
    """Fewer tokens than special tokens: every token is a special token (literal and canonical agree)."""
    Q = _rng(40).standard_normal((3, 2, 4)).astype(F32)
    lit = xo.pooled_query_literal(Q, 5, 16)
    assert lit.shape == (2, 4) == (xo.n_pooled(2, 5, 16), 4)
    np.testing.assert_allclose(lit, Q.astype(np.float64).mean(0))
    np.testing.assert_allclose(xo.pooled_query_canonical(Q, 5, 16), lit, rtol=1e-6, atol=1e-7)


def test_score_canonical_matches_literal():
    rng = _rng(6)
    H, n, d, Tp = 16, 261, 64, 300
    Q = _bf16(rng.standard_normal((H, n, d)))
    K = (rng.standard_normal((H, Tp, d)) * rng.uniform(0.5, 15, (H, 1, d))).astype(F32)
    lit = xo.score_literal(Q, K, 5, 16)
    w = xo.query_vector_canonical(xo.pooled_query_canonical(Q, 5, 16))
    can = xo.score_canonical(w, K)
    Kbar = K.astype(np.float64).mean(0)
    mag = (np.abs(w.astype(np.float64))[None] * np.abs(Kbar)).sum(1)
    assert np.all(np.abs(can - lit) <= 2e-5 * mag + 1e-12)


def test_score_special_case_is_gemv():
    """H = 1, g = 1: S = mean_i(q_i) . k_j (Eq. 2-6 collapse to a matrix-vector product)."""
    rng = _rng(7)
    Q = rng.standard_normal((1, 40, 8))
    K = rng.standard_normal((1, 33, 8))
    S = xo.score_literal(Q, K, 5, 1)
    np.testing.assert_allclose(S, K[0] @ Q[0].mean(0), rtol=1e-12, atol=1e-12)
    # no softmax and no 1/sqrt(d): doubling Q doubles S exactly
    np.testing.assert_allclose(xo.score_literal(2 * Q, K, 5, 1), 2 * S, rtol=1e-12)


def test_score_linear_and_head_permutation_invariant():
    rng = _rng(8)
    Q1 = rng.standard_normal((4, 50, 8))
    Q2 = rng.standard_normal((4, 50, 8))
    K = rng.standard_normal((4, 21, 8))
    S1, S2 = xo.score_literal(Q1, K, 5, 16), xo.score_literal(Q2, K, 5, 16)
    np.testing.assert_allclose(xo.score_literal(Q1 + 3 * Q2, K, 5, 16), S1 + 3 * S2, rtol=1e-10, atol=1e-12)
    perm = np.array([2, 0, 3, 1])
    # Q and K are averaged over heads separately (Eq. 3, Eq. 4): permuting either alone changes nothing
    np.testing.assert_allclose(xo.score_literal(Q1[perm], K, 5, 16), S1, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(xo.score_literal(Q1, K[perm], 5, 16), S1, rtol=1e-10, atol=1e-12)
    # weights: a special token counts as much as a whole 16-token group
    Qe = np.zeros((1, 5 + 32, 2))
    Qe[0, 0, 0] = 1.0
    Qg = np.zeros((1, 5 + 32, 2))
    Qg[0, 5:21, 0] = 1.0
    Ke = np.ones((1, 1, 2))
    np.testing.assert_allclose(xo.score_literal(Qe, Ke, 5, 16), xo.score_literal(Qg, Ke, 5, 16))


# ---------------------------------------------------------------- selection
def _brute_topk(S, k):
    key = xo.order_key(S).tolist()
    alive = list(range(len(key)))
    chosen = []
    for _ in range(min(k, len(alive))):
        best = alive[0]
        for j in alive[1:]:
            if key[j] > key[best]:           # strict: equal keys keep the lower position
                best = j
        chosen.append(best)
        alive.remove(best)
    return sorted(chosen)


def test_select_topk_brute_force_with_ties():
    rng = _rng(9)
    cases = [
        np.array([0.0, -0.0, 0.0, -0.0, 1.0, 1.0, -1.0], dtype=F32),
        np.zeros(9, dtype=F32),
        np.array([3, 1, 2, 3, 3, 0, 3], dtype=F32),
        rng.standard_normal(37).astype(F32),
        rng.integers(-3, 3, 50).astype(F32),
    ]
    for S in cases:
        for k in range(0, len(S) + 2):
            got = xo.select_topk(S, k).tolist()
            assert got == _brute_topk(S, k), (S, k)
    # +0 outranks -0; among equal keys the lower position wins
    S = np.array([-0.0, 0.0, 0.0], dtype=F32)
    assert xo.select_topk(S, 1).tolist() == [1]
    assert xo.select_topk(S, 2).tolist() == [1, 2]
    # largest wins (not smallest)
    assert xo.select_topk(np.array([1, 5, 3], dtype=F32), 1).tolist() == [1]


# ---------------------------------------------------------------- attention
def test_attention_against_library_and_closed_forms():
    rng = _rng(10)
    Q = rng.standard_normal((3, 17, 8)).astype(F32)
    K = rng.standard_normal((3, 29, 8)).astype(F32)
    V = rng.standard_normal((3, 29, 8)).astype(F32)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q).double(), torch.from_numpy(K).double(), torch.from_numpy(V).double(),
        scale=0.3).numpy()
    np.testing.assert_allclose(xo.attention(Q, K, V, 0.3), ref, rtol=1e-5, atol=1e-6)
    # one key: the output is that value
    np.testing.assert_allclose(xo.attention(Q, K[:, :1], V[:, :1], 0.3), np.repeat(V[:, :1], 17, 1), rtol=1e-6)
    # identical keys: uniform weights, the output is the mean value
    Ku = np.repeat(K[:, :1], 29, axis=1)
    np.testing.assert_allclose(xo.attention(Q, Ku, V, 0.3), np.repeat(V.mean(1, keepdims=True), 17, 1),
                               rtol=1e-5, atol=1e-6)
    # second, independently written routine (two-pass, row by row, with a frame mask)
    fq = np.zeros(17, dtype=np.int64)
    fk = np.zeros(29, dtype=np.int64)
    np.testing.assert_allclose(xo.attention_frame_causal(Q, K, V, fq, fk, 0.3), ref, rtol=1e-5, atol=1e-6)


def test_streaming_equals_one_shot_frame_causal_when_uncompressed():
    """Budget >= all tokens and 16-bit storage: the stream reproduces Eq. 1 exactly."""
    H, n, d, F = 2, 23, 16, 4
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=8, kv_bits=16, budget=F * n)
    L = xo.OracleLayer(p)
    Qs, Ks, Vs, outs = [], [], [], []
    for t in range(F):
        q, k, v = [synth.bf16_bits_to_f32(a) for a in synth.gen_frame(11, 0, t, H, n, d)]
        Qs.append(q), Ks.append(k), Vs.append(v)
        outs.append(L.step(q, k, v))
    Qa, Ka, Va = [np.concatenate(x, axis=1) for x in (Qs, Ks, Vs)]
    fid = np.repeat(np.arange(F), n)
    ref = xo.attention_frame_causal(Qa, Ka, Va, fid, fid, 1.0 / np.sqrt(d))      # [H][F*n][d]
    got = np.concatenate(outs, axis=0).transpose(1, 0, 2)
    np.testing.assert_allclose(got, ref, rtol=1e-5, atol=1e-6)
    assert L.T == F * n and np.array_equal(L.origin >> 16, fid + 1)


def test_streaming_4bit_no_pruning_equals_quantize_then_attend():
    """n a multiple of G: groups never change once complete, so the stream equals
    attention over K, V quantised in one go (Eq. 7-10)."""
    H, n, d, F, G = 2, 32, 16, 3, 16
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=10 ** 6)
    L = xo.OracleLayer(p)
    Ks, Vs = [], []
    for t in range(F):
        q, k, v = [synth.bf16_bits_to_f32(a) for a in synth.gen_frame(12, 0, t, H, n, d)]
        Ks.append(k), Vs.append(v)
        out = L.step(q, k, v)
    Ka, Va = np.concatenate(Ks, 1), np.concatenate(Vs, 1)
    kc, ks, kz = xo.quantize_keys(Ka, G, 4)
    vc, vs, vz = xo.quantize_values(Va, 4)
    ref = xo.attention(q, xo.dequantize_keys(kc, ks, kz, G), xo.dequantize_values(vc, vs, vz), 1 / np.sqrt(d))
    np.testing.assert_allclose(out.transpose(1, 0, 2), ref, rtol=1e-6, atol=1e-7)
    assert np.array_equal(L.k_codes, kc) and np.array_equal(L.v_codes, vc)


def test_full_precision_tail_reading_of_eq1():
    """attend(full_precision_tail=True): the frame attends to its own K_t, V_t unquantised and to
    the dequantised cache for older tokens (Eq. 1 read literally).  Pinned by:
    the first frame is plain softmax(Q K^T / sqrt(d)) V on the raw tensors (torch, fp64);
    with 16-bit storage both readings coincide; with 4-bit storage and pruning the result equals
    attention over [dequantised older part of the cache | raw K_t, V_t] assembled by hand from the
    exported cache, and the cache state is the same in both readings; and on average it is closer
    to the unquantised attention than the packed reading."""
    H, n, d, G = 2, 24, 16, 8
    scale = 1.0 / np.sqrt(d)
    frames = [[synth.bf16_bits_to_f32(a) for a in synth.gen_frame(13, 0, t, H, n, d)] for t in range(5)]

    # first frame: everything is tail
    p4 = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=3 * n)
    L = xo.OracleLayer(p4)
    q, k, v = frames[0]
    out = L.step(q, k, v, full_precision_tail=True)                      # [n][H][d]
    tq, tk, tv = [torch.from_numpy(x).double() for x in (q, k, v)]
    ref = torch.softmax(tq @ tk.transpose(1, 2) * scale, dim=-1) @ tv    # [H][n][d]
    np.testing.assert_allclose(out.transpose(1, 0, 2), ref.numpy(), rtol=1e-5, atol=1e-6)
    assert np.abs(L.attend(q) - out).max() > 1e-3                        # the packed reading differs

    # later frames, pruning active (budget 3n): hand-assembled reference, same cache in both readings
    La, Lb = xo.OracleLayer(p4), xo.OracleLayer(p4)
    err_tail, err_packed = [], []
    Kraw, Vraw, fid = [], [], []
    for t, (q, k, v) in enumerate(frames):
        oa = La.step(q, k, v, full_precision_tail=True)
        ob = Lb.step(q, k, v)
        ea, eb = La.export(), Lb.export()
        assert all(np.array_equal(ea[key], eb[key]) for key in ea)
        T = La.T
        Kd, Vd = La.keys_dequantized(), La.values_dequantized()
        Kh = np.concatenate([Kd[:, :T - n], k], axis=1)
        Vh = np.concatenate([Vd[:, :T - n], v], axis=1)
        np.testing.assert_allclose(oa.transpose(1, 0, 2), xo.attention(q, Kh, Vh, scale), rtol=1e-6, atol=1e-7)
        # against attention over the unquantised survivors
        Kraw.append(k), Vraw.append(v), fid.append(np.full(n, t + 1))
        org = La.origin
        allk, allv = np.concatenate(Kraw, 1), np.concatenate(Vraw, 1)
        pos = ((org >> 16) - 1) * n + (org & 0xFFFF)
        exact = xo.attention(q, allk[:, pos], allv[:, pos], scale).transpose(1, 0, 2)
        err_tail.append(np.linalg.norm(oa - exact)), err_packed.append(np.linalg.norm(ob - exact))
    assert La.T == 3 * n                                                 # pruning happened
    assert sum(err_tail) < sum(err_packed)

    # 16-bit storage: nothing is quantised, the readings coincide
    p16 = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=16, budget=3 * n)
    L16 = xo.OracleLayer(p16)
    for q, k, v in frames:
        L16.append(k, v); L16.score_evict(q); L16.quant_pack()
        np.testing.assert_array_equal(L16.attend(q, full_precision_tail=True), L16.attend(q))


# ------------------------------------------------------------------ eviction
@pytest.mark.parametrize("bits", [4, 16])
def test_eviction_invariants(bits):
    H, n, d = 4, 37, 16
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=8, kv_bits=bits, budget=150)
    L = xo.OracleLayer(p)
    for t in range(9):
        q, k, v = [synth.bf16_bits_to_f32(a) for a in synth.gen_frame(13, 0, t, H, n, d)]
        prev_origin = L.origin.copy()
        prev_T = L.T
        L.step(q, k, v)
        T_after_append = prev_T + n
        assert np.all(np.diff(L.origin.astype(np.int64)) > 0)              # temporal order kept
        assert np.array_equal(L.origin[:n], (1 << 16) | np.arange(n))      # first frame intact
        assert np.array_equal(L.origin[-n:], ((t + 1) << 16) | np.arange(n))  # current frame intact
        if T_after_append > p.budget:
            assert L.T == p.budget                                          # k = L_max - T_first - T_cur > 0
            kept_mid = L.origin[n:-n]
            assert len(kept_mid) == p.budget - 2 * n
            assert np.all(np.isin(kept_mid, prev_origin[n:]))               # survivors come from the old middle
            # the survivors are exactly the top-k scores
            S = L.last_scores
            thr = np.sort(S)[::-1][len(kept_mid) - 1]
            dropped = np.setdiff1d(np.arange(len(S)), L.last_kept_mid)
            assert np.all(S[L.last_kept_mid] >= thr) and np.all(S[dropped] <= thr)
        else:
            assert L.T == T_after_append and L.last_scores is None          # no pruning below the budget


def test_budget_smaller_than_first_plus_current_keeps_both():
    H, n, d = 2, 20, 8
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=8, kv_bits=4, budget=30)
    L = xo.OracleLayer(p)
    for t in range(4):
        q, k, v = [synth.bf16_bits_to_f32(a) for a in synth.gen_frame(14, 0, t, H, n, d)]
        L.step(q, k, v)
    assert L.T == 2 * n                                                     # k = max(0, 30 - 40) = 0
    assert np.array_equal(L.origin >> 16, np.repeat([1, 4], n))


def test_requantisation_of_changed_groups_only():
    """A complete group whose members all survive in place keeps codes and parameters."""
    H, n, d, G = 2, 24, 8, 8
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=10 ** 6)
    L = xo.OracleLayer(p)
    snaps = []
    for t in range(4):
        q, k, v = [synth.bf16_bits_to_f32(a) for a in synth.gen_frame(15, 0, t, H, n, d)]
        L.step(q, k, v)
        snaps.append(L.export())
    a, b = snaps[2], snaps[3]
    ng_old = a["k_s_rest"].shape[1]
    assert np.array_equal(b["k_s_rest"][:, :ng_old], a["k_s_rest"])
    assert np.array_equal(b["k_packed"][:, :a["T"]], a["k_packed"])


# ----------------------------------------------------------- input generator
def test_generator_statistics_and_outliers():
    q, k, v = [synth.bf16_bits_to_f32(a) for a in synth.gen_frame(1, 3, 7, 16, 261, 64)]
    for x in (q, v):
        assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01 and np.abs(x).max() < 6.0
    oc = synth.outlier_channels(1, 3, 16, 64)
    assert oc.shape == (16, 4) and all(len(set(r)) == 4 for r in oc.tolist())
    for h in range(16):
        sd = k[h].std(axis=0)
        assert np.all(sd[oc[h]] > 12) and np.all(np.delete(sd, oc[h]) < 1.3)
    # counter based: the same call gives the same bytes, another frame does not
    again = synth.gen_tensor_bits(1, 3, 7, synth.TENSOR_K, 16, 261, 64)
    assert np.array_equal(again, synth.f32_to_bf16_bits(k))
    other = synth.gen_tensor_bits(1, 3, 8, synth.TENSOR_K, 16, 261, 64)
    assert not np.array_equal(again, other)
    # bf16 conversion is round-to-nearest-even and exact on representable values
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5], dtype=F32)      # 1+2^-8 ties to even -> 1.0
    assert synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x)).tolist() == [1.0, 1.0, 1.015625, -2.5]
    xt = torch.randn(1000)
    assert np.array_equal(synth.f32_to_bf16_bits(xt.numpy()),
                          xt.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
