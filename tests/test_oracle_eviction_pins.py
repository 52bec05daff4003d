"""Pins of the oracle's stateful composition: OracleLayer.score_evict and
OracleLayer.quant_pack with pruning active (Sec. 3.2-3.3).

The leaf routines (quantiser, top-k, scores, attention) are pinned in
test_oracle_pins.py.  What is pinned here is that the *data* which survives an
eviction belongs to the tokens its origins name:

  P1  values are quantised once, on arrival (Eq. 7-9 per token): at every later frame the
      cached codes and parameters of a survivor are those of quantising its raw row, found
      through its origin; 16-bit caches hold the raw rows themselves.
  P2  a cached key stays within the accumulated Eq. 7-8 error bound (half a quantisation
      step per re-quantisation) of the raw key its origin names; first-frame keys are
      quantised once and never touched again.
  P3  the scores of an evicting step are Eq. 2-6 evaluated (literally, fp64) on the frame's
      queries and on the dequantised keys of the middle segment as the cache stood BEFORE
      the step; the survivors are the old middle tokens at the kept positions.
  P4  the regroup rule on crafted steps: a complete key group whose tokens all survive in
      place is carried over verbatim; a group that lost a token is the quantiser applied to
      the hand-assembled dequantised survivors and raw new keys.
  P5  key_mode "once" (keys quantised once, on arrival, in groups of G tokens of their frame):
      at every later frame a survivor's codes and dequantised key are exactly those of
      quantising its own frame alone, found through its origin; the parameter table holds
      exactly the groups that still have a token (bounded by the cache length, reclaimed);
      without pruning the stream equals quantise-each-frame-then-attend.

Each pin is a function of the oracle module, so that test_planted_mistakes_are_caught can
run the same pins against copies of the oracle with one plausible mistake planted in each
(on the CPU, in the oracle's source text) and require that every mistake fails a pin.
"""
import os
import types

import numpy as np
import pytest

from oracle import xkv_oracle as xo_real
from paper_2601_01204_b200 import synth

F32 = np.float32
ORACLE_SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "xkv_oracle.py")


def _frame(seed, t, H, n, d):
    return [synth.bf16_bits_to_f32(a) for a in synth.gen_frame(seed, 0, t, H, n, d)]


def _origin_to_pos(org, n):
    """origin (frame << 16 | token), frames from 1 -> (frame index from 0, token)."""
    return (org >> 16) - 1, org & 0xFFFF


# ---------------------------------------------------------------------------- P1 + P2 + P3
def pin_survivor_data_follows_origins(xo, bits, seed=23, frames=10, key_mode="regroup"):
    H, n, d, G = 4, 37, 16, 8
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=bits, budget=150,
                        key_mode=key_mode)
    arrival = []                               # key_mode "once": each frame quantised alone, (codes, dequantised)
    peak_groups = 0
    L = xo.OracleLayer(p)
    raw = []                                   # (K, V) of every frame
    kbound = {}                                # origin -> accumulated Eq. 7-8 bound per (head, channel)
    first_snapshot = None
    evicting = 0
    for t in range(frames):
        q, k, v = _frame(seed, t, H, n, d)
        raw.append((k, v))
        K_before = L.keys_dequantized().copy() if t > 0 else None
        org_before, T_before, Tf = L.origin.copy(), L.T, L.T_first
        L.step(q, k, v)
        org = L.origin.astype(np.int64)
        fi, ti = _origin_to_pos(org, n)
        Kraw = np.stack([raw[f][0][:, tok] for f, tok in zip(fi, ti)], axis=1)       # [H][T][d]
        Vraw = np.stack([raw[f][1][:, tok] for f, tok in zip(fi, ti)], axis=1)

        # ---- P3: scores from the cache as it stood before the step; survivors by kept index ----
        if T_before + n > p.budget and t > 0:
            evicting += 1
            S_lit = xo_real.score_literal(q, K_before[:, Tf:T_before], p.n_special, p.pool_g)
            Qbar = xo_real.pooled_query_literal(q, p.n_special, p.pool_g)
            Kbar = K_before[:, Tf:T_before].astype(np.float64).mean(0)
            mag = (np.abs(Qbar.mean(0))[None] * np.abs(Kbar)).sum(1)
            assert L.last_scores.shape == S_lit.shape
            assert np.all(np.abs(L.last_scores - S_lit) <= 2e-5 * mag + 1e-12), f"frame {t}: scores"
            kept = np.asarray(L.last_kept_mid)
            assert len(kept) == p.budget - Tf - n
            assert np.array_equal(kept, xo_real.select_topk(L.last_scores, len(kept)))
            want_org = np.concatenate([org_before[:Tf], org_before[Tf + kept], ((t + 1) << 16) | np.arange(n)])
            assert np.array_equal(org, want_org), f"frame {t}: origins"
            evicted = np.setdiff1d(org_before[Tf:], org)
            assert len(evicted) == (T_before - Tf) - len(kept)                       # kept + evicted = old middle

        # ---- P1: values ----
        if bits == 16:
            assert np.array_equal(L.v_val, Vraw) and np.array_equal(L.k_val, Kraw), f"frame {t}: 16-bit rows"
            continue
        vc, vs, vz = xo_real.quantize_values(Vraw.reshape(H, -1, d), bits)
        assert np.array_equal(L.v_codes, vc), f"frame {t}: value codes"
        assert np.array_equal(L.v_s.view(np.uint32), vs.view(np.uint32)), f"frame {t}: value scales"
        assert np.array_equal(L.v_z.view(np.uint32), vz.view(np.uint32)), f"frame {t}: value zero-points"
        assert np.array_equal(L.values_dequantized(), xo_real.dequantize_values(vc, vs, vz))

        # ---- P5: keys quantised once ----
        if key_mode == "once":
            kc, ks, kz = xo_real.quantize_keys(k, G, bits)
            arrival.append((kc, xo_real.dequantize_keys(kc, ks, kz, G), ks))
            want_codes = np.stack([arrival[f][0][:, tok] for f, tok in zip(fi, ti)], axis=1)
            want_deq = np.stack([arrival[f][1][:, tok] for f, tok in zip(fi, ti)], axis=1)
            assert np.array_equal(L.k_codes, want_codes), f"frame {t}: key codes"
            Kd = L.keys_dequantized()
            assert np.array_equal(Kd.view(np.uint32), want_deq.view(np.uint32)), f"frame {t}: dequantised keys"
            s_tok = np.stack([arrival[f][2][:, tok // G] for f, tok in zip(fi, ti)], axis=1)
            assert np.all(np.abs(Kd.astype(np.float64) - Kraw) <= 0.5 * s_tok * (1 + 1e-4) + 1e-6)   # one quantisation only
            live = {(int(f), int(tok) // G) for f, tok in zip(fi, ti)}
            assert len(L.k_table) == len(live) <= L.T, f"frame {t}: parameter table holds {len(L.k_table)} groups, {len(live)} live"
            assert L.export()["k_groups_live"] == len(live)
            peak_groups = max(peak_groups, len(live))
            continue

        # ---- P2: keys ----
        Kd = L.keys_dequantized()
        Tf = L.T_first
        if t == 0:
            first_snapshot = (L.k_codes.copy(), L.k_s_first.copy(), L.k_z_first.copy())
            kc, ks, kz = xo_real.quantize_keys(k, G, bits)                           # one shot, groups from 0
            assert np.array_equal(L.k_codes, kc) and np.array_equal(L.k_s_first, ks) and np.array_equal(L.k_z_first, kz)
        else:
            assert np.array_equal(L.k_codes[:, :Tf], first_snapshot[0])               # the first frame is never touched
            assert np.array_equal(L.k_s_first, first_snapshot[1]) and np.array_equal(L.k_z_first, first_snapshot[2])
        s_now = np.concatenate([L.k_s_first[:, np.arange(Tf) // G], L.k_s_rest[:, np.arange(L.T - Tf) // G]], axis=1)
        new_bound = {}
        for i, o in enumerate(org.tolist()):
            if i < Tf:
                b = kbound.get(o, 0.5 * s_now[:, i])                                  # quantised once
            else:
                b = kbound.get(o, 0.0) + 0.5 * s_now[:, i]                            # at most one more half step
            new_bound[o] = b
        kbound = new_bound
        bound = np.stack([kbound[o] for o in org.tolist()], axis=1)                   # [H][T][d]
        err = np.abs(Kd.astype(np.float64) - Kraw)
        assert np.all(err <= bound * (1 + 1e-4) + 1e-6), f"frame {t}: key error {float((err - bound).max())} over the bound"
    assert evicting >= 5
    if key_mode == "once":      # groups did die and were given back: the table is smaller than "every group ever made"
        assert peak_groups < frames * -(-n // G)


def pin_quantise_once_without_pruning_is_framewise_quantisation(xo):
    """key_mode "once", budget never reached, ragged frame sizes: the stream's attention equals
    attention over the frames quantised one by one (Eq. 7-10), bit for bit in the cache and to
    rounding in the output."""
    H, d, G = 2, 16, 16
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=10 ** 6,
                        key_mode="once")
    L = xo.OracleLayer(p)
    Kd, Vd = [], []
    for t, n in enumerate([40, 23, 64, 7]):
        q, k, v = _frame(31, t, H, n, d)
        out = L.step(q, k, v)
        kc, ks, kz = xo_real.quantize_keys(k, G, 4)
        vc, vs, vz = xo_real.quantize_values(v, 4)
        Kd.append(xo_real.dequantize_keys(kc, ks, kz, G)), Vd.append(xo_real.dequantize_values(vc, vs, vz))
        ref = xo_real.attention(q, np.concatenate(Kd, 1), np.concatenate(Vd, 1), 1 / np.sqrt(d))
        np.testing.assert_allclose(out.transpose(1, 0, 2), ref, rtol=1e-6, atol=1e-7)
        assert np.array_equal(L.keys_dequantized(), np.concatenate(Kd, 1))
    assert len(L.k_table) == 3 + 2 + 4 + 1


# ---------------------------------------------------------------------------- P4
def _crafted_stream(xo, evict_token):
    """Three frames of 16 tokens, G = 8, budget 47: at frame 3 exactly one token of frame 2 (the
    middle segment: two complete key groups) is evicted.  The queries are e_0 on every token, so
    w = e_0 and the score of a middle token is the head mean of its dequantised channel-0 key
    (Eq. 2-6); channel 0 of the keys is +8 everywhere except -8 at `evict_token`."""
    H, n, d, G = 2, 16, 8, 8
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=47)
    L = xo.OracleLayer(p)
    frames = []
    for t in range(3):
        q, k, v = _frame(73, t, H, n, d)
        q = np.zeros_like(q)
        q[:, :, 0] = 1.0
        k = k.copy()
        k[:, :, 0] = 8.0
        if t == 1:
            k[:, evict_token, 0] = -8.0
        frames.append((q, k, v))
    for t in range(2):
        L.step(*frames[t])
    before = dict(codes=L.k_codes[:, n:].copy(), s=L.k_s_rest.copy(), z=L.k_z_rest.copy(),
                  deq=L.keys_dequantized()[:, n:].copy())
    L.step(*frames[2])
    assert L.T == 47 and L.last_kept_mid.tolist() == [j for j in range(16) if j != evict_token]
    return L, before, frames[2][1], n, G


def pin_regroup_rule_on_crafted_steps(xo):
    # (A) token 3 of the middle leaves: every group of the new rest segment holds other tokens than before
    L, before, k_new, n, G = _crafted_stream(xo, evict_token=3)
    keep = [j for j in range(16) if j != 3]
    vals = np.concatenate([before["deq"][:, keep], k_new], axis=1)                    # [H][31][d] hand-assembled
    for gi in range(4):
        a, b = gi * G, min(gi * G + G, vals.shape[1])
        c, s, z = xo_real.quantize_groups(np.moveaxis(vals[:, a:b], 1, 0), 4)
        assert np.array_equal(L.k_codes[:, n + a:n + b], np.moveaxis(c, 0, 1)), f"A: group {gi} codes"
        assert np.array_equal(L.k_s_rest[:, gi], s) and np.array_equal(L.k_z_rest[:, gi], z), f"A: group {gi} parameters"
    # group 0 now holds tokens 0,1,2,4,...,8: copying the old group 0 would be wrong, and visibly so
    assert not np.array_equal(L.k_codes[:, n:n + G], before["codes"][:, :G])

    # (B) token 11 leaves: group 0 (tokens 0..7) is complete and in place -> verbatim; group 1 is rebuilt
    L, before, k_new, n, G = _crafted_stream(xo, evict_token=11)
    keep = [j for j in range(16) if j != 11]
    vals = np.concatenate([before["deq"][:, keep], k_new], axis=1)
    assert np.array_equal(L.k_codes[:, n:n + G], before["codes"][:, :G]), "B: carried codes"
    assert np.array_equal(L.k_s_rest[:, 0].view(np.uint32), before["s"][:, 0].view(np.uint32)), "B: carried scales"
    assert np.array_equal(L.k_z_rest[:, 0].view(np.uint32), before["z"][:, 0].view(np.uint32)), "B: carried zero-points"
    # the pin is sharp only if re-quantising that group would have changed something
    c0, s0, z0 = xo_real.quantize_groups(np.moveaxis(before["deq"][:, :G], 1, 0), 4)
    assert not (np.array_equal(s0.view(np.uint32), before["s"][:, 0].view(np.uint32)) and
                np.array_equal(np.moveaxis(c0, 0, 1), before["codes"][:, :G])), "crafted data: re-quantisation is a no-op"
    for gi in range(1, 4):
        a, b = gi * G, min(gi * G + G, vals.shape[1])
        c, s, z = xo_real.quantize_groups(np.moveaxis(vals[:, a:b], 1, 0), 4)
        assert np.array_equal(L.k_codes[:, n + a:n + b], np.moveaxis(c, 0, 1)), f"B: group {gi} codes"
        assert np.array_equal(L.k_s_rest[:, gi], s) and np.array_equal(L.k_z_rest[:, gi], z), f"B: group {gi} parameters"


def pin_budget_change_and_given_query_vector(xo):
    """The budget in force can be lowered between frames (mechanism for per-layer adaptive budgets,
    the paper's stated future work): the next step evicts down to it with the same rule (first and
    current frame whole, top-k of the middle).  And the row mean w of the pooled query (Eq. 2-3) may
    come from the caller instead of Q: same scores, same survivors."""
    H, n, d, G = 4, 37, 16, 8
    p = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=260)
    La, Lb = xo.OracleLayer(p), xo.OracleLayer(p)
    for t in range(9):
        q, k, v = _frame(29, t, H, n, d)
        if t == 5:
            La.set_budget(150); Lb.set_budget(150)
        if t == 8:
            La.set_budget(260); Lb.set_budget(260)
        T_before, Tf = La.T, La.T_first
        K_before = La.keys_dequantized().copy() if t else None
        La.step(q, k, v)
        w = xo_real.query_vector_canonical(xo_real.pooled_query_canonical(q, p.n_special, p.pool_g))
        Lb.append(k, v); Lb.score_evict(None, w=w); Lb.quant_pack()
        ea, eb = La.export(), Lb.export()
        assert all(np.array_equal(ea[key], eb[key]) for key in ea), f"frame {t}: given w"
        budget = 150 if 5 <= t < 8 else 260
        assert La.T == min(T_before + n, max(budget, 2 * n if t else n)), f"frame {t}: length {La.T}"
        assert np.array_equal(La.origin[:n], (1 << 16) | np.arange(n)) and np.array_equal(La.origin[-n:], ((t + 1) << 16) | np.arange(n))
        if T_before + n > budget:
            kk = budget - Tf - n
            S = xo_real.score_literal(q, K_before[:, Tf:T_before], p.n_special, p.pool_g)
            assert len(La.last_kept_mid) == kk and np.array_equal(La.last_kept_mid, xo_real.select_topk(La.last_scores, kk))
            assert np.all(np.abs(La.last_scores - S) <= 1e-4 * (np.abs(S) + 1.0))
    assert La.T == 150 + n                      # the raised budget lets the cache grow again


def pin_chunked_prefill_is_frame_causal(xo):
    """step_chunk.  (1) Nothing pruned, 16-bit: two chunks of frames give, frame by frame, what
    one-shot frame-causal attention over all tokens gives (block-triangular mask, Eq. 1), and what
    streaming the frames one by one gives.  (2) A chunk of one frame is step().  (3) With pruning
    and 4-bit storage: the cache is first arrival + top-k of the middle + the whole chunk, and frame
    f's output is attention over the dequantised cache with every token of a later chunk frame
    masked (mask built from the origins, by the independently written masked routine)."""
    H, d, G = 2, 16, 8
    sizes = [[11, 24], [16, 9, 20]]
    p16 = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=16, budget=10 ** 6)
    Lc, Ls = xo.OracleLayer(p16), xo.OracleLayer(p16)
    allq, allk, allv, fid, outs_c, outs_s = [], [], [], [], [], []
    t = 0
    for chunk in sizes:
        fr = []
        for n in chunk:
            q, k, v = _frame(41, t, H, n, d)
            fr.append((q, k, v)); allq.append(q); allk.append(k); allv.append(v); fid.append(np.full(n, t)); t += 1
            outs_s.append(Ls.step(q, k, v))
        outs_c += Lc.step_chunk([f[0] for f in fr], [f[1] for f in fr], [f[2] for f in fr])
    fid = np.concatenate(fid)
    ref = xo_real.attention_frame_causal(np.concatenate(allq, 1), np.concatenate(allk, 1), np.concatenate(allv, 1),
                                         fid, fid, 1.0 / np.sqrt(d))
    np.testing.assert_allclose(np.concatenate(outs_c, 0).transpose(1, 0, 2), ref, rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(np.concatenate(outs_c, 0), np.concatenate(outs_s, 0), rtol=1e-5, atol=1e-6)
    # (2)
    p4 = xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=60)
    La, Lb = xo.OracleLayer(p4), xo.OracleLayer(p4)
    for tt in range(5):
        q, k, v = _frame(42, tt, H, 20, d)
        oa = La.step(q, k, v)
        ob = Lb.step_chunk([q], [k], [v])[0]
        assert np.array_equal(oa, ob) and all(np.array_equal(La.export()[key], Lb.export()[key]) for key in La.export())
    # (3)
    L = xo.OracleLayer(xo.OracleParams(n_heads=H, head_dim=d, n_special=5, pool_g=4, quant_group=G, kv_bits=4, budget=90))
    chunks = [[24], [16, 16], [12, 20, 8], [16, 24]]
    t = 0
    for ci, chunk in enumerate(chunks):
        fr = [_frame(43, t + j, H, n, d) for j, n in enumerate(chunk)]
        t += len(chunk)
        T_before, org_before = L.T, L.origin.copy()
        K_before = L.keys_dequantized().copy() if ci else None
        outs = L.step_chunk([f[0] for f in fr], [f[1] for f in fr], [f[2] for f in fr])
        M = sum(chunk)
        org = L.origin
        assert np.array_equal(org[-M:], ((ci + 1) << 16) | np.arange(M))                 # the chunk is whole, as one arrival
        assert np.array_equal(org[:24], (1 << 16) | np.arange(24))                       # so is the first arrival
        if T_before + M > 90:
            assert L.T == max(90, 24 + M) and len(L.last_kept_mid) == max(0, 90 - 24 - M)
            assert np.array_equal(org[24:L.T - M], org_before[24:][L.last_kept_mid])
            if len(L.last_kept_mid):                                                     # scored with the LAST frame's query
                S = xo_real.score_literal(fr[-1][0], K_before[:, 24:T_before], 5, 4)
                assert np.all(np.abs(L.last_scores - S) <= 1e-4 * (np.abs(S) + 1.0))
        # frame ids of the cached tokens: older than the chunk -> -1, chunk tokens -> their frame in the chunk
        kf = np.full(L.T, -1)
        kf[-M:] = np.repeat(np.arange(len(chunk)), chunk)
        K, V = L.keys_dequantized(), L.values_dequantized()
        for f, (q, _, _) in enumerate(fr):
            ref = xo_real.attention_frame_causal(q, K, V, np.full(q.shape[1], f), kf, 1.0 / np.sqrt(d))
            np.testing.assert_allclose(outs[f].transpose(1, 0, 2), ref, rtol=1e-5, atol=1e-6)
    assert L.T == 90


PINS = [
    ("survivors-4bit", lambda xo: pin_survivor_data_follows_origins(xo, 4)),
    ("survivors-8bit", lambda xo: pin_survivor_data_follows_origins(xo, 8, seed=24)),
    ("survivors-16bit", lambda xo: pin_survivor_data_follows_origins(xo, 16, seed=25)),
    ("regroup-rule", pin_regroup_rule_on_crafted_steps),
    ("once-4bit", lambda xo: pin_survivor_data_follows_origins(xo, 4, seed=26, key_mode="once")),
    ("once-8bit", lambda xo: pin_survivor_data_follows_origins(xo, 8, seed=27, key_mode="once")),
    ("once-no-pruning", pin_quantise_once_without_pruning_is_framewise_quantisation),
    ("budget-and-given-w", pin_budget_change_and_given_query_vector),
    ("chunked-prefill", pin_chunked_prefill_is_frame_causal),
]


@pytest.mark.parametrize("name", [p[0] for p in PINS])
def test_eviction_path_pin(name):
    dict(PINS)[name](xo_real)


# ---------------------------------------------------------------------------- planted mistakes
# (label, text in the oracle's source, replacement).  Each is a slip that leaves every leaf routine
# intact and only breaks the bookkeeping of an evicting step.
MUTATIONS = [
    ("key regroup forgets the gather",
     "vals = np.concatenate([old_deq[:, kept], K_new], axis=1)",
     "vals = np.concatenate([old_deq[:, :kk], K_new], axis=1)"),
    ("value codes not gathered",
     "self.v_codes = np.concatenate([self.v_codes[:, keep_abs], vc], axis=1)",
     "self.v_codes = np.concatenate([self.v_codes[:, :len(keep_abs)], vc], axis=1)"),
    ("value scales not gathered",
     "self.v_s = np.concatenate([self.v_s[:, keep_abs], vs], axis=1)",
     "self.v_s = np.concatenate([self.v_s[:, :len(keep_abs)], vs], axis=1)"),
    ("value zero-points not gathered",
     "self.v_z = np.concatenate([self.v_z[:, keep_abs], vz], axis=1)",
     "self.v_z = np.concatenate([self.v_z[:, :len(keep_abs)], vz], axis=1)"),
    ("scores computed on the wrong segment",
     "K_mid = self.keys_dequantized()[:, self.T_first:, :]",
     "K_mid = self.keys_dequantized()[:, :R_old, :]"),
    ("no group is ever carried over",
     "carried = (b - a == G) and (b <= kk) and (kept[b - 1] == b - 1)",
     "carried = False"),
    ("carried without the same-tokens-in-place test",
     "carried = (b - a == G) and (b <= kk) and (kept[b - 1] == b - 1)",
     "carried = (b - a == G) and (b <= kk)"),
    ("16-bit keys not gathered",
     "self.k_val = np.concatenate([self.k_val[:, keep_abs], K_new], axis=1)",
     "self.k_val = np.concatenate([self.k_val[:, :len(keep_abs)], K_new], axis=1)"),
    ("16-bit values not gathered",
     "self.v_val = np.concatenate([self.v_val[:, keep_abs], V_new], axis=1)",
     "self.v_val = np.concatenate([self.v_val[:, :len(keep_abs)], V_new], axis=1)"),
    ("query vector from the first pooled row only",
     "w = query_vector_canonical(Qbar)",
     "w = Qbar[0].astype(F32)"),
    ("origins not gathered",
     "self.origin = np.concatenate([self.origin[keep_abs], frame_origin])",
     "self.origin = np.concatenate([self.origin[:len(keep_abs)], frame_origin])"),
    ("k counted without the first frame",
     "k = max(0, self.budget - self.T_first - n)",
     "k = max(0, self.budget - n)"),
    ("survivors re-quantised from their codes, not their values",
     "old_deq = dequantize_keys(old_codes, self.k_s_rest, self.k_z_rest, G)",
     "old_deq = old_codes.astype(F32)"),
    ("once: key codes not gathered",
     "codes_kept = self.k_codes[:, keep_abs]",
     "codes_kept = self.k_codes[:, :len(keep_abs)]"),
    ("once: group references not gathered",
     "gid_kept = self.k_gid[keep_abs]",
     "gid_kept = self.k_gid[:len(keep_abs)]"),
    ("once: parameter table never reclaimed",
     "self.k_table = {g: v for g, v in self.k_table.items() if g in live}",
     "self.k_table = dict(self.k_table)"),
    ("once: a frame's groups counted from the cache position, not from the frame's first token",
     "codes, s, z = quantize_keys(K_new, p.quant_group, p.kv_bits)\n        base",
     "codes, s, z = quantize_keys(np.concatenate([K_new[:, :self.T % p.quant_group], K_new], 1), p.quant_group, p.kv_bits)\n"
     "        codes = codes[:, self.T % p.quant_group:]\n        base"),
    ("changed budget ignored by the trigger",
     "if T <= self.budget:                           # trigger",
     "if T <= p.budget:                           # trigger"),
    ("chunk: every frame sees the whole chunk",
     "            O = attention(q, K[:, :end], V[:, :end], scale)",
     "            O = attention(q, K, V, scale)"),
    ("chunk: scored with the first frame's query",
     "        self.score_evict(Qs[-1])",
     "        self.score_evict(Qs[0])"),
    ("first frame re-quantised with the rest",
     "self.k_codes = np.concatenate([self.k_codes[:, :Tf], new_codes], axis=1)",
     "self.k_codes = np.concatenate([self.k_codes[:, :Tf] * 0, new_codes], axis=1)"),
]


def _mutant(old, new):
    src = open(ORACLE_SRC).read()
    assert src.count(old) == 1, f"mutation site not found exactly once: {old!r}"
    mod = types.ModuleType("xkv_oracle_mutant")
    mod.__dict__["__name__"] = "xkv_oracle_mutant"
    import sys
    sys.modules["xkv_oracle_mutant"] = mod               # dataclasses look their module up
    try:
        exec(compile(src.replace(old, new), ORACLE_SRC + "<mutant>", "exec"), mod.__dict__)
    finally:
        sys.modules.pop("xkv_oracle_mutant", None)
    return mod


@pytest.mark.parametrize("label,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistakes_are_caught(label, old, new):
    """Every planted mistake must fail at least one pin (the unmodified oracle passes all of them)."""
    mod = _mutant(old, new)
    caught = []
    for name, pin in PINS:
        try:
            pin(mod)
        except (AssertionError, ValueError, IndexError):
            caught.append(name)
    assert caught, f"planted mistake survives every pin: {label}"
