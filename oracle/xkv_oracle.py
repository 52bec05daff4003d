"""CPU oracle for the compressed-KV streaming attention path (numpy only).

TEST INFRASTRUCTURE.  This file is the slow, plain statement of what the path
computes, written from the paper's equations.  It shares no code with the CUDA
library and imports nothing from it; only tests, the smoke check and the
benchmark's CPU-baseline leg may call it.

Per layer and per incoming frame t (Q, K, V given as [H][n][d] fp32 arrays that
hold exact bf16 values) the path is, in this order:

  1. append      K_t, V_t join the cache (Sec. 3.1, text after Eq. 1)
  2. score       pooled query (Eq. 2-3) x head-averaged dequantised middle keys
                 (Eq. 4) -> S (Eq. 5-6); only when T > L_max (Sec. 3.2)
  3. evict       keep first frame, top-k of the middle, current frame (Sec. 3.2)
  4. quantise    asymmetric uniform codes (Eq. 7-8); keys per channel in groups
                 of G cache positions, values per token (Eq. 9; Sec. 4.1)
  5. attend      softmax(Q K~^T / sqrt(d)) V~ over the dequantised cache
                 (Eq. 1 with Eq. 10)

Two kinds of arithmetic live here:

  * "canonical" fp32 routines (score_canonical, quantize_groups): floating
    point decides integers there (which tokens are kept; the 4-bit codes), so
    every operation and its order is fixed and done in IEEE fp32, one rounding
    per operation, no fused multiply-add.  numpy ufuncs on float32 arrays give
    exactly that.
  * fp64 routines (score_literal, attention, attention_frame_causal): the
    plain definition, used for tolerance checks and to validate the canonical
    ones.

Readings taken where the paper is silent (each also listed in the design notes):
  - N not divisible by g: the last pooling group is averaged over its true size.
  - pooling is 1-D over consecutive patch tokens.
  - the first segment is quantised once at t = 1 in groups of G from position
    0; everything after it ("rest") is grouped in runs of G positions counted
    from the start of the rest segment.  After an update a rest group is
    carried over verbatim when it is complete and holds exactly the same
    tokens, in place, as before; every other rest group is re-quantised from
    the fp32 dequantised survivors and the fp32 new keys.
  - key_mode = "once" is the other reading of Sec. 3.3 / Sec. 4.1 (the quantiser the paper
    names quantises a group once): a frame's keys are quantised on arrival in groups of G
    consecutive tokens of that frame (the last group of a frame may be partial), codes and
    group parameters are never rewritten, a survivor carries a reference to its group's
    parameters, and a group's parameters are dropped when its last token is evicted.
  - values are quantised once per (head, token) over the d channels.
  - rounding is to nearest, ties to even; x/s is evaluated as x * (1/s).
  - max == min in a group gives s = 1.
  - the zero-point is stored unclamped as an integer-valued fp32.
  - top-k ties: larger score first under the total order of the fp32 bit
    pattern (so -0 < +0), equal scores -> lower cache position wins.
  - kept tokens stay in ascending cache order.
  - one kept set per layer, shared by all heads.

Pins (tests/test_oracle_*.py): worked quantiser example derived from Eq. 7-8,
error bound s/2, brute-force top-k, GEMV special case of the score, linearity,
streaming == one-shot frame-causal attention when nothing is pruned or
quantised, library softmax-attention on CPU, T = 1 and uniform-key closed
forms, pack/unpack vectors.  The stateful composition under pruning
(OracleLayer.score_evict, OracleLayer.quant_pack) is pinned in
tests/test_oracle_eviction_pins.py: survivors' value codes equal the
quantisation of the raw rows their origins name, cached keys stay within the
accumulated s/2 bound of those raw rows, scores equal the literal Eq. 2-6 on
the cache as it stood before the step, the regroup rule on crafted steps; the
same file plants a dozen bookkeeping mistakes in copies of this source and
requires each to fail a pin.  The reading "re-quantise changed groups" is a
choice, not something the paper fixes: parity unpinned for that reading only.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

F32 = np.float32


# --------------------------------------------------------------------------
# parameters
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class OracleParams:
    n_heads: int = 16        # H
    head_dim: int = 64       # d
    n_special: int = 5       # camera + register tokens at the head of a frame (Sec. 3.1)
    pool_g: int = 16         # g, pooling size (Sec. 4.1)
    quant_group: int = 64    # G, tokens per key group (Sec. 4.1)
    kv_bits: int = 4         # b: 4 (the paper's), 8 (same Eq. 7-8, beyond what the paper evaluates); 16 = keep bf16 values
    budget: int = 2048       # L_max
    # how the per-channel key groups (Eq. 9) live with eviction:
    #   "regroup": groups are runs of G cache positions; a group that changed is re-quantised
    #   "once":    groups are runs of G arrival positions of one frame, quantised once when the
    #              frame arrives (KIVI-style); a survivor keeps its codes and its group's (s, z)
    key_mode: str = "regroup"


# --------------------------------------------------------------------------
# Eq. 2-3: pooled query
# --------------------------------------------------------------------------
def n_pooled(n: int, n_special: int, g: int) -> int:
    """Rows of the pooled query.  A frame with fewer tokens than special tokens has only special
    tokens (Eq. 2 splits the frame's tokens; there is nothing else to split)."""
    n_special = min(n_special, n)
    return n_special + (n - n_special + g - 1) // g


def pooled_query_literal(Q: np.ndarray, n_special: int, g: int) -> np.ndarray:
    """Eq. 2-3 in fp64.  Q [H][n][d] -> Qbar [N_pooled][d]."""
    Q = Q.astype(np.float64)
    H, n, d = Q.shape
    rows = [Q[:, i, :] for i in range(min(n_special, n))]
    for a in range(n_special, n, g):
        rows.append(Q[:, a:min(a + g, n), :].mean(axis=1))
    pooled = np.stack(rows, axis=1)                    # [H][N_pooled][d]  (Eq. 2)
    return pooled.mean(axis=0)                         # (Eq. 3)


def pooled_query_canonical(Q: np.ndarray, n_special: int, g: int) -> np.ndarray:
    """Eq. 2-3 in fixed-order fp32.  Returns Qbar float32 [N_pooled][d].

    pooled[h][i][c]: special rows unchanged; a group is the sequential fp32
    sum of its tokens in order, divided by float(count).  Qbar = sequential
    sum over heads 0..H-1, times float(1/H).
    """
    Q = np.ascontiguousarray(Q, dtype=F32)
    H, n, d = Q.shape
    n_special = min(n_special, n)
    Np = n_pooled(n, n_special, g)
    Qbar = np.zeros((Np, d), dtype=F32)
    inv_h = F32(1.0) / F32(H)
    for i in range(Np):
        if i < n_special:
            pooled = Q[:, i, :].copy()                 # [H][d]
        else:
            a = n_special + (i - n_special) * g
            b = min(a + g, n)
            pooled = Q[:, a, :].copy()
            for t in range(a + 1, b):
                pooled = pooled + Q[:, t, :]
            pooled = pooled / F32(b - a)
        acc = pooled[0].copy()
        for h in range(1, H):
            acc = acc + pooled[h]
        Qbar[i] = acc * inv_h
    return Qbar


def query_vector_canonical(Qbar: np.ndarray) -> np.ndarray:
    """w[c] = (sequential sum_i Qbar[i][c]) / float(N_pooled), fp32.

    Eq. 5-6 average the rows of Qbar Kbar^T; by linearity that is w . Kbar[j].
    """
    acc = Qbar[0].astype(F32).copy()
    for i in range(1, Qbar.shape[0]):
        acc = acc + Qbar[i]
    return acc / F32(Qbar.shape[0])


# --------------------------------------------------------------------------
# Eq. 4-6: importance scores of the middle segment
# --------------------------------------------------------------------------
def score_literal(Q: np.ndarray, K_mid: np.ndarray, n_special: int, g: int) -> np.ndarray:
    """Eq. 2-6 verbatim in fp64 with S_matrix materialised.

    Q [H][n][d], K_mid [H][T_prunable][d] (dequantised middle keys).
    """
    Qbar = pooled_query_literal(Q, n_special, g)       # [Np][d]
    Kbar = K_mid.astype(np.float64).mean(axis=0)       # Eq. 4  [Tp][d]
    S_matrix = Qbar @ Kbar.T                           # Eq. 5  [Np][Tp]
    return S_matrix.mean(axis=0)                       # Eq. 6


def score_canonical(w: np.ndarray, K_mid: np.ndarray) -> np.ndarray:
    """Fixed-order fp32 scores.  w float32[d]; K_mid float32 [H][Tp][d].

    Kbar[j][c] = (sequential sum over heads) * float(1/H);
    S[j] = balanced binary tree, natural channel order, over w[c]*Kbar[j][c].
    """
    K_mid = np.ascontiguousarray(K_mid, dtype=F32)
    H, Tp, d = K_mid.shape
    assert d & (d - 1) == 0, "head_dim must be a power of two for the tree"
    acc = K_mid[0].copy()
    for h in range(1, H):
        acc = acc + K_mid[h]
    Kbar = acc * (F32(1.0) / F32(H))
    p = Kbar * w.astype(F32)[None, :]
    while p.shape[1] > 1:
        p = p[:, 0::2] + p[:, 1::2]
    return p[:, 0].astype(F32)


# --------------------------------------------------------------------------
# top-k selection of the middle segment (Sec. 3.2)
# --------------------------------------------------------------------------
def order_key(S: np.ndarray) -> np.ndarray:
    """uint32 key whose unsigned order is the total order of fp32 bit patterns."""
    u = np.ascontiguousarray(S, dtype=F32).view(np.uint32)
    neg = (u >> np.uint32(31)).astype(bool)
    return np.where(neg, ~u, u | np.uint32(0x80000000)).astype(np.uint32)


def select_topk(S: np.ndarray, k: int) -> np.ndarray:
    """Positions (ascending) of the k largest scores; ties -> lower position."""
    Tp = S.shape[0]
    if k <= 0:
        return np.zeros(0, dtype=np.int64)
    if k >= Tp:
        return np.arange(Tp, dtype=np.int64)
    key = order_key(S).astype(np.int64)
    pos = np.arange(Tp, dtype=np.int64)
    order = np.lexsort((pos, -key))                    # key descending, then position ascending
    return np.sort(order[:k])


# --------------------------------------------------------------------------
# Eq. 7-8: asymmetric uniform quantiser, canonical fp32
# --------------------------------------------------------------------------
def quantize_groups(x: np.ndarray, bits: int):
    """Quantise along axis 0.  x float32 [m][...] is one group per trailing index.

    Returns (codes uint8 [m][...], s float32 [...], z float32 [...]).
      r = max - min; s = r / (2^b - 1), or 1 when r == 0       (Eq. 8)
      inv = 1 / s;  z = rint(-min * inv) + 0.0                  (Eq. 8)
      q = clamp(rint(x * inv) + z, 0, 2^b - 1)                  (Eq. 7)
    """
    x = np.ascontiguousarray(x, dtype=F32)
    qmax = F32((1 << bits) - 1)
    mn = x.min(axis=0)
    mx = x.max(axis=0)
    r = mx - mn
    s = np.where(r == 0, F32(1.0), r / qmax).astype(F32)
    inv = (F32(1.0) / s).astype(F32)
    z = (np.rint((-mn) * inv) + F32(0.0)).astype(F32)
    q = np.rint(x * inv[None]) + z[None]
    q = np.minimum(np.maximum(q, F32(0.0)), qmax)
    return q.astype(np.uint8), s, z


def dequantize(codes: np.ndarray, s: np.ndarray, z: np.ndarray) -> np.ndarray:
    """Eq. 10: x~ = s * (q - z) in fp32; the subtraction is exact."""
    return (s * (codes.astype(F32) - z)).astype(F32)


def quantize_keys(K: np.ndarray, G: int, bits: int):
    """Per-channel key quantisation (Eq. 9), groups of G positions from 0.

    K float32 [H][T][d] -> codes uint8 [H][T][d], s, z float32 [H][ceil(T/G)][d].
    """
    H, T, d = K.shape
    ng = (T + G - 1) // G
    codes = np.zeros((H, T, d), dtype=np.uint8)
    s = np.zeros((H, ng, d), dtype=F32)
    z = np.zeros((H, ng, d), dtype=F32)
    for gi in range(ng):
        a, b = gi * G, min(gi * G + G, T)
        c, s[:, gi], z[:, gi] = quantize_groups(np.moveaxis(K[:, a:b], 1, 0), bits)
        codes[:, a:b] = np.moveaxis(c, 0, 1)
    return codes, s, z


def dequantize_keys(codes: np.ndarray, s: np.ndarray, z: np.ndarray, G: int) -> np.ndarray:
    H, T, d = codes.shape
    gi = np.arange(T) // G
    return dequantize(codes, s[:, gi, :], z[:, gi, :])


def quantize_values(V: np.ndarray, bits: int):
    """Per-token value quantisation (Eq. 9): one group per (head, token).

    V float32 [H][n][d] -> codes uint8 [H][n][d], s, z float32 [H][n].
    """
    codes, s, z = quantize_groups(np.moveaxis(V, 2, 0), bits)   # groups along d
    return np.moveaxis(codes, 0, 2).copy(), s, z


def dequantize_values(codes: np.ndarray, s: np.ndarray, z: np.ndarray) -> np.ndarray:
    return dequantize(codes, s[:, :, None], z[:, :, None])


# --------------------------------------------------------------------------
# 4-bit packing: 8 channels -> one little-endian 32-bit word
# --------------------------------------------------------------------------
# Channels 8w..8w+7 of a row go to word w.  Even channels fill the low 16 bits,
# odd channels the high 16 bits, so that the two nibbles selected by the mask
# 0x000F000F << 4j are the adjacent channels (2j, 2j+1):
#   word = c0 | c2<<4 | c4<<8 | c6<<12 | c1<<16 | c3<<20 | c5<<24 | c7<<28
_NIBBLE_SHIFT = np.array([0, 16, 4, 20, 8, 24, 12, 28], dtype=np.uint32)


def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    """uint8 codes [...][d] (values 0..15) -> uint8 [...][d/2] packed bytes."""
    d = codes.shape[-1]
    assert d % 8 == 0
    c = codes.astype(np.uint32).reshape(codes.shape[:-1] + (d // 8, 8))
    words = np.zeros(c.shape[:-1], dtype=np.uint32)
    for i in range(8):
        words |= c[..., i] << _NIBBLE_SHIFT[i]
    b = np.ascontiguousarray(words.astype("<u4")).view(np.uint8)
    return b.reshape(codes.shape[:-1] + (d // 2,))


def unpack_nibbles(packed: np.ndarray) -> np.ndarray:
    """Inverse of pack_nibbles."""
    dh = packed.shape[-1]
    words = np.ascontiguousarray(packed).view("<u4").astype(np.uint32)
    words = words.reshape(packed.shape[:-1] + (dh // 4,))
    out = np.zeros(words.shape + (8,), dtype=np.uint8)
    for i in range(8):
        out[..., i] = ((words >> _NIBBLE_SHIFT[i]) & np.uint32(0xF)).astype(np.uint8)
    return out.reshape(packed.shape[:-1] + (dh * 2,))


# 8-bit packing: 4 channels -> one little-endian 32-bit word c0 | c2<<8 | c1<<16 | c3<<24, i.e. the
# bytes of channels (0, 2, 1, 3) in memory order, so that the mask 0x00FF00FF selects the adjacent
# channels (0, 1) and the same mask on the word shifted right by 8 selects (2, 3).
def pack_bytes8(codes: np.ndarray) -> np.ndarray:
    """uint8 codes [...][d] (values 0..255) -> uint8 [...][d] in storage order."""
    d = codes.shape[-1]
    assert d % 4 == 0
    c = codes.reshape(codes.shape[:-1] + (d // 4, 4))
    return np.ascontiguousarray(c[..., [0, 2, 1, 3]]).reshape(codes.shape)


def unpack_bytes8(packed: np.ndarray) -> np.ndarray:
    """Inverse of pack_bytes8 (the permutation is its own inverse)."""
    return pack_bytes8(packed)


# --------------------------------------------------------------------------
# Eq. 1: attention
# --------------------------------------------------------------------------
def attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """softmax(Q K^T * scale) V per head, fp64 inside.  [H][n][d],[H][T][d] -> [H][n][d] fp32."""
    Q = Q.astype(np.float64)
    K = K.astype(np.float64)
    V = V.astype(np.float64)
    out = np.zeros(Q.shape, dtype=np.float64)
    for h in range(Q.shape[0]):
        logits = (Q[h] @ K[h].T) * scale
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        out[h] = p @ V[h]
    return out.astype(F32)


def attention_frame_causal(Q: np.ndarray, K: np.ndarray, V: np.ndarray,
                           frame_of_q: np.ndarray, frame_of_k: np.ndarray,
                           scale: float) -> np.ndarray:
    """One-shot frame-causal attention: query of frame a sees keys of frames <= a.

    Row-by-row two-pass softmax (max, then sum), written independently of
    attention() above.  Q [H][M][d], K, V [H][T][d]; frame ids int arrays.
    """
    H, M, d = Q.shape
    out = np.zeros((H, M, d), dtype=np.float64)
    Kd = K.astype(np.float64)
    Vd = V.astype(np.float64)
    for h in range(H):
        for i in range(M):
            vis = frame_of_k <= frame_of_q[i]
            lg = (Kd[h][vis] @ Q[h, i].astype(np.float64)) * scale
            m = lg.max()
            e = np.exp(lg - m)
            out[h, i] = (e[:, None] * Vd[h][vis]).sum(axis=0) / e.sum()
    return out.astype(F32)


# --------------------------------------------------------------------------
# per-layer streaming state
# --------------------------------------------------------------------------
class OracleLayer:
    """KV cache of one global-attention layer under joint pruning + quantisation."""

    def __init__(self, p: OracleParams):
        self.p = p
        H, d = p.n_heads, p.head_dim
        self.budget = p.budget                         # L_max in force (set_budget may lower or restore it)
        self.frames = 0
        self.T_first = 0
        # quantised cache, logical order.  bits == 16: k_val/v_val hold fp32 copies of bf16.
        self.k_codes = np.zeros((H, 0, d), dtype=np.uint8)
        self.k_s_first = np.zeros((H, 0, d), dtype=F32)
        self.k_z_first = np.zeros((H, 0, d), dtype=F32)
        self.k_s_rest = np.zeros((H, 0, d), dtype=F32)
        self.k_z_rest = np.zeros((H, 0, d), dtype=F32)
        self.v_codes = np.zeros((H, 0, d), dtype=np.uint8)
        self.v_s = np.zeros((H, 0), dtype=F32)
        self.v_z = np.zeros((H, 0), dtype=F32)
        self.k_val = np.zeros((H, 0, d), dtype=F32)
        self.v_val = np.zeros((H, 0, d), dtype=F32)
        self.origin = np.zeros(0, dtype=np.int32)      # (frame << 16) | token
        # key_mode "once": group id (frame << 16 | group within the frame) of every cached token and
        # the parameter table {group id: (s [H][d], z [H][d])} of the groups that still have a token
        self.k_gid = np.zeros(0, dtype=np.int64)
        self.k_table = {}
        # pending (appended, not yet quantised) frame
        self._new_k = None
        self._new_v = None
        self._kept_rest = None                         # ascending old rest indices that survive
        # the newest frame as it arrived (bf16 values in fp32), kept for attend(full_precision_tail=True)
        self._cur_k = None
        self._cur_v = None
        # diagnostics of the last step
        self.last_scores = None
        self.last_kept_mid = None
        self.last_w = None

    # ---- sizes -----------------------------------------------------------
    @property
    def T(self) -> int:
        """Tokens in the quantised cache (a pending, un-quantised frame is not counted)."""
        return int(self.origin.shape[0])

    def _rest_len(self) -> int:
        return self.origin.shape[0] - self.T_first

    # ---- dequantised views ----------------------------------------------
    def keys_dequantized(self) -> np.ndarray:
        """K~ of the whole quantised cache, fp32 [H][T][d] (Eq. 10)."""
        p = self.p
        if p.kv_bits == 16:
            return self.k_val
        if p.key_mode == "once":
            s, z = self.key_params_per_token()
            return dequantize(self.k_codes, s, z)
        Tf = self.T_first
        first = dequantize_keys(self.k_codes[:, :Tf], self.k_s_first, self.k_z_first, p.quant_group)
        rest = dequantize_keys(self.k_codes[:, Tf:], self.k_s_rest, self.k_z_rest, p.quant_group)
        return np.concatenate([first, rest], axis=1)

    def key_params_per_token(self):
        """key_mode "once": (s, z) fp32 [H][T][d], every token looked up through its group id."""
        H, d = self.p.n_heads, self.p.head_dim
        s = np.zeros((H, self.T, d), dtype=F32)
        z = np.zeros((H, self.T, d), dtype=F32)
        for i, g in enumerate(self.k_gid.tolist()):
            s[:, i], z[:, i] = self.k_table[g]
        return s, z

    def values_dequantized(self) -> np.ndarray:
        if self.p.kv_bits == 16:
            return self.v_val
        return dequantize_values(self.v_codes, self.v_s, self.v_z)

    # ---- step 1: append --------------------------------------------------
    def append(self, K: np.ndarray, V: np.ndarray) -> None:
        """Take frame t's K, V ([H][n][d] fp32 holding bf16 values)."""
        assert self._new_k is None, "append called twice without quant_pack"
        self.frames += 1
        self._new_k = np.ascontiguousarray(K, dtype=F32)
        self._new_v = np.ascontiguousarray(V, dtype=F32)
        self._cur_k, self._cur_v = self._new_k, self._new_v
        self._kept_rest = None
        self.last_scores = None
        self.last_kept_mid = None

    def set_budget(self, budget: int) -> None:
        """Token budget L_max used from the next frame on (per-layer adaptive budgets are the
        paper's stated future work; this is only the mechanism).  At most the budget the layer was
        created with."""
        assert self._new_k is None and 1 <= budget <= self.p.budget
        self.budget = int(budget)

    # ---- steps 2-3: score and evict ---------------------------------------
    def score_evict(self, Q: np.ndarray | None, w: np.ndarray | None = None) -> None:
        """Decide which middle tokens survive (Sec. 3.2).  Q [H][n][d]; or, with Q = None, the
        row mean w [d] of the pooled query (Eq. 2-3, fp32) as computed by whoever produced Q."""
        p = self.p
        assert self._new_k is not None
        n = self._new_k.shape[1]
        R_old = self._rest_len()
        if self.frames == 1:
            self._kept_rest = np.zeros(0, dtype=np.int64)
            return
        T = self.origin.shape[0] + n                   # cache length after the append
        if T <= self.budget:                           # trigger: only when T > L_max
            self._kept_rest = np.arange(R_old, dtype=np.int64)
            return
        k = max(0, self.budget - self.T_first - n)
        # the middle segment is exactly the old rest segment (first | middle | current)
        K_mid = self.keys_dequantized()[:, self.T_first:, :]
        if w is None:
            Qbar = pooled_query_canonical(Q, p.n_special, p.pool_g)
            w = query_vector_canonical(Qbar)
        w = np.ascontiguousarray(w, dtype=F32)
        S = score_canonical(w, K_mid)
        kept = select_topk(S, k)
        self.last_w, self.last_scores, self.last_kept_mid = w, S, kept
        self._kept_rest = kept

    # ---- step 4: quantise the final cache ---------------------------------
    def quant_pack(self) -> None:
        p = self.p
        H, d, G = p.n_heads, p.head_dim, p.quant_group
        assert self._new_k is not None and self._kept_rest is not None
        K_new, V_new = self._new_k, self._new_v
        n = K_new.shape[1]
        frame_origin = (np.int32(self.frames) << 16) | np.arange(n, dtype=np.int32)

        if self.frames == 1:
            self.T_first = n
            self.origin = frame_origin
            if p.kv_bits == 16:
                self.k_val, self.v_val = K_new, V_new
            elif p.key_mode == "once":
                self.k_codes = self._quantise_frame_keys_once(K_new)
                self.v_codes, self.v_s, self.v_z = quantize_values(V_new, p.kv_bits)
            else:
                self.k_codes, self.k_s_first, self.k_z_first = quantize_keys(K_new, G, p.kv_bits)
                self.v_codes, self.v_s, self.v_z = quantize_values(V_new, p.kv_bits)
            self._new_k = self._new_v = None
            return

        Tf = self.T_first
        kept = self._kept_rest
        kk = kept.shape[0]
        keep_abs = np.concatenate([np.arange(Tf, dtype=np.int64), Tf + kept])
        self.origin = np.concatenate([self.origin[keep_abs], frame_origin])

        if p.kv_bits == 16:
            self.k_val = np.concatenate([self.k_val[:, keep_abs], K_new], axis=1)
            self.v_val = np.concatenate([self.v_val[:, keep_abs], V_new], axis=1)
            self._new_k = self._new_v = None
            return

        # values: quantised once on arrival, afterwards only gathered
        vc, vs, vz = quantize_values(V_new, p.kv_bits)
        self.v_codes = np.concatenate([self.v_codes[:, keep_abs], vc], axis=1)
        self.v_s = np.concatenate([self.v_s[:, keep_abs], vs], axis=1)
        self.v_z = np.concatenate([self.v_z[:, keep_abs], vz], axis=1)

        if p.key_mode == "once":
            # keys: survivors keep codes and group; the frame is quantised on its own; groups
            # without a token left give their parameters back
            gid_kept = self.k_gid[keep_abs]
            codes_kept = self.k_codes[:, keep_abs]
            self.k_gid = gid_kept
            new_codes = self._quantise_frame_keys_once(K_new)
            self.k_codes = np.concatenate([codes_kept, new_codes], axis=1)
            live = set(self.k_gid.tolist())
            self.k_table = {g: v for g, v in self.k_table.items() if g in live}
            self._new_k = self._new_v = None
            return

        # keys: regroup the rest segment
        old_codes = self.k_codes[:, Tf:]
        old_deq = dequantize_keys(old_codes, self.k_s_rest, self.k_z_rest, G)
        R_new = kk + n
        ng = (R_new + G - 1) // G
        new_codes = np.zeros((H, R_new, d), dtype=np.uint8)
        new_s = np.zeros((H, ng, d), dtype=F32)
        new_z = np.zeros((H, ng, d), dtype=F32)
        vals = np.concatenate([old_deq[:, kept], K_new], axis=1)     # fp32 [H][R_new][d]
        for gi in range(ng):
            a, b = gi * G, min(gi * G + G, R_new)
            carried = (b - a == G) and (b <= kk) and (kept[b - 1] == b - 1)
            if carried:
                new_codes[:, a:b] = old_codes[:, a:b]
                new_s[:, gi] = self.k_s_rest[:, gi]
                new_z[:, gi] = self.k_z_rest[:, gi]
            else:
                c, new_s[:, gi], new_z[:, gi] = \
                    quantize_groups(np.moveaxis(vals[:, a:b], 1, 0), p.kv_bits)
                new_codes[:, a:b] = np.moveaxis(c, 0, 1)
        self.k_codes = np.concatenate([self.k_codes[:, :Tf], new_codes], axis=1)
        self.k_s_rest, self.k_z_rest = new_s, new_z
        self._new_k = self._new_v = None

    def _quantise_frame_keys_once(self, K_new: np.ndarray) -> np.ndarray:
        """key_mode "once": Eq. 7-9 on the frame alone, groups of G tokens from its first token;
        registers the groups' parameters and appends the tokens' group ids.  Returns the codes."""
        p = self.p
        n = K_new.shape[1]
        codes, s, z = quantize_keys(K_new, p.quant_group, p.kv_bits)
        base = np.int64(self.frames) << 16
        for g in range(s.shape[1]):
            self.k_table[int(base | g)] = (s[:, g].copy(), z[:, g].copy())
        self.k_gid = np.concatenate([self.k_gid, base | (np.arange(n, dtype=np.int64) // p.quant_group)])
        return codes

    # ---- step 5: attention over the packed cache ---------------------------
    def attend(self, Q: np.ndarray, scale: float | None = None, full_precision_tail: bool = False) -> np.ndarray:
        """Eq. 1 with Eq. 10.  Every cached token is from a frame <= t, so all are visible.

        full_precision_tail: Eq. 1 read literally -- the frame attends to its own K_t, V_t as they
        arrived and to the dequantised cache for everything older.  The newest frame holds the last
        n positions of the cache; the cache itself (what later frames will see) is the same in
        both readings.

        Returns fp32 [n][H][d].
        """
        if scale is None:
            scale = 1.0 / np.sqrt(self.p.head_dim)
        K, V = self.keys_dequantized(), self.values_dequantized()
        if full_precision_tail:
            n = self._cur_k.shape[1]
            K = np.concatenate([K[:, :K.shape[1] - n], self._cur_k], axis=1)
            V = np.concatenate([V[:, :V.shape[1] - n], self._cur_v], axis=1)
        O = attention(Q, K, V, scale)
        return np.ascontiguousarray(np.transpose(O, (1, 0, 2)))

    def step(self, Q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float | None = None,
             full_precision_tail: bool = False):
        self.append(K, V)
        self.score_evict(Q)
        self.quant_pack()
        return self.attend(Q, scale, full_precision_tail)

    # ---- a chunk of frames at once -----------------------------------------
    def step_chunk(self, Qs, Ks, Vs, scale: float | None = None):
        """Several frames arriving together (offline sequences): the chunk is one arrival for the
        maintenance of Sec. 3.2 -- it plays the part of the current frame, the middle segment is
        scored with the query of the chunk's last frame -- and its attention is frame-causal
        (Eq. 1): frame f of the chunk sees everything older than the chunk and the chunk's frames
        0..f, i.e. a prefix of the cache.  Returns the outputs per frame, each fp32 [n_f][H][d]."""
        if scale is None:
            scale = 1.0 / np.sqrt(self.p.head_dim)
        self.append(np.concatenate(Ks, axis=1), np.concatenate(Vs, axis=1))
        self.score_evict(Qs[-1])
        self.quant_pack()
        K, V = self.keys_dequantized(), self.values_dequantized()
        total = sum(q.shape[1] for q in Qs)
        end = self.T - total
        outs = []
        for q in Qs:
            end += q.shape[1]
            O = attention(q, K[:, :end], V[:, :end], scale)
            outs.append(np.ascontiguousarray(np.transpose(O, (1, 0, 2))))
        return outs

    # ---- export for bit-exact comparison ----------------------------------
    def export(self) -> dict:
        """Logical-order arrays in the storage formats of the library."""
        p = self.p
        out = {"T": int(self.origin.shape[0]), "T_first": int(self.T_first),
               "origin": self.origin.copy()}
        if p.kv_bits == 16:
            out["k_val"] = self.k_val.copy()
            out["v_val"] = self.v_val.copy()
        else:
            pack = pack_nibbles if p.kv_bits == 4 else pack_bytes8
            out["k_packed"] = pack(self.k_codes)
            out["v_packed"] = pack(self.v_codes)
            if p.key_mode == "once":
                out["k_s_tok"], out["k_z_tok"] = self.key_params_per_token()
                out["k_groups_live"] = len(self.k_table)
            else:
                out["k_s_first"], out["k_z_first"] = self.k_s_first.copy(), self.k_z_first.copy()
                out["k_s_rest"], out["k_z_rest"] = self.k_s_rest.copy(), self.k_z_rest.copy()
            out["v_s"], out["v_z"] = self.v_s.copy(), self.v_z.copy()
        return out
