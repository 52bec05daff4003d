"""Shared helpers of the GPU parity tests: drive the CUDA library and the oracle
with the same seeded frames and compare."""
from __future__ import annotations

import numpy as np

from oracle import xkv_oracle as xo
from paper_2601_01204_b200 import synth

ATTN_MAXABS = 1e-2      # max |err| <= 1e-2 * max |ref|
ATTN_RELL2 = 5e-3       # ||err||_2 <= 5e-3 * ||ref||_2


def to_device_bf16(bits: np.ndarray):
    import torch
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).cuda()


def bf16_tensor_to_f32(t) -> np.ndarray:
    import torch
    return t.detach().to(torch.float32).cpu().numpy()


def oracle_params(p) -> xo.OracleParams:
    return xo.OracleParams(n_heads=p.n_heads, head_dim=p.head_dim, n_special=p.n_special, pool_g=p.pool_g,
                           quant_group=p.quant_group, kv_bits=p.kv_bits, budget=p.budget,
                           key_mode="once" if getattr(p, "key_mode", 0) == 1 else "regroup")


def compare_state(gpu: dict, ora: dict, tag: str = "") -> None:
    assert gpu["T"] == ora["T"] and gpu["T_first"] == ora["T_first"], tag
    for key in ora:
        if key in ("T", "T_first"):
            continue
        a, b = np.asarray(gpu[key]), np.asarray(ora[key])
        assert a.shape == b.shape, (tag, key, a.shape, b.shape)
        if a.dtype.kind == "f":
            same = np.array_equal(a.view(np.uint32), b.view(np.uint32))
        else:
            same = np.array_equal(a, b)
        if not same:
            bad = np.argwhere(a != b)
            raise AssertionError(f"{tag}: {key} differs at {len(bad)} places, first {bad[:5].tolist()}: "
                                 f"gpu {a[tuple(bad[0])]} oracle {b[tuple(bad[0])]}")


def attn_errors(got: np.ndarray, ref: np.ndarray) -> tuple[float, float]:
    err = got.astype(np.float64) - ref.astype(np.float64)
    return float(np.abs(err).max() / np.abs(ref).max()), float(np.linalg.norm(err) / np.linalg.norm(ref))


def check_attention(got: np.ndarray, ref: np.ndarray, tag: str = "") -> None:
    maxabs, rell2 = attn_errors(got, ref)
    assert maxabs <= ATTN_MAXABS and rell2 <= ATTN_RELL2, f"{tag}: max-abs {maxabs:.3e}, rel-L2 {rell2:.3e}"


def run_stream(xkv, p, n_tokens, n_frames, seed, impl=0, layer=0, token_major=False, check_attn_every=1,
               tail=False, force_plain=False, max_blocks=0):
    """Stream n_frames through one GPU cache and one oracle layer, comparing after every call."""
    import torch
    cache = xkv.Cache(p)
    if force_plain:
        cache.xkv_debug_force_plain(True)
    if max_blocks:
        cache.xkv_debug_limit_attention_blocks(max_blocks)
    ora = xo.OracleLayer(oracle_params(p))
    n_list = n_tokens if isinstance(n_tokens, (list, tuple)) else [n_tokens] * n_frames
    H, d = p.n_heads, p.head_dim
    worst = (0.0, 0.0)
    for t, n in enumerate(n_list):
        qb, kb, vb = synth.gen_frame(seed, layer, t, H, n, d)
        qf, kf, vf = (synth.bf16_bits_to_f32(x) for x in (qb, kb, vb))
        if token_major:    # [n][H*d] storage viewed as [H][n][d]
            q, k, v = (to_device_bf16(np.ascontiguousarray(x.transpose(1, 0, 2))).permute(1, 0, 2) for x in (qb, kb, vb))
        else:
            q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        cache.kv_append(k, v)
        cache.kv_score_evict(q)
        ora.append(kf, vf)
        ora.score_evict(qf)
        info = cache.xkv_get_info()
        if ora.last_scores is not None and info.last_kept > 0:
            w = cache.xkv_debug_export(xkv.BUF_QVEC, 64 * 4).view(np.float32)
            assert np.array_equal(w.view(np.uint32), ora.last_w.view(np.uint32)), f"frame {t}: query vector"
            s = cache.xkv_debug_export(xkv.BUF_SCORES, info.last_prunable * 4).view(np.float32)
            assert np.array_equal(s.view(np.uint32), ora.last_scores.view(np.uint32)), f"frame {t}: scores"
            kept = cache.xkv_debug_export(xkv.BUF_KEPT, info.last_kept * 4).view(np.int32)
            assert np.array_equal(kept, ora.last_kept_mid), f"frame {t}: kept indices"
        cache.kv_quant_pack()
        ora.quant_pack()
        compare_state(cache.export(), ora.export(), f"frame {t}")
        out = torch.empty_like(q)
        if tail:      # the frame's own K, V unquantised (attn_packed_causal_tail)
            cache.attn_packed_causal_tail(q, k, v, out)
        else:
            cache.attn_packed_causal(q, out, impl=impl)
        if t % check_attn_every == 0 or t == len(n_list) - 1:
            ref = ora.attend(qf, full_precision_tail=tail)         # [n][H][d]
            got = bf16_tensor_to_f32(out).transpose(1, 0, 2)
            check_attention(got, ref, f"frame {t}")
            e = attn_errors(got, ref)
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        assert cache.xkv_poll_status() == 0
    return cache, ora, worst
