"""GPU parity at the full workload sizes, in the launch configuration the benchmark times.

One layer of the full-stack workload (1374 tokens per frame, budget 16384, INT4) and of the
long-stream workload (1004 tokens per frame) is streamed until the cache is full and evicting.
After every frame the whole packed state (origins, codes, scales, zero-points) is compared bit
for bit with the oracle; scores and kept indices are compared on every evicting frame; the
attention output is compared on sampled query rows (rows are independent, so the oracle
evaluates only those) within the usual tolerance.
"""
import numpy as np
import pytest

from oracle import xkv_oracle as xo
from paper_2601_01204_b200 import synth
from xkv_testlib import (ATTN_MAXABS, ATTN_RELL2, bf16_tensor_to_f32, compare_state, oracle_params,
                         to_device_bf16)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def xkv():
    import torch
    assert torch.cuda.is_available()
    import paper_2601_01204_b200.xkv as m
    return m


def _stream(xkv, n, budget, frames, seed, attn_from, bits=4):
    import torch
    H, d = 16, 64
    p = xkv.Params(n_heads=H, head_dim=d, budget=budget, max_frame_tokens=n, kv_bits=bits)
    cache = xkv.Cache(p)
    ora = xo.OracleLayer(oracle_params(p))
    rng = np.random.default_rng(seed)
    evicting = 0
    for t in range(frames):
        qb, kb, vb = synth.gen_frame(seed, 0, t, H, n, d)
        qf, kf, vf = (synth.bf16_bits_to_f32(x) for x in (qb, kb, vb))
        q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        cache.kv_append(k, v)
        cache.kv_score_evict(q)
        ora.append(kf, vf)
        ora.score_evict(qf)
        info = cache.xkv_get_info()
        if ora.last_scores is not None and info.last_kept > 0:
            evicting += 1
            s = cache.xkv_debug_export(xkv.BUF_SCORES, info.last_prunable * 4).view(np.float32)
            assert np.array_equal(s.view(np.uint32), ora.last_scores.view(np.uint32)), f"frame {t}: scores"
            kept = cache.xkv_debug_export(xkv.BUF_KEPT, info.last_kept * 4).view(np.int32)
            assert np.array_equal(kept, ora.last_kept_mid), f"frame {t}: kept indices"
        cache.kv_quant_pack()
        ora.quant_pack()
        compare_state(cache.export(), ora.export(), f"frame {t}")
        out = torch.empty_like(q)
        cache.attn_packed_causal(q, out)
        if t >= attn_from:
            rows = np.sort(rng.choice(n, size=24, replace=False))
            rows[0], rows[-1] = 0, n - 1                      # first row of the first tile, last row of the ragged tile
            scale = 1.0 / np.sqrt(d)
            ref = xo.attention(qf[:, rows], ora.keys_dequantized(), ora.values_dequantized(), scale)   # [H][rows][d]
            got = bf16_tensor_to_f32(out)[:, rows]
            err = got.astype(np.float64) - ref
            assert np.abs(err).max() <= ATTN_MAXABS * np.abs(ref).max(), f"frame {t}"
            assert np.linalg.norm(err) <= ATTN_RELL2 * np.linalg.norm(ref), f"frame {t}"
            # the same frame once more with its own K, V unquantised (Eq. 1 read literally)
            cache.xkv_debug_rewind_attention()
            cache.attn_packed_causal_tail(q, k, v, out)
            Kt = np.concatenate([ora.keys_dequantized()[:, :ora.T - n], kf], axis=1)
            Vt = np.concatenate([ora.values_dequantized()[:, :ora.T - n], vf], axis=1)
            ref_t = xo.attention(qf[:, rows], Kt, Vt, scale)
            got_t = bf16_tensor_to_f32(out)[:, rows]
            err_t = got_t.astype(np.float64) - ref_t
            assert np.abs(err_t).max() <= ATTN_MAXABS * np.abs(ref_t).max(), f"frame {t} (tail)"
            assert np.linalg.norm(err_t) <= ATTN_RELL2 * np.linalg.norm(ref_t), f"frame {t} (tail)"
            if bits == 4:   # and it is that reading, not the packed one
                assert np.linalg.norm(err_t) < 0.5 * np.linalg.norm(got_t.astype(np.float64) - ref), f"frame {t}"
        assert cache.xkv_poll_status() == 0
    return cache, evicting


def test_full_stack_layer_1374_tokens_budget_16384(xkv):
    cache, evicting = _stream(xkv, 1374, 16384, 14, seed=3, attn_from=11)
    info = cache.xkv_get_info()
    assert info.T == 16384 and evicting >= 2 and info.last_evicted == 1374


def test_long_stream_layer_1004_tokens_budget_16384(xkv):
    cache, evicting = _stream(xkv, 1004, 16384, 18, seed=4, attn_from=16)
    assert cache.xkv_get_info().T == 16384 and evicting >= 1


def test_single_layer_1374_tokens_budget_8192(xkv):
    cache, evicting = _stream(xkv, 1374, 8192, 8, seed=2, attn_from=5)
    assert cache.xkv_get_info().T == 8192 and evicting >= 2


def test_prune_only_16bit_budget_4096(xkv):
    cache, evicting = _stream(xkv, 1374, 4096, 5, seed=5, attn_from=2, bits=16)
    assert cache.xkv_get_info().T == 4096 and evicting >= 2


def test_workspace_is_the_only_memory_and_stays_flat(xkv):
    """The library allocates nothing: device memory in use does not move over a stream."""
    import torch
    H, n, d = 16, 1004, 64
    p = xkv.Params(budget=4096, max_frame_tokens=n)
    cache = xkv.Cache(p)
    q = torch.empty(H, n, d, dtype=torch.bfloat16, device="cuda")
    k, v, out = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for t in range(40):
        xkv.xkv_synth_fill(q, 9, 0, t, synth.TENSOR_Q)
        xkv.xkv_synth_fill(k, 9, 0, t, synth.TENSOR_K)
        xkv.xkv_synth_fill(v, 9, 0, t, synth.TENSOR_V)
        cache.step(q, k, v, out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    info = cache.xkv_get_info()
    assert info.T == 4096 and info.workspace_bytes == xkv.xkv_workspace_bytes(p)
