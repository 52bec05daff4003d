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


def _stream(xkv, n, budget, frames, seed, attn_from, bits=4, layer=0, via_stream_step=False, key_mode=0):
    """One layer's cache against the oracle.  via_stream_step: the frame goes through
    xkv_stream_step (scores and kept indices are read back after the step) instead of the four
    per-layer calls."""
    import torch
    H, d = 16, 64
    p = xkv.Params(n_heads=H, head_dim=d, budget=budget, max_frame_tokens=n, kv_bits=bits, key_mode=key_mode)
    cache = xkv.Cache(p)
    ora = xo.OracleLayer(oracle_params(p))
    rng = np.random.default_rng(seed)
    evicting = 0
    for t in range(frames):
        qb, kb, vb = synth.gen_frame(seed, layer, t, H, n, d)
        qf, kf, vf = (synth.bf16_bits_to_f32(x) for x in (qb, kb, vb))
        q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        out = torch.empty_like(q)
        ora.append(kf, vf)
        ora.score_evict(qf)
        if via_stream_step:
            xkv.xkv_stream_step([cache], [q], [k], [v], [out])
        else:
            cache.kv_append(k, v)
            cache.kv_score_evict(q)
        info = cache.xkv_get_info()
        if ora.last_scores is not None and info.last_kept > 0:
            evicting += 1
            s = cache.xkv_debug_export(xkv.BUF_SCORES, info.last_prunable * 4).view(np.float32)
            assert np.array_equal(s.view(np.uint32), ora.last_scores.view(np.uint32)), f"frame {t}: scores"
            kept = cache.xkv_debug_export(xkv.BUF_KEPT, info.last_kept * 4).view(np.int32)
            assert np.array_equal(kept, ora.last_kept_mid), f"frame {t}: kept indices"
        if not via_stream_step:
            cache.kv_quant_pack()
        ora.quant_pack()
        compare_state(cache.export(), ora.export(), f"frame {t}")
        if not via_stream_step:
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
            if bits != 8:       # (the unquantised tail is built for 4-bit and 16-bit caches)
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


def test_full_stack_layer_keys_quantised_once(xkv):
    """The full-stack workload's layer 0 with XKV_KEYS_ONCE, through xkv_stream_step."""
    cache, evicting = _stream(xkv, 1374, 16384, 15, seed=3, attn_from=12, via_stream_step=True, key_mode=1)
    info = cache.xkv_get_info()
    assert info.T == 16384 and evicting >= 3 and info.last_evicted == 1374


def test_full_stack_layer_8bit_keys_quantised_once(xkv):
    """The same layer with 8-bit codes (beyond the paper's INT4), quantise-once mode."""
    cache, evicting = _stream(xkv, 1374, 16384, 14, seed=3, attn_from=12, via_stream_step=True, key_mode=1, bits=8)
    assert cache.xkv_get_info().T == 16384 and evicting >= 2


def test_full_stack_last_layer_through_stream_step(xkv):
    """The full-stack workload seeds every layer on its own (seed 3 + layer, the layer's own
    outlier channels): layer 23, through xkv_stream_step."""
    cache, evicting = _stream(xkv, 1374, 16384, 14, seed=3 + 23, attn_from=12, layer=23, via_stream_step=True)
    info = cache.xkv_get_info()
    assert info.T == 16384 and evicting >= 2 and info.last_evicted == 1374


def test_single_layer_1374_tokens_budget_8192_all_32_frames(xkv):
    """The single-layer workload at its full length: 32 frames, 27 of them evicting."""
    cache, evicting = _stream(xkv, 1374, 8192, 32, seed=2, attn_from=29)
    assert cache.xkv_get_info().T == 8192 and evicting >= 26


def test_ablation_budget_4096_int4(xkv):
    cache, evicting = _stream(xkv, 1374, 4096, 6, seed=5, attn_from=3)
    assert cache.xkv_get_info().T == 4096 and evicting >= 3


def test_prune_only_16bit_budget_8192(xkv):
    cache, evicting = _stream(xkv, 1374, 8192, 8, seed=5, attn_from=6, bits=16)
    assert cache.xkv_get_info().T == 8192 and evicting >= 2


def test_prune_only_16bit_budget_16384(xkv):
    cache, evicting = _stream(xkv, 1374, 16384, 14, seed=5, attn_from=12, bits=16)
    assert cache.xkv_get_info().T == 16384 and evicting >= 2


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


def test_long_stream_1000_frames_24_layers(xkv):
    """The long-stream workload at its full length: 24 layers, 1004 tokens per frame, 1000 frames,
    budget 16384, INT4, through xkv_stream_step.  The oracle cannot follow that far (seconds per
    layer-step); checked here: device memory in use does not move after the caches are created,
    every cache sits at the budget, no kernel reported an error, the outputs are finite, and the
    survivors of every layer are the whole first frame, an increasing selection of later frames and
    the whole last frame, in arrival order.  An uncompressed bf16 cache would hold
    1000 x 1004 x 16 x 64 x 2 x 2 B x 24 layers = 98.7 GB by then."""
    import torch
    L, H, n, d, frames = 24, 16, 1004, 64, 1000
    p = xkv.Params(n_heads=H, budget=16384, max_frame_tokens=n, kv_bits=4)
    caches = [xkv.Cache(p) for _ in range(L)]
    q = [torch.empty(H, n, d, dtype=torch.bfloat16, device="cuda") for _ in range(L)]
    k = [torch.empty_like(x) for x in q]
    v = [torch.empty_like(x) for x in q]
    out = [torch.empty_like(x) for x in q]
    pool = 6          # distinct frames per layer, generated once and cycled (their content is arbitrary here)
    bank = []
    for f in range(pool):
        fr = []
        for l in range(L):
            t3 = [torch.empty(H, n, d, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
            for x, which in zip(t3, (synth.TENSOR_Q, synth.TENSOR_K, synth.TENSOR_V)):
                xkv.xkv_synth_fill(x, 4 + l, l, f, which)
            fr.append(t3)
        bank.append(fr)
    xkv.xkv_stream_step(caches, [b[0] for b in bank[0]], [b[1] for b in bank[0]], [b[2] for b in bank[0]], out)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held = sum(xkv.xkv_workspace_bytes(p) for _ in range(L))
    for t in range(1, frames):
        fr = bank[t % pool]
        xkv.xkv_stream_step(caches, [b[0] for b in fr], [b[1] for b in fr], [b[2] for b in fr], out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert held < 2.5e9 < 98.7e9                      # about 1.9 GB of workspaces for the whole stack
    for l, c in enumerate(caches):
        info = c.xkv_get_info()
        assert info.T == 16384 and info.frames == frames and c.xkv_poll_status() == 0, l
        assert bool(torch.isfinite(out[l].float()).all()), l
    for l in (0, 11, 23):
        info = caches[l].xkv_get_info()
        org = caches[l].xkv_debug_export(xkv.BUF_ORIGIN, info.capacity * 4).view(np.int32)
        sl = np.concatenate([np.arange(info.T_first), info.rest_base + np.arange(info.T - info.T_first)])
        org = org[sl].astype(np.int64)
        assert np.all(np.diff(org) > 0), l                                   # arrival order, no duplicates
        assert np.array_equal(org[:n], (1 << 16) | np.arange(n)), l          # the first frame, whole
        assert np.array_equal(org[-n:], (frames << 16) | np.arange(n)), l    # the newest frame, whole
        mid = org[n:-n] >> 16
        assert mid.min() >= 2 and mid.max() <= frames - 1, l


def test_ablation_budget_32768_int4(xkv):
    """The largest budget of the ablation sweep: 1374 tokens per frame, budget 32768 (257 key tiles,
    every item of the attention is cut into three or four pieces), first evicting frame 24."""
    cache, evicting = _stream(xkv, 1374, 32768, 26, seed=5, attn_from=24)
    assert cache.xkv_get_info().T == 32768 and evicting >= 2


@pytest.mark.parametrize("variant", ["int4", "int4-tail", "bf16", "int4-once", "int8-once", "int4-20-blocks"])
def test_attention_repeated_launches_are_bit_identical(xkv, variant):
    """The attention kernel passes tensor-memory buffers between its warps through barriers (one score
    buffer serves both query tiles in turn, P has two buffers per tile).  A protocol error there is a
    race: it shows as launches on the same inputs that differ.  Full-size layer (1374 tokens, budget
    16384, cache full and evicting), 12 launches per variant, outputs compared bit for bit."""
    import torch
    H, n, d = 16, 1374, 64
    bits = 16 if variant == "bf16" else (8 if variant == "int8-once" else 4)
    once = variant.endswith("once")
    p = xkv.Params(n_heads=H, budget=16384, max_frame_tokens=n, kv_bits=bits, key_mode=xkv.KEYS_ONCE if once else 0)
    cache = xkv.Cache(p)
    if variant == "int4-20-blocks":
        cache.xkv_debug_limit_attention_blocks(20)
    q = torch.empty(H, n, d, dtype=torch.bfloat16, device="cuda")
    k, v, out = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    for t in range(14):
        for x, w in ((q, 0), (k, 1), (v, 2)):
            xkv.xkv_synth_fill(x, 5, 0, t, w)
        cache.step(q, k, v, out)
    first = None
    for rep in range(12):
        cache.xkv_debug_rewind_attention()
        out.zero_()
        if variant == "int4-tail":
            cache.attn_packed_causal_tail(q, k, v, out)
        else:
            cache.attn_packed_causal(q, out)
        torch.cuda.synchronize()
        assert cache.xkv_poll_status() == 0
        bits_out = out.view(torch.int16).clone()
        if first is None:
            first = bits_out
            assert bool(torch.isfinite(out.float()).all())
        else:
            assert torch.equal(first, bits_out), f"{variant}: launch {rep} differs from launch 0"
    cache.close()
