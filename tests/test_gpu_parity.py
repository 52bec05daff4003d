"""GPU parity: the CUDA library against the CPU oracle on the same seeded frames.

Integer results (kept indices, 4-bit codes, origins) and the fp32 quantities
that decide them (query vector, scores, scales, zero-points) must match bit for
bit; attention outputs within max-abs 1e-2 * max|ref| and relative L2 5e-3.
"""
import numpy as np
import pytest

from paper_2601_01204_b200 import synth
from xkv_testlib import run_stream, to_device_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def xkv():
    import torch
    assert torch.cuda.is_available()
    import paper_2601_01204_b200.xkv as m
    return m


@pytest.mark.parametrize("impl", [0, 1])
def test_tiny_stream_4bit(xkv, impl):
    """Config 1: 1 layer, 16 x 64, 261 tokens/frame, 8 frames, budget 1024, 4-bit."""
    p = xkv.Params(budget=1024, max_frame_tokens=261, kv_bits=4)
    cache, ora, worst = run_stream(xkv, p, 261, 8, seed=1, impl=impl)
    info = cache.xkv_get_info()
    assert info.T == 1024 and info.frames == 8 and info.last_evicted == 261
    print("tiny 4-bit impl", impl, "worst (max-abs, rel-L2)", worst)


def test_tiny_stream_4bit_plain_arithmetic_forms(xkv):
    """The maintenance kernels dequantise and quantise without conversion instructions when the
    zero-points and scaled values are small enough, and fall back to the plain forms otherwise.
    xkv_debug_force_plain sends every kernel of the cache down the fallback: both must give the
    oracle's bits."""
    p = xkv.Params(budget=1024, max_frame_tokens=261, kv_bits=4)
    cache, ora, worst = run_stream(xkv, p, 261, 7, seed=11, force_plain=True)
    assert cache.xkv_get_info().T == 1024


def test_large_offset_keys(xkv):
    """Keys with a large common offset on every channel: zero-points of a few thousand and |x / s|
    far from 0.  The packed state must be bit-exact.  Keys near 100 with a spread of 0.05 lose that
    spread in any 16-bit operand (spacing 0.06), so the attention check of this case uses the fp32
    CUDA-core kernel."""
    from xkv_testlib import compare_state, oracle_params, bf16_tensor_to_f32, check_attention
    from oracle import xkv_oracle as xo
    p = xkv.Params(n_heads=4, budget=400, max_frame_tokens=128, kv_bits=4)
    cache, ora = xkv.Cache(p), xo.OracleLayer(oracle_params(p))
    H, n, d = 4, 128, 64
    for t in range(6):
        qb, kb, vb = synth.gen_frame(12, 0, t, H, n, d)
        kf = synth.bf16_bits_to_f32(kb) * np.float32(0.05) + np.float32(100.0)
        kb = synth.f32_to_bf16_bits(kf)
        qf, kf, vf = (synth.bf16_bits_to_f32(x) for x in (qb, kb, vb))
        q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        cache.kv_append(k, v); cache.kv_score_evict(q); cache.kv_quant_pack()
        ora.append(kf, vf); ora.score_evict(qf); ora.quant_pack()
        compare_state(cache.export(), ora.export(), f"frame {t}")
        out = cache.attn_packed_causal(q, impl=1)
        check_attention(bf16_tensor_to_f32(out).transpose(1, 0, 2), ora.attend(qf), f"frame {t}")
    assert cache.xkv_get_info().T == 400


def _offset_channel_frame(t, H, n, d):
    """Ordinary keys except four channels per head that sit at +254 / -255 and move by one step:
    the channel-wise key outliers of Fig. 3 in their hardest form for Eq. 8, zero-points of -3810
    and +3825.  Every seventh token has a value row of range 1e-4 (scale 7e-6)."""
    qb, kb, vb = synth.gen_frame(12, 0, t, H, n, d)
    kf, vf = synth.bf16_bits_to_f32(kb).copy(), synth.bf16_bits_to_f32(vb).copy()
    bit = (synth.gen_tensor_bits(99, 0, t, synth.TENSOR_Q, H, n, d) & 1).astype(np.float32)
    for c, base in ((3, 254.0), (17, 254.0), (40, -255.0), (63, -255.0)):
        kf[:, :, c] = base + bit[:, :, c]
    vf[:, ::7, :] *= np.float32(1e-5)
    return qb, synth.f32_to_bf16_bits(kf), synth.f32_to_bf16_bits(vf)


@pytest.mark.parametrize("tail", [False, True])
def test_offset_channels_through_the_tensor_core_kernel(xkv, tail):
    """Zero-points in the thousands and tiny value scales through impl = 0: the fp16 operand path
    forms s * q + (-s z) with the constant taken in fp32, which holds for any integer zero-point
    (Eq. 10).  State bit-exact, attention within the usual tolerance, no status raised."""
    from xkv_testlib import compare_state, oracle_params, bf16_tensor_to_f32, check_attention
    from oracle import xkv_oracle as xo
    H, n, d = 4, 128, 64
    p = xkv.Params(n_heads=H, budget=400, max_frame_tokens=n, kv_bits=4)
    cache, ora = xkv.Cache(p), xo.OracleLayer(oracle_params(p))
    zmax = 0.0
    for t in range(6):
        qb, kb, vb = _offset_channel_frame(t, H, n, d)
        qf, kf, vf = (synth.bf16_bits_to_f32(x) for x in (qb, kb, vb))
        q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        cache.kv_append(k, v); cache.kv_score_evict(q); cache.kv_quant_pack()
        ora.append(kf, vf); ora.score_evict(qf); ora.quant_pack()
        compare_state(cache.export(), ora.export(), f"frame {t}")
        out = cache.attn_packed_causal_tail(q, k, v) if tail else cache.attn_packed_causal(q, impl=0)
        check_attention(bf16_tensor_to_f32(out).transpose(1, 0, 2), ora.attend(qf, full_precision_tail=tail), f"frame {t}")
        assert cache.xkv_poll_status() == 0
        zmax = max(zmax, float(np.abs(ora.k_z_first).max()), float(np.abs(ora.k_z_rest).max()) if ora.T > n else 0.0)
    assert zmax > 3000 and float(ora.v_s.min()) < 2e-5


def test_values_beyond_fp16_are_reported_not_silent(xkv):
    """Magnitudes above 65504 cannot be tensor-core operands of a 4-bit cache: the call records
    XKV_E_RANGE in the status word (queries, dequantised keys, raw tail rows), the fp32 kernel and a
    16-bit cache take the same inputs without complaint, and xkv_reset clears the word."""
    import torch
    H, n, d = 2, 64, 64
    qb, kb, vb = synth.gen_frame(14, 0, 0, H, n, d)
    q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
    big_k = k.clone(); big_k[1, 5, 9] = 1.0e5
    big_q = q.clone(); big_q[0, 3, 2] = -7.0e4
    p = xkv.Params(n_heads=H, budget=256, max_frame_tokens=n, kv_bits=4)
    cache = xkv.Cache(p)
    for qq, kk, use_tail, want in ((q, k, False, 0), (q, big_k, False, xkv.XKV_E_RANGE), (big_q, k, False, xkv.XKV_E_RANGE),
                                   (q, big_k, True, xkv.XKV_E_RANGE)):
        cache.xkv_reset()
        cache.kv_append(kk, v); cache.kv_score_evict(qq); cache.kv_quant_pack()
        if use_tail:
            cache.attn_packed_causal_tail(qq, kk, v)
        else:
            cache.attn_packed_causal(qq, impl=0)
        assert cache.xkv_poll_status() == want
    # the fp32 kernel has no such limit
    cache.xkv_reset()
    cache.kv_append(big_k, v); cache.kv_score_evict(q); cache.kv_quant_pack()
    out = cache.attn_packed_causal(q, impl=1)
    assert cache.xkv_poll_status() == 0 and bool(torch.isfinite(out.float()).all())
    # a 16-bit cache multiplies in bf16
    c16 = xkv.Cache(xkv.Params(n_heads=H, budget=256, max_frame_tokens=n, kv_bits=16))
    c16.kv_append(big_k, v); c16.kv_score_evict(big_q); c16.kv_quant_pack()
    out = c16.attn_packed_causal(big_q, impl=0)
    assert c16.xkv_poll_status() == 0 and bool(torch.isfinite(out.float()).all())


def test_bounded_wait_reports_timeout_and_the_context_survives(xkv):
    """Every wait inside the attention kernel is bounded.  The probe runs that wait on a barrier
    nothing completes: it gives up at its limit, the kernel ends, the status word reads
    XKV_E_TIMEOUT, and after xkv_reset the same cache streams a frame normally."""
    import torch
    H, n, d = 2, 64, 64
    p = xkv.Params(n_heads=H, budget=256, max_frame_tokens=n, kv_bits=4)
    cache = xkv.Cache(p)
    assert cache.xkv_poll_status() == 0
    cache.xkv_debug_timeout_probe()
    assert cache.xkv_poll_status() == xkv.XKV_E_TIMEOUT
    assert xkv.lib.xkv_strerror(xkv.XKV_E_TIMEOUT) == b"bounded device-side wait ran out"
    cache.xkv_reset()
    assert cache.xkv_poll_status() == 0
    cache2, ora, _ = run_stream(xkv, p, n, 3, seed=8)
    q, k, v = (to_device_bf16(x) for x in synth.gen_frame(8, 0, 0, H, n, d))
    out = cache.step(q, k, v)
    assert cache.xkv_poll_status() == 0 and bool(torch.isfinite(out.float()).all())


@pytest.mark.parametrize("blocks", [1, 5, 20])
def test_attention_with_fewer_blocks_than_multiprocessors(xkv, blocks):
    """The attention cuts its line of (item, key tile) steps into one piece per thread block.  With
    the block count capped a piece spans several items and an item few pieces: same result."""
    p = xkv.Params(n_heads=6, budget=900, max_frame_tokens=300, kv_bits=4)
    run_stream(xkv, p, 300, 5, seed=16, max_blocks=blocks)
    p = xkv.Params(n_heads=3, budget=600, max_frame_tokens=200, kv_bits=16)
    run_stream(xkv, p, 200, 4, seed=17, max_blocks=blocks, tail=False)


@pytest.mark.parametrize("impl", [0, 1])
def test_tiny_stream_16bit(xkv, impl):
    p = xkv.Params(budget=1024, max_frame_tokens=261, kv_bits=16)
    cache, ora, worst = run_stream(xkv, p, 261, 8, seed=2, impl=impl)
    assert cache.xkv_get_info().T == 1024
    print("tiny 16-bit impl", impl, "worst", worst)


@pytest.mark.parametrize("bits", [4, 16])
def test_token_major_layout(xkv, bits):
    """[n][H*d] storage (tok_stride = H*d, head_stride = d)."""
    p = xkv.Params(budget=600, max_frame_tokens=200, kv_bits=bits)
    run_stream(xkv, p, 197, 5, seed=3, token_major=True)


def test_budget_below_first_plus_current(xkv):
    """k = max(0, L_max - T_first - n) = 0: the cache is first + current frame."""
    p = xkv.Params(budget=300, max_frame_tokens=261, kv_bits=4)
    cache, ora, _ = run_stream(xkv, p, 261, 4, seed=4)
    assert cache.xkv_get_info().T == 522


def test_ragged_frame_sizes_and_small_heads(xkv):
    """Frame sizes that leave partial pooling groups and partial key groups; H = 3."""
    p = xkv.Params(n_heads=3, budget=500, max_frame_tokens=150, kv_bits=4, pool_g=7, n_special=2)
    run_stream(xkv, p, [129, 64, 150, 5, 77, 150, 33, 128], 8, seed=5)


def test_single_token_frames_and_exact_budget(xkv):
    p = xkv.Params(n_heads=2, budget=256, max_frame_tokens=128, kv_bits=4, n_special=1, pool_g=16)
    run_stream(xkv, p, [128, 128, 1, 128, 64], 5, seed=6)


def test_score_ties_are_broken_by_position(xkv):
    """All-zero queries give all-equal scores (+0): the lowest positions must survive."""
    import torch
    p = xkv.Params(n_heads=2, budget=200, max_frame_tokens=64, kv_bits=4)
    cache = xkv.Cache(p)
    H, n, d = 2, 64, 64
    for t in range(5):
        _, kb, vb = synth.gen_frame(7, 0, t, H, n, d)
        q = torch.zeros(H, n, d, dtype=torch.bfloat16, device="cuda")
        cache.step(q, to_device_bf16(kb), to_device_bf16(vb))
        info = cache.xkv_get_info()
        if info.last_evicted:
            kept = cache.xkv_debug_export(xkv.BUF_KEPT, info.last_kept * 4).view(np.int32)
            assert np.array_equal(kept, np.arange(info.last_kept))
    assert cache.xkv_get_info().T == 200


def test_state_machine_and_argument_errors(xkv):
    import torch
    p = xkv.Params(budget=512, max_frame_tokens=100)
    cache = xkv.Cache(p)
    q = torch.zeros(16, 100, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(xkv.XkvError) as e:
        cache.kv_quant_pack()
    assert e.value.status == xkv.XKV_E_STATE
    with pytest.raises(xkv.XkvError) as e:
        cache.attn_packed_causal(q)
    assert e.value.status == xkv.XKV_E_STATE
    big = torch.zeros(16, 101, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(xkv.XkvError) as e:
        cache.kv_append(big, big)
    assert e.value.status == xkv.XKV_E_INVALID
    cache.kv_append(q, q)
    with pytest.raises(xkv.XkvError) as e:
        cache.kv_append(q, q)
    assert e.value.status == xkv.XKV_E_STATE
    with pytest.raises(xkv.XkvError) as e:
        cache.kv_score_evict(big)              # more tokens than were appended (fewer is the last frame of a chunk)
    assert e.value.status == xkv.XKV_E_INVALID
    cache.kv_score_evict(q)
    cache.kv_quant_pack()
    cache.attn_packed_causal(q)
    assert cache.xkv_get_info().stage == 0
    cache.xkv_reset()
    assert cache.xkv_get_info().T == 0
    # too-small workspace is refused before anything is launched
    import ctypes as C
    h = C.c_void_p()
    rc = xkv.lib.xkv_create(C.byref(p.c()), cache.workspace.data_ptr(), 1024, 0, C.byref(h))
    assert rc == xkv.XKV_E_NOMEM


def test_synth_kernel_matches_numpy_generator(xkv):
    import torch
    H, n, d = 16, 261, 64
    for tensor in (synth.TENSOR_Q, synth.TENSOR_K, synth.TENSOR_V):
        dst = torch.empty(H, n, d, dtype=torch.bfloat16, device="cuda")
        xkv.xkv_synth_fill(dst, 9, 2, 5, tensor)
        got = dst.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got, synth.gen_tensor_bits(9, 2, 5, tensor, H, n, d))


@pytest.mark.parametrize("bits", [4, 16])
def test_stream_step_scoring_from_stored_head_means(xkv, bits):
    """The stream step computes the head means of the keys (Eq. 4) beside the attention and the next
    frame's scoring starts from them; the per-call sequence computes them inside the scoring.  Both
    must give the same bits: scores, kept indices, the whole packed state and the outputs, frame
    after frame, also across a reset."""
    import torch
    L, H, n, d = 2, 4, 150, 64
    p = xkv.Params(n_heads=H, budget=400, max_frame_tokens=n, kv_bits=bits)
    step_caches = [xkv.Cache(p) for _ in range(L)]
    call_caches = [xkv.Cache(p) for _ in range(L)]
    for rnd in range(2):
        for t in range(6):
            frames = [synth.gen_frame(51 + rnd, l, t, H, n, d) for l in range(L)]
            q, k, v = ([to_device_bf16(f[i]) for f in frames] for i in range(3))
            out = [torch.empty_like(x) for x in q]
            xkv.xkv_stream_step(step_caches, q, k, v, out)
            for l, c in enumerate(call_caches):
                c.kv_append(k[l], v[l]); c.kv_score_evict(q[l]); c.kv_quant_pack()
                ref = c.attn_packed_causal(q[l])
                torch.cuda.synchronize()
                assert torch.equal(out[l].view(torch.int16), ref.view(torch.int16)), (rnd, t, l)
                ia, ib = step_caches[l].xkv_get_info(), c.xkv_get_info()
                assert (ia.T, ia.last_kept, ia.last_evicted) == (ib.T, ib.last_kept, ib.last_evicted)
                if ib.last_evicted > 0:
                    for buf, nb in ((xkv.BUF_SCORES, ib.last_prunable * 4), (xkv.BUF_KEPT, ib.last_kept * 4)):
                        assert np.array_equal(step_caches[l].xkv_debug_export(buf, nb), c.xkv_debug_export(buf, nb)), (rnd, t, l)
                ea, eb = step_caches[l].export(), c.export()
                assert all(np.array_equal(np.asarray(ea[key]), np.asarray(eb[key])) for key in eb), (rnd, t, l)
        assert step_caches[0].xkv_get_info().last_evicted > 0
        for c in step_caches + call_caches:
            c.xkv_reset()


def test_stream_step_with_unquantised_tail_option(xkv):
    """xkv_set_unquantised_tail(1): the stream step gives what the per-call sequence with
    attn_packed_causal_tail gives, bit for bit."""
    import torch
    L, H, n, d = 2, 4, 180, 64
    p = xkv.Params(n_heads=H, budget=500, max_frame_tokens=n, kv_bits=4)
    step_caches = [xkv.Cache(p) for _ in range(L)]
    call_caches = [xkv.Cache(p) for _ in range(L)]
    for c in step_caches:
        c.xkv_set_unquantised_tail(True)
    for t in range(5):
        frames = [synth.gen_frame(41, l, t, H, n, d) for l in range(L)]
        q, k, v = ([to_device_bf16(f[i]) for f in frames] for i in range(3))
        out = [torch.empty_like(x) for x in q]
        xkv.xkv_stream_step(step_caches, q, k, v, out)
        for l, c in enumerate(call_caches):
            c.kv_append(k[l], v[l]); c.kv_score_evict(q[l]); c.kv_quant_pack()
            ref = c.attn_packed_causal_tail(q[l], k[l], v[l])
            torch.cuda.synchronize()
            assert torch.equal(out[l].view(torch.int16), ref.view(torch.int16)), (t, l)


def test_host_buffer_step_equals_device_step(xkv):
    """xkv_stream_step_host (inputs and outputs in pinned host memory, copies overlapped with the
    kernels on the library's own copy streams) gives the bits of xkv_stream_step on device
    tensors: three layers (so that both halves of the staging buffer are reused), frames past
    the point where eviction starts."""
    import torch
    L, H, n, d, budget = 3, 4, 200, 64, 512
    p = xkv.Params(n_heads=H, budget=budget, max_frame_tokens=n, kv_bits=4)
    dev_caches = [xkv.Cache(p) for _ in range(L)]
    host_caches = [xkv.Cache(p) for _ in range(L)]
    staging = torch.empty(xkv.xkv_stream_step_host_bytes(p, n), dtype=torch.uint8, device="cuda")
    for t in range(5):
        frames = [synth.gen_frame(21, l, t, H, n, d) for l in range(L)]
        dq, dk, dv = ([to_device_bf16(f[i]) for f in frames] for i in range(3))
        dout = [torch.empty_like(x) for x in dq]
        xkv.xkv_stream_step(dev_caches, dq, dk, dv, dout)
        hq, hk, hv = ([x.cpu().pin_memory() for x in xs] for xs in (dq, dk, dv))
        hout = [torch.empty_like(x).pin_memory() for x in hq]
        xkv.xkv_stream_step_host(host_caches, hq, hk, hv, hout, staging)
        torch.cuda.synchronize()
        for l in range(L):
            assert torch.equal(hout[l].view(torch.int16), dout[l].cpu().view(torch.int16)), (t, l)
    assert host_caches[0].xkv_get_info().last_evicted > 0


def test_unquantised_tail_streams(xkv):
    """attn_packed_causal_tail against the oracle's full_precision_tail reading: the tiny stream
    (first frame = all tail, eviction from frame 4), ragged frame sizes with small heads (tail start
    anywhere inside a key tile), token-major layout, a single-token frame, and a budget below
    first + current (cache = first frame + tail).  The packed state stays bit-exact throughout."""
    run_stream(xkv, xkv.Params(budget=1024, max_frame_tokens=261), 261, 8, seed=1, tail=True)
    run_stream(xkv, xkv.Params(n_heads=3, budget=500, max_frame_tokens=150, pool_g=7, n_special=2),
               [129, 64, 150, 5, 77, 150, 33, 128], 8, seed=5, tail=True)
    run_stream(xkv, xkv.Params(budget=700, max_frame_tokens=261), 261, 5, seed=6, token_major=True, tail=True)
    run_stream(xkv, xkv.Params(n_heads=2, budget=256, max_frame_tokens=128, n_special=1, pool_g=16),
               [128, 128, 1, 128, 64], 5, seed=6, tail=True)
    run_stream(xkv, xkv.Params(n_heads=4, budget=300, max_frame_tokens=200), 200, 4, seed=9, tail=True)


def test_unquantised_tail_on_16bit_cache_is_the_packed_result(xkv):
    import torch
    H, n, d = 4, 150, 64
    p = xkv.Params(n_heads=H, budget=400, max_frame_tokens=n, kv_bits=16)
    cache = xkv.Cache(p)
    for t in range(5):
        q, k, v = (to_device_bf16(x) for x in synth.gen_frame(31, 0, t, H, n, d))
        cache.kv_append(k, v); cache.kv_score_evict(q); cache.kv_quant_pack()
        a = cache.attn_packed_causal(q)
        cache.xkv_debug_rewind_attention()
        b = cache.attn_packed_causal_tail(q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(a.view(torch.int16), b.view(torch.int16)), t
    # argument check: the tail has to be the frame appended last
    q, k, v = (to_device_bf16(x) for x in synth.gen_frame(31, 0, 9, H, n, d))
    cache.kv_append(k, v); cache.kv_score_evict(q); cache.kv_quant_pack()
    o = torch.empty_like(q)
    with pytest.raises(xkv.XkvError):
        cache.attn_packed_causal_tail(q[:, :100], k[:, :100], v[:, :100], o[:, :100])
    cache.attn_packed_causal_tail(q, k, v)


# ------------------------------------------------------------------ keys quantised once
@pytest.mark.parametrize("impl", [0, 1])
def test_tiny_stream_keys_quantised_once(xkv, impl):
    """XKV_KEYS_ONCE on the tiny workload: a frame's keys are quantised on arrival in groups of 64 of
    its tokens, survivors keep codes and group parameters.  Codes, per-token parameters (through the
    table), the number of live groups, scores, kept indices: bit-exact; attention in tolerance."""
    p = xkv.Params(budget=1024, max_frame_tokens=261, kv_bits=4, key_mode=xkv.KEYS_ONCE)
    cache, ora, worst = run_stream(xkv, p, 261, 9, seed=1, impl=impl)
    info = cache.xkv_get_info()
    assert info.T == 1024 and info.last_evicted == 261 and info.key_table_slots == info.capacity
    print("tiny once impl", impl, "worst (max-abs, rel-L2)", worst)


def test_keys_quantised_once_ragged_tail_and_block_cap(xkv):
    """Ragged frame sizes (partial arrival groups, single-token frames), few heads, the unquantised
    tail reading, token-major tensors, and a capped attention grid, all with XKV_KEYS_ONCE."""
    p = xkv.Params(n_heads=3, budget=500, max_frame_tokens=150, kv_bits=4, pool_g=7, n_special=2, key_mode=xkv.KEYS_ONCE)
    run_stream(xkv, p, [129, 64, 150, 5, 77, 150, 33, 128, 150, 1, 150], 11, seed=5)
    run_stream(xkv, p, [129, 64, 150, 5, 77, 150, 33, 128], 8, seed=6, tail=True)
    p = xkv.Params(budget=700, max_frame_tokens=261, key_mode=xkv.KEYS_ONCE)
    run_stream(xkv, p, 261, 5, seed=7, token_major=True, max_blocks=7)
    p = xkv.Params(n_heads=2, budget=100, max_frame_tokens=64, key_mode=xkv.KEYS_ONCE)      # k = 0: first + current only
    run_stream(xkv, p, 64, 4, seed=8)


def test_keys_quantised_once_stream_step_and_reset(xkv):
    """xkv_stream_step (one maintenance launch per layer) against the per-call sequence, bit for bit,
    with XKV_KEYS_ONCE; then both again after xkv_reset (the table's free ring is rebuilt)."""
    import torch
    L, H, n, d = 2, 4, 150, 64
    p = xkv.Params(n_heads=H, budget=400, max_frame_tokens=n, kv_bits=4, key_mode=xkv.KEYS_ONCE)
    step_caches = [xkv.Cache(p) for _ in range(L)]
    call_caches = [xkv.Cache(p) for _ in range(L)]
    for rnd in range(2):
        for t in range(7):
            frames = [synth.gen_frame(61 + rnd, l, t, H, n, d) for l in range(L)]
            q, k, v = ([to_device_bf16(f[i]) for f in frames] for i in range(3))
            out = [torch.empty_like(x) for x in q]
            xkv.xkv_stream_step(step_caches, q, k, v, out)
            for l, c in enumerate(call_caches):
                c.kv_append(k[l], v[l]); c.kv_score_evict(q[l]); c.kv_quant_pack()
                ref = c.attn_packed_causal(q[l])
                torch.cuda.synchronize()
                assert torch.equal(out[l].view(torch.int16), ref.view(torch.int16)), (rnd, t, l)
                ea, eb = step_caches[l].export(), c.export()
                assert all(np.array_equal(np.asarray(ea[key]), np.asarray(eb[key])) for key in eb), (rnd, t, l)
                assert step_caches[l].xkv_poll_status() == 0 and c.xkv_poll_status() == 0
        assert step_caches[0].xkv_get_info().last_evicted > 0
        for c in step_caches + call_caches:
            c.xkv_reset()


def test_key_table_too_small_is_reported(xkv):
    """A parameter table sized below the worst case can run out (every survivor of an old frame may
    be the last of its group): the status word then reads XKV_E_LIMIT instead of anything silent."""
    H, n, d = 2, 64, 64
    p = xkv.Params(n_heads=H, budget=640, max_frame_tokens=n, kv_bits=4, key_mode=xkv.KEYS_ONCE, key_table_slots=3)
    cache = xkv.Cache(p)
    assert cache.xkv_get_info().key_table_slots == 3          # two frames' groups + 1 is the least the library accepts
    status = 0
    for t in range(6):                                         # no eviction before frame 10: a fourth live group appears at t = 3
        q, k, v = (to_device_bf16(x) for x in synth.gen_frame(71, 0, t, H, n, d))
        cache.step(q, k, v)
        status = cache.xkv_poll_status()
        if status:
            break
    assert status == xkv.XKV_E_LIMIT and t == 3
    assert xkv.lib.xkv_create is not None


# ------------------------------------------------------------------ budget changes, caller's w
@pytest.mark.parametrize("key_mode", [0, 1])
def test_budget_changes_query_vector_from_caller_and_score_statistics(xkv, key_mode):
    """xkv_set_budget lowers and restores the budget mid-stream (the cache shrinks to it at the next
    frame, bit-exact against the oracle's set_budget); kv_score_evict_w takes the pooled query's row
    mean from the caller and gives the state kv_score_evict gives; xkv_read_score_stats returns sum,
    sum of squares and the k-th largest of the scores S (Eq. 6)."""
    import torch
    from xkv_testlib import compare_state, oracle_params, bf16_tensor_to_f32, check_attention
    from oracle import xkv_oracle as xo
    H, n, d = 4, 100, 64
    p = xkv.Params(n_heads=H, budget=700, max_frame_tokens=n, kv_bits=4, key_mode=key_mode)
    ca, cb = xkv.Cache(p), xkv.Cache(p)
    ora = xo.OracleLayer(oracle_params(p))
    assert ca.xkv_read_score_stats().count == 0
    for t in range(12):
        if t == 6:
            for c in (ca, cb): c.xkv_set_budget(380)
            ora.set_budget(380)
        if t == 10:
            for c in (ca, cb): c.xkv_set_budget(700)
            ora.set_budget(700)
        qb, kb, vb = synth.gen_frame(81, 0, t, H, n, d)
        qf, kf, vf = (synth.bf16_bits_to_f32(x) for x in (qb, kb, vb))
        q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        ca.kv_append(k, v); ca.kv_score_evict(q); ca.kv_quant_pack()
        ora.append(kf, vf); ora.score_evict(qf); ora.quant_pack()
        compare_state(ca.export(), ora.export(), f"frame {t}")
        check_attention(bf16_tensor_to_f32(ca.attn_packed_causal(q)).transpose(1, 0, 2), ora.attend(qf), f"frame {t}")
        # the second cache gets w from "the producer of Q" (here: the oracle's canonical arithmetic)
        w = xo.query_vector_canonical(xo.pooled_query_canonical(qf, p.n_special, p.pool_g))
        cb.kv_append(k, v); cb.kv_score_evict_w(torch.from_numpy(w).cuda(), n); cb.kv_quant_pack()
        cb.attn_packed_causal(q)
        ea, eb = ca.export(), cb.export()
        assert all(np.array_equal(np.asarray(ea[key]), np.asarray(eb[key])) for key in ea), f"frame {t}: given w"
        if ora.last_scores is not None:
            st = ca.xkv_read_score_stats()
            S = ora.last_scores.astype(np.float64)
            assert st.count == len(S) and st.kept == len(ora.last_kept_mid)
            assert abs(st.sum - S.sum()) <= 1e-4 * np.abs(S).sum() and abs(st.sum_sq - (S * S).sum()) <= 1e-4 * (S * S).sum()
            assert np.float32(st.threshold) == np.sort(ora.last_scores)[::-1][st.kept - 1]
        info = ca.xkv_get_info()
        assert info.budget == (380 if 6 <= t < 10 else 700) and info.T == ora.T
    assert ca.xkv_get_info().T == 380 + 2 * n and ca.xkv_poll_status() == 0
    with pytest.raises(xkv.XkvError):
        ca.xkv_set_budget(701)


# ------------------------------------------------------------------ chunks of frames
@pytest.mark.parametrize("bits,key_mode", [(4, 0), (4, 1), (16, 0)])
def test_chunked_prefill_is_frame_causal(xkv, bits, key_mode):
    """xkv_prefill_chunk: several frames arrive together; the chunk is one arrival for the cache
    maintenance (scored with its last frame's query) and its attention is frame-causal (Eq. 1): frame
    f of the chunk sees the older cache and the chunk's frames 0..f.  Against the oracle's step_chunk:
    state bit-exact, every frame's output within tolerance; chunk sizes that put frame boundaries
    inside key tiles and query tiles, the first chunk being the first arrival, pruning active later."""
    import torch
    from xkv_testlib import compare_state, oracle_params, bf16_tensor_to_f32, check_attention
    from oracle import xkv_oracle as xo
    H, d = 4, 64
    p = xkv.Params(n_heads=H, budget=1100, max_frame_tokens=700, kv_bits=bits, key_mode=key_mode)
    cache, ora = xkv.Cache(p), xo.OracleLayer(oracle_params(p))
    chunks = [[150, 261], [261], [100, 200, 150, 37], [261, 261], [8, 136, 300]]
    t = 0
    for ci, chunk in enumerate(chunks):
        fr = [synth.gen_frame(91, 0, t + j, H, n, d) for j, n in enumerate(chunk)]
        t += len(chunk)
        qf, kf, vf = ([synth.bf16_bits_to_f32(f[i]) for f in fr] for i in range(3))
        q, k, v = (to_device_bf16(np.concatenate([f[i] for f in fr], axis=1)) for i in range(3))
        out = cache.xkv_prefill_chunk(q, k, v, chunk)
        refs = ora.step_chunk(qf, kf, vf)
        compare_state(cache.export(), ora.export(), f"chunk {ci}")
        got = bf16_tensor_to_f32(out).transpose(1, 0, 2)
        r0 = 0
        for f, n in enumerate(chunk):
            check_attention(got[r0:r0 + n], refs[f], f"chunk {ci} frame {f}")
            r0 += n
        assert cache.xkv_poll_status() == 0
    assert cache.xkv_get_info().T == 1100 and ora.last_scores is not None
    # the pieces by hand, and the argument checks
    fr = [synth.gen_frame(91, 0, t + j, H, n, d) for j, n in enumerate([64, 64])]
    q, k, v = (to_device_bf16(np.concatenate([f[i] for f in fr], axis=1)) for i in range(3))
    cache.kv_append(k, v); cache.kv_score_evict(q[:, 64:], ); cache.kv_quant_pack()
    with pytest.raises(xkv.XkvError):
        cache.attn_packed_frame_causal(q, [64, 32])              # sizes must add up to what was appended
    cache.attn_packed_frame_causal(q, [64, 64])
    assert cache.xkv_get_info().stage == 0


# ------------------------------------------------------------------ 8-bit codes
@pytest.mark.parametrize("impl", [0, 1])
def test_tiny_stream_8bit_keys_quantised_once(xkv, impl):
    """kv_bits = 8 (Eq. 7-8 with 256 levels; the paper evaluates INT4 only) through the quantise-once
    path: codes (bytes in the order c0, c2, c1, c3 per word), parameters through the table, scores,
    kept indices bit-exact; attention within the usual tolerance."""
    p = xkv.Params(budget=1024, max_frame_tokens=261, kv_bits=8, key_mode=xkv.KEYS_ONCE)
    cache, ora, worst = run_stream(xkv, p, 261, 9, seed=1, impl=impl)
    assert cache.xkv_get_info().T == 1024
    print("tiny 8-bit impl", impl, "worst (max-abs, rel-L2)", worst)
    # 8-bit codes are only built for the quantise-once mode
    import ctypes as C
    h = C.c_void_p()
    bad = xkv.Params(budget=1024, max_frame_tokens=261, kv_bits=8)
    assert xkv.lib.xkv_create(C.byref(bad.c()), cache.workspace.data_ptr(), 1 << 40, 0, C.byref(h)) == xkv.XKV_E_UNSUPPORTED


def test_8bit_ragged_frames_chunks_and_budget_changes(xkv):
    """8-bit codes with ragged frame sizes and few heads, a capped attention grid, a chunk of frames
    and a budget change."""
    import torch
    from xkv_testlib import compare_state, oracle_params, bf16_tensor_to_f32, check_attention
    from oracle import xkv_oracle as xo
    p = xkv.Params(n_heads=3, budget=500, max_frame_tokens=150, kv_bits=8, pool_g=7, n_special=2, key_mode=xkv.KEYS_ONCE)
    run_stream(xkv, p, [129, 64, 150, 5, 77, 150, 33, 128, 150, 1, 150], 11, seed=5, max_blocks=9)
    H, d = 4, 64
    p = xkv.Params(n_heads=H, budget=700, max_frame_tokens=400, kv_bits=8, key_mode=xkv.KEYS_ONCE)
    cache, ora = xkv.Cache(p), xo.OracleLayer(oracle_params(p))
    t = 0
    for ci, chunk in enumerate([[150, 200], [261], [100, 200, 37], [261], [261]]):
        if ci == 3:
            cache.xkv_set_budget(500); ora.set_budget(500)
        fr = [synth.gen_frame(93, 0, t + j, H, n, d) for j, n in enumerate(chunk)]
        t += len(chunk)
        qf, kf, vf = ([synth.bf16_bits_to_f32(f[i]) for f in fr] for i in range(3))
        q, k, v = (to_device_bf16(np.concatenate([f[i] for f in fr], axis=1)) for i in range(3))
        out = cache.xkv_prefill_chunk(q, k, v, chunk)
        refs = ora.step_chunk(qf, kf, vf)
        compare_state(cache.export(), ora.export(), f"chunk {ci}")
        got = bf16_tensor_to_f32(out).transpose(1, 0, 2)
        r0 = 0
        for f, n in enumerate(chunk):
            check_attention(got[r0:r0 + n], refs[f], f"chunk {ci} frame {f}")
            r0 += n
        assert cache.xkv_poll_status() == 0
    assert cache.xkv_get_info().T == ora.T and ora.last_scores is not None
