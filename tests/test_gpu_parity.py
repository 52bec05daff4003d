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


def test_tiny_stream_4bit_plain_arithmetic_forms(xkv, monkeypatch):
    """The maintenance kernels dequantise and quantise without conversion instructions when the
    zero-points and scaled values are small enough, and fall back to the plain forms otherwise.
    XKV_FORCE_PLAIN=1 (read when a cache is created) sends every kernel down the fallback:
    both must give the oracle's bits."""
    monkeypatch.setenv("XKV_FORCE_PLAIN", "1")
    p = xkv.Params(budget=1024, max_frame_tokens=261, kv_bits=4)
    cache, ora, worst = run_stream(xkv, p, 261, 7, seed=11)
    assert cache.xkv_get_info().T == 1024


def test_large_offset_keys(xkv):
    """Keys with a large common offset: zero-points of a few thousand and |x / s| far from 0."""
    import torch
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
        # keys near 100 with a spread of 0.05 cannot be held in 16-bit operands (spacing 0.06), so the
        # attention check uses the fp32 CUDA-core kernel; the point here is the bit-exact state above
        out = cache.attn_packed_causal(q, impl=1)
        check_attention(bf16_tensor_to_f32(out).transpose(1, 0, 2), ora.attend(qf), f"frame {t}")
    assert cache.xkv_get_info().T == 400


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
        cache.kv_score_evict(q[:, :50])
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
