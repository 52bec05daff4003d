"""attn_packed_causal_static: attention for callers that must not allocate.

Some users of the library run where cudaMalloc is forbidden (a host that bans
allocation after start-up, a plug-in without its own allocator).  For them the
library offers attention with the split-KV partials in a fixed device array
that belongs to the library image.  This file checks, through the C ABI, that
the variant returns what attn_packed_causal returns and what the CPU oracle
computes, on several frames in a row (the array is shared and keeps the previous
call's contents), also with fewer thread blocks than the GPU has multiprocessors
(the array holds 496 partial slots of 67 584 bytes, two per block: a GPU with more
than 248 multiprocessors would run capped; a B200 has 148, so the test caps the
block count through the library's test hook to walk that path).

The file name sorts last on purpose: a run that stops at the first failure has
then already executed every other test.
"""
import numpy as np
import pytest

from oracle import xkv_oracle as xo
from paper_2601_01204_b200 import synth
from xkv_testlib import (ATTN_MAXABS, ATTN_RELL2, attn_errors, bf16_tensor_to_f32, check_attention, oracle_params,
                         to_device_bf16)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def xkv():
    import torch
    assert torch.cuda.is_available()
    import paper_2601_01204_b200.xkv as m
    return m


def _frames(seed, n_frames, H, n, d):
    return [synth.gen_frame(seed, 0, t, H, n, d) for t in range(n_frames)]


def test_static_scratch_attention_matches_workspace_attention(xkv):
    import torch
    H, n, d = 16, 261, 64
    p = xkv.Params(budget=1024, max_frame_tokens=n, kv_bits=4)
    ref_cache, sta_cache = xkv.Cache(p), xkv.Cache(p)
    checked = 0
    for t, (qb, kb, vb) in enumerate(_frames(31, 7, H, n, d)):
        q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        outs = []
        for cache, static in ((ref_cache, False), (sta_cache, True)):
            cache.kv_append(k, v)
            cache.kv_score_evict(q)
            cache.kv_quant_pack()
            out = torch.full_like(q, float("nan"))
            if static:
                cache.attn_packed_causal_static(q, out)
            else:
                cache.attn_packed_causal(q, out)
            assert cache.xkv_poll_status() == 0
            outs.append(bf16_tensor_to_f32(out))
        ref, got = outs
        assert np.isfinite(got).all()
        maxabs, rell2 = attn_errors(got, ref)
        assert maxabs <= ATTN_MAXABS and rell2 <= ATTN_RELL2, (t, maxabs, rell2)
        checked += 1
    # the last frames run with a full cache and several key splits, back to back on the shared array
    assert checked >= 2 and sta_cache.xkv_get_info().T == 1024


@pytest.mark.parametrize("max_blocks", [0, 24])
def test_static_scratch_attention_larger_frames(xkv, max_blocks):
    """Frames of several query-tile pairs and many heads: the fixed array must still do (its size
    does not depend on the frame).  max_blocks = 24 runs both variants with fewer thread blocks
    than multiprocessors, as the static variant would on a GPU too large for its array.  Checked
    against attn_packed_causal and against the oracle."""
    import torch
    H, n, d = 24, 700, 64
    p = xkv.Params(n_heads=H, budget=2048, max_frame_tokens=n, kv_bits=4)
    ref_cache, sta_cache = xkv.Cache(p), xkv.Cache(p)
    ora = xo.OracleLayer(oracle_params(p))
    for c in (ref_cache, sta_cache):
        c.xkv_debug_limit_attention_blocks(max_blocks)
    for t, (qb, kb, vb) in enumerate(_frames(32, 4, H, n, d)):
        q, k, v = (to_device_bf16(x) for x in (qb, kb, vb))
        outs = []
        for cache, static in ((ref_cache, False), (sta_cache, True)):
            cache.kv_append(k, v)
            cache.kv_score_evict(q)
            cache.kv_quant_pack()
            out = torch.full_like(q, float("nan"))
            if static:
                cache.attn_packed_causal_static(q, out)
            else:
                cache.attn_packed_causal(q, out)
            assert cache.xkv_poll_status() == 0
            outs.append(bf16_tensor_to_f32(out))
        maxabs, rell2 = attn_errors(outs[1], outs[0])
        assert maxabs <= ATTN_MAXABS and rell2 <= ATTN_RELL2, (t, maxabs, rell2)
        qf, kf, vf = (synth.bf16_bits_to_f32(x) for x in (qb, kb, vb))
        check_attention(outs[1].transpose(1, 0, 2), ora.step(qf, kf, vf), f"frame {t} against the oracle")
