"""Parity at the full size of the benchmark configuration, in the launch configuration bench.py
times (32K context, 8 KV heads, GQA 4, bf16, M = 1024, 64 classes of 512 slots, FFT decode):
the whole GPU cache is built and decoded; the oracle recomputes sampled KV heads one by one."""
import numpy as np
import pytest
import torch

from oracle import fa_oracle as fo
from paper_2506_11886_b200 import fa, synth
from tests.parity_util import COEF_REL, OUT_ABS_BF16, layout_of, to64, unswizzle_v_rows

pytestmark = pytest.mark.gpu


def _sampled_head_check(shape, layout, heads, steps, seed, rows=None):
    rows = list(range(shape.B)) if rows is None else list(rows)      # batch rows the oracle recomputes
    stream = synth.KVStream(shape, seed=seed, device="cuda")
    K, V = stream.tokens(0, shape.L, work_dtype=torch.float32)
    cache = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
    ws = fa.new_workspace(layout)
    fa.fa_validate(layout, cache)
    fa.fa_compress(layout, cache, K, V, ws)
    Kn, Vn = stream.tokens(shape.L, shape.L + steps, work_dtype=torch.float32)
    for t in range(steps):
        fa.fa_append(layout, cache, Kn[:, t].contiguous(), Vn[:, t].contiguous())
    q = synth.queries(shape, seed=seed, device="cuda")
    out = torch.empty_like(q)
    fa.fa_decode_attention(layout, cache, q, out, ws)
    torch.cuda.synchronize()
    assert fa.fa_poll_status(cache) == fa.FA_OK
    G = shape.Hq // shape.Hkv
    worst_out = worst_coef = 0.0
    for h in heads:
        sub = fo.OracleConfig(B=len(rows), Hq=G, Hkv=1, d=shape.d, n_full_k=shape.n_full_k, n_full_v=shape.n_full_v,
                              k=shape.k, T=shape.T, L_init=shape.L_init, L_local=shape.L_local, cap_mid=layout.max_mid,
                              scale=shape.softmax_scale)
        ref = fo.OracleCache(sub, stream.idx_full_k[h:h + 1].numpy(), stream.idx_full_v[h:h + 1].numpy())
        ref.compress(to64(K[rows][:, :, h:h + 1]), to64(V[rows][:, :, h:h + 1]))
        for t in range(steps):
            ref.append(to64(Kn[rows][:, t, h:h + 1]), to64(Vn[rows][:, t, h:h + 1]))
        want = ref.decode(to64(q[rows][:, h * G:(h + 1) * G]))
        got = to64(out[rows][:, h * G:(h + 1) * G])
        worst_out = max(worst_out, np.abs(got - want).max())
        # metadata and stored rows of the sampled head: bit-exact; coefficients: norm-wise
        st = cache.state.cpu().numpy()[rows]
        assert (st[:, 2] == ref.n_mid).all() and (st[:, 1] == ref.n_local).all() and (st[:, 0] == ref.n_init).all()
        for bi, b in enumerate(rows):
            nm, head = int(st[bi, 2]), int(st[bi, 3])
            j = np.arange(nm)
            gk = to64(cache.k_mid[b, h])[j % layout.mid_classes, j // layout.mid_classes]
            gv = to64(cache.v_mid[b, h])[j % layout.mid_classes, j // layout.mid_classes]
            gv = unswizzle_v_rows(gv[None], j // layout.mid_classes, layout)[0]
            np.testing.assert_array_equal(gk, ref.k_mid[bi, 0, :nm])
            np.testing.assert_array_equal(gv, ref.v_mid[bi, 0, :nm])
            order = (head + np.arange(shape.L_local)) % shape.L_local
            np.testing.assert_array_equal(to64(cache.k_local[b, h])[order], ref.k_local[bi, 0])
            for name in ("coef_k", "coef_v"):
                r = getattr(ref, name)[bi, 0]
                g = to64(getattr(cache, name)[b, h])
                worst_coef = max(worst_coef, np.abs(g - r).max() / np.abs(r).max())
    assert worst_coef <= COEF_REL, worst_coef
    assert worst_out <= OUT_ABS_BF16, worst_out
    return worst_out, worst_coef


def test_llama31_8b_32k_sampled_heads():
    shape = synth.CONFIGS[1]
    layout = layout_of(shape, max_mid=shape.T, P=shape.T // shape.k)
    assert layout.mid_classes == 64
    _sampled_head_check(shape, layout, heads=(0, 7), steps=3, seed=1000)


def test_llama2_7b_mha_batch8_sampled_heads():
    """Serving configuration: MHA (G = 1), batch 8, 4K prompt, 48 kept / 80 compressed dims, M = 256;
    a few append + decode steps, first and last head recomputed by the oracle for all batch rows."""
    shape = synth.CONFIGS[3]
    layout = layout_of(shape, max_mid=shape.T, P=shape.T // shape.k)
    _sampled_head_check(shape, layout, heads=(0, 31), steps=5, seed=3000)


def test_128k_batch4_one_sampled_head():
    """Long-context stress shape: 128K tokens, batch 4, M = 2048, 2048-token recent window; the
    oracle recomputes one (batch row, KV head)."""
    shape = synth.CONFIGS[4]
    layout = layout_of(shape, max_mid=shape.T, P=shape.T // shape.k)
    assert fa.fa_launch_count(layout, 4) == 1                  # the split build of the fused kernel serves this shape
    _sampled_head_check(shape, layout, heads=(5,), steps=2, seed=4000, rows=(3,))


def _timed_entry_points_check(shape, layout, heads, seed, rows=None, n_dev=40, n_host=8, check_at=(0, 39, 47)):
    """The two calls the benchmark times, at its sizes and in its launch configuration: n_dev
    fa_decode_step calls (device inputs) followed by n_host fa_decode_step_host calls (pinned host
    buffers) on one cache.  The oracle appends the same tokens for the sampled (row, KV head) pairs
    and decodes at the checkpoint steps: outputs within the absolute tolerance, and at the end
    counters, K^mu / V^mu, the ring bit-exact and the coefficients norm-wise within 1e-3."""
    rows = list(range(shape.B)) if rows is None else list(rows)
    stream = synth.KVStream(shape, seed=seed, device="cuda")
    K, V = stream.tokens(0, shape.L, work_dtype=torch.float32)
    cache = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
    ws = fa.new_workspace(layout)
    fa.fa_validate(layout, cache)
    fa.fa_compress(layout, cache, K, V, ws)
    steps = n_dev + n_host
    Kn, Vn = stream.tokens(shape.L, shape.L + steps, work_dtype=torch.float32)
    qs = torch.stack([synth.queries(shape, seed=seed, step=t, device="cuda") for t in range(steps)])
    outs = torch.full_like(qs, float("nan"))
    for t in range(n_dev):
        fa.fa_decode_step(layout, cache, qs[t], Kn[:, t].contiguous(), Vn[:, t].contiguous(), outs[t], ws)
    staging = torch.zeros(fa.fa_step_staging_bytes(layout), dtype=torch.uint8, device="cuda")
    q_h = qs.cpu().pin_memory()
    k_h, v_h = Kn.transpose(0, 1).contiguous().cpu().pin_memory(), Vn.transpose(0, 1).contiguous().cpu().pin_memory()
    out_h = torch.full(tuple(qs.shape), float("nan"), dtype=qs.dtype).pin_memory()
    for t in range(n_dev, steps):
        fa.fa_decode_step_host(layout, cache, q_h[t], k_h[t], v_h[t], out_h[t], staging, ws)
    torch.cuda.synchronize()
    assert fa.fa_poll_status(cache) == fa.FA_OK
    outs[n_dev:] = out_h[n_dev:].cuda()
    assert torch.isfinite(outs.float()).all()
    G = shape.Hq // shape.Hkv
    worst_out = worst_coef = 0.0
    st = cache.state.cpu().numpy()[rows]
    for h in heads:
        sub = fo.OracleConfig(B=len(rows), Hq=G, Hkv=1, d=shape.d, n_full_k=shape.n_full_k, n_full_v=shape.n_full_v,
                              k=shape.k, T=shape.T, L_init=shape.L_init, L_local=shape.L_local, cap_mid=layout.max_mid,
                              scale=shape.softmax_scale)
        ref = fo.OracleCache(sub, stream.idx_full_k[h:h + 1].numpy(), stream.idx_full_v[h:h + 1].numpy())
        ref.compress(to64(K[rows][:, :, h:h + 1]), to64(V[rows][:, :, h:h + 1]))
        for t in range(steps):
            ref.append(to64(Kn[rows][:, t, h:h + 1]), to64(Vn[rows][:, t, h:h + 1]))
            if t in check_at:
                want = ref.decode(to64(qs[t][rows][:, h * G:(h + 1) * G]))
                got = to64(outs[t][rows][:, h * G:(h + 1) * G])
                err = np.abs(got - want).max()
                assert err <= OUT_ABS_BF16, (h, t, err)
                worst_out = max(worst_out, err)
        assert (st[:, 2] == ref.n_mid).all() and (st[:, 1] == ref.n_local).all() and (st[:, 0] == ref.n_init).all()
        for bi, b in enumerate(rows):
            nm, head = int(st[bi, 2]), int(st[bi, 3])
            j = np.arange(nm)
            gk = to64(cache.k_mid[b, h])[j % layout.mid_classes, j // layout.mid_classes]
            gv = to64(cache.v_mid[b, h])[j % layout.mid_classes, j // layout.mid_classes]
            gv = unswizzle_v_rows(gv[None], j // layout.mid_classes, layout)[0]
            np.testing.assert_array_equal(gk, ref.k_mid[bi, 0, :nm])
            np.testing.assert_array_equal(gv, ref.v_mid[bi, 0, :nm])
            order = (head + np.arange(shape.L_local)) % shape.L_local
            np.testing.assert_array_equal(to64(cache.k_local[b, h])[order], ref.k_local[bi, 0])
            np.testing.assert_array_equal(to64(cache.v_local[b, h])[order], ref.v_local[bi, 0])
            for name in ("coef_k", "coef_v"):
                r = getattr(ref, name)[bi, 0]
                g = to64(getattr(cache, name)[b, h])
                worst_coef = max(worst_coef, np.abs(g - r).max() / np.abs(r).max())
    assert worst_coef <= COEF_REL, worst_coef
    return worst_out, worst_coef


def test_timed_entry_points_llama31_8b_32k():
    """fa_decode_step x 40 and fa_decode_step_host x 8 on the headline configuration, layout as the
    benchmark builds it (64 classes of 512 slots, period 32768)."""
    shape = synth.CONFIGS[1]
    layout = layout_of(shape, max_mid=shape.T, P=shape.T // shape.k)
    _timed_entry_points_check(shape, layout, heads=(0, 7), seed=1001)


def test_timed_entry_points_llama2_7b_mha_batch8():
    shape = synth.CONFIGS[3]
    layout = layout_of(shape, max_mid=shape.T, P=shape.T // shape.k)
    _timed_entry_points_check(shape, layout, heads=(0, 31), seed=3001, rows=(0, 7))


def test_timed_entry_points_128k_batch4():
    shape = synth.CONFIGS[4]
    layout = layout_of(shape, max_mid=shape.T, P=shape.T // shape.k)
    _timed_entry_points_check(shape, layout, heads=(5,), seed=4001, rows=(3,), check_at=(0, 47))


def test_compress_by_transform_32k_one_head():
    """FA_COMPRESS_FFT on the 32K prefill of the headline configuration: coefficients of one KV head against the oracle."""
    shape = synth.CONFIGS[1]
    layout = layout_of(shape, max_mid=shape.T, P=shape.T // shape.k)
    stream = synth.KVStream(shape, seed=1002, device="cuda")
    K, V = stream.tokens(0, shape.L, work_dtype=torch.float32)
    cache = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
    ws = fa.new_workspace(layout)
    fa.fa_compress(layout, cache, K, V, ws, flags=fa.FA_COMPRESS_FFT)
    torch.cuda.synchronize()
    h = 3
    sub = fo.OracleConfig(B=1, Hq=4, Hkv=1, d=shape.d, n_full_k=shape.n_full_k, n_full_v=shape.n_full_v, k=shape.k, T=shape.T,
                          L_init=shape.L_init, L_local=shape.L_local, cap_mid=layout.max_mid, scale=1.0)
    ref = fo.OracleCache(sub, stream.idx_full_k[h:h + 1].numpy(), stream.idx_full_v[h:h + 1].numpy())
    ref.compress(to64(K[:, :, h:h + 1]), to64(V[:, :, h:h + 1]))
    for name in ("coef_k", "coef_v"):
        r = getattr(ref, name)[0, 0]
        g = to64(getattr(cache, name)[0, h])
        assert np.abs(g - r).max() / np.abs(r).max() <= 2e-5, name
    assert fa.fa_poll_status(cache) == fa.FA_OK
