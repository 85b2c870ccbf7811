"""Parity of the CUDA path (through the C ABI) against the fp64 oracle on the
same seeded inputs: cache metadata and stored rows bit-exact, coefficients and
attention outputs within the stated tolerances.  Small and medium sizes that
still span several tiles, classes and a ragged tail, plus the edge cases."""
import numpy as np
import pytest
import torch

from paper_2506_11886_b200 import fa, synth
from tests.parity_util import Pair, layout_of, make_pair as _make_pair, to64

pytestmark = pytest.mark.gpu


def make_pair(*a, **kw):
    """make_pair, skipping the case if the requested decode algorithm cannot serve the layout."""
    try:
        return _make_pair(*a, **kw)
    except fa.FaError as e:
        if e.status == fa.FA_ERR_UNSUPPORTED and kw.get("algo") in (fa.FA_DECODE_FFT, fa.FA_DECODE_FFT_SPLIT):
            pytest.skip("layout outside the FFT kernel's range")
        raise

CFG0 = synth.CONFIGS[0]
SMALL_BF16 = synth.Shape("small_bf16_gqa", B=2, layers=1, Hq=8, Hkv=2, d=128, L=1500, dtype="bf16", n_full_k=32,
                         n_full_v=48, M=128, T=2048, L_init=4, L_local=64, decode_steps=40)
ALGOS = [fa.FA_DECODE_DIRECT, fa.FA_DECODE_FFT, fa.FA_DECODE_FFT_SPLIT]


@pytest.mark.parametrize("P", [1, 32])
@pytest.mark.parametrize("algo", ALGOS)
def test_cfg0_toy_compress_then_decode(P, algo):
    """Configuration 0: fp32, GQA 4, L = 1024, 32 kept / 96 compressed dims, M = 64."""
    pair, _ = make_pair(CFG0, seed=0, P=P, algo=algo)
    pair.check_state()
    for step in range(3):
        pair.check_decode(synth.queries(CFG0, seed=0, step=step))
    pair.check_decode(synth.queries(CFG0, seed=0, step=9, peak=8.0))      # peaked softmax


@pytest.mark.parametrize("algo", ALGOS)
def test_cfg0_with_windows_and_offgrid_frequencies(algo):
    shape = CFG0.with_(L_init=4, L_local=64)
    pair, _ = make_pair(shape, seed=1, algo=algo, freq="offgrid")
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=1))


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("P", [1, 32])
def test_bf16_gqa_append_and_decode(algo, P):
    """bf16, 2 batch rows, GQA 4, asymmetric K/V index sets, ragged classes; appends wrap the ring."""
    shape = SMALL_BF16
    pair, stream = make_pair(shape, seed=2, algo=algo, P=P, max_mid=2048)
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=2))
    t = shape.L
    for step in range(70):                       # more than l_local appends: the ring wraps
        k_new, v_new = stream.tokens(t, t + 1)
        pair.append(k_new[:, 0], v_new[:, 0])
        t += 1
        if step in (0, 1, 63, 64, 69):
            pair.check_state()
            pair.check_decode(synth.queries(shape, seed=2, step=step + 1))


@pytest.mark.parametrize("algo", ALGOS)
def test_append_from_empty_equals_compress(algo):
    """Tokens fill init, then local, then spill into the middle; compare with one compress call."""
    shape = SMALL_BF16.with_(B=1, Hq=2, Hkv=1, L=0, L_init=3, L_local=8, T=256, M=32, n_full_k=16, n_full_v=8)
    layout = layout_of(shape, max_mid=256, P=8, algo=algo)
    assert fa.fa_workspace_bytes(layout) > 0
    stream = synth.KVStream(shape, seed=3)
    pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    fa.fa_cache_reset(layout, pair.gpu)
    K0, V0 = stream.tokens(0, 0)
    pair.ref.compress(to64(K0), to64(V0))
    K, V = stream.tokens(0, 40)
    for t in range(40):
        pair.append(K[:, t], V[:, t])
        if t in (0, 2, 3, 10, 11, 39):
            pair.check_state()
            pair.check_decode(synth.queries(shape, seed=3, step=t))
    again = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    again.compress(K, V)
    for name in ("k_init", "v_init", "k_mid", "v_mid"):
        assert torch.equal(getattr(again.gpu, name), getattr(pair.gpu, name)), name
    den = again.gpu.coef_k.abs().max()
    assert (again.gpu.coef_k - pair.gpu.coef_k).abs().max() / den < 1e-4
    assert torch.equal(again.gpu.state[:, :3], pair.gpu.state[:, :3])


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("nfk,nfv", [(0, 0), (128, 128), (128, 32), (8, 120), (0, 64), (64, 0), (8, 56)])
def test_degenerate_index_sets(algo, nfk, nfv):
    """Everything compressed, nothing compressed (plain attention), and mixed extremes."""
    shape = SMALL_BF16.with_(B=1, Hq=4, Hkv=2, L=700, n_full_k=nfk, n_full_v=nfv, T=1024, M=64)
    pair, stream = make_pair(shape, seed=4, algo=algo, P=32, max_mid=1024)
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=4))
    k_new, v_new = stream.tokens(shape.L, shape.L + 1)
    pair.append(k_new[:, 0], v_new[:, 0])
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=4, step=1))


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("L", [0, 1, 3, 4, 5, 67, 68, 69, 100])
def test_short_prompts(algo, L):
    """Prompts shorter than the windows, and the first few middle tokens."""
    shape = SMALL_BF16.with_(B=2, L=L, T=512, M=32)
    pair, _ = make_pair(shape, seed=5, L=L, algo=algo, P=16, max_mid=512)
    pair.check_state()
    got, want = pair.decode(synth.queries(shape, seed=5))
    if L == 0:
        assert not got.any() and not want.any()
    else:
        assert np.abs(got - want).max() < 2e-2


@pytest.mark.parametrize("algo", ALGOS)
def test_no_local_window_and_odd_period(algo):
    """l_local = 0 (appended tokens go straight to the middle), period not a power of two, G = 1, fp32."""
    shape = synth.Shape("odd", B=1, layers=1, Hq=2, Hkv=2, d=64, L=300, dtype="f32", n_full_k=16, n_full_v=24, M=50,
                        T=777, L_init=2, L_local=0)
    pair, stream = make_pair(shape, seed=6, algo=fa.FA_DECODE_DIRECT, P=7, max_mid=777)
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=6))
    K, V = stream.tokens(300, 310)
    for t in range(10):
        pair.append(K[:, t], V[:, t])
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=6, step=1))


def test_paper_literal_scale():
    shape = CFG0.with_(L_init=4, L_local=64)
    pair, _ = make_pair(shape, seed=7, norm=fa.FA_NORM_PAPER)
    pair.check_decode(synth.queries(shape, seed=7))


def test_strided_prefill_input():
    """K, V given as slices of a larger [B][L][H][2d] buffer."""
    shape = SMALL_BF16.with_(B=2, L=300, T=512, M=32)
    layout = layout_of(shape, max_mid=512, P=16)
    stream = synth.KVStream(shape, seed=8)
    K, V = stream.tokens(0, 300)
    big = torch.zeros((2, 300, shape.Hkv, 2, 2 * shape.d), dtype=K.dtype, device="cuda")
    big[:, :, :, 0, :shape.d] = K.cuda()
    big[:, :, :, 1, :shape.d] = V.cuda()
    pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    fa.fa_compress(layout, pair.gpu, big[:, :, :, 0, :shape.d], big[:, :, :, 1, :shape.d], pair.ws)
    pair.ref.compress(to64(K), to64(V))
    pair.check_state()


def test_errors_are_reported_not_raised_on_device():
    shape = SMALL_BF16.with_(B=1, Hq=2, Hkv=1, L=80, T=128, M=16)
    layout = layout_of(shape, max_mid=10, P=4)
    stream = synth.KVStream(shape, seed=9)
    pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    K, V = stream.tokens(0, 80)
    with pytest.raises(fa.FaError) as e:                      # 80 - 4 - 64 = 12 middle tokens > 10
        fa.fa_compress(layout, pair.gpu, K.cuda(), V.cuda(), pair.ws)
    assert e.value.status == fa.FA_ERR_CAPACITY
    pair.compress(K[:, :78], V[:, :78])                       # exactly full
    pair.check_state()
    before = {n: getattr(pair.gpu, n).clone() for n in ("coef_k", "coef_v", "k_mid", "k_local", "state")}
    fa.fa_append(layout, pair.gpu, K[:, 79].cuda().contiguous(), V[:, 79].cuda().contiguous())
    assert fa.fa_poll_status(pair.gpu) == fa.FA_ERR_CAPACITY   # reported through the status word
    assert fa.fa_poll_status(pair.gpu) == fa.FA_OK             # and cleared by the poll
    for n, t in before.items():
        assert torch.equal(getattr(pair.gpu, n), t), n         # the refused append changed nothing
    # prefill rows off the 16-byte grid (a view one element into a wider buffer) are refused, nothing is launched
    wide = torch.zeros((1, 78, shape.Hkv, shape.d + 8), dtype=K.dtype, device="cuda")
    with pytest.raises(fa.FaError) as e:
        fa.fa_compress(layout, pair.gpu, wide[..., 1:shape.d + 1], wide[..., 1:shape.d + 1], pair.ws)
    assert e.value.status == fa.FA_ERR_INVALID_ARG
    # workspace too small / missing
    q = synth.queries(shape, seed=9).cuda()
    out = torch.empty_like(q)
    with pytest.raises(fa.FaError) as e:
        fa.fa_decode_attention(layout, pair.gpu, q, out, pair.ws[:64])
    assert e.value.status == fa.FA_ERR_WORKSPACE
    # broken index sets are caught by fa_validate
    bad = stream.idx_full_k.clone()
    bad[0, 0], bad[0, 1] = bad[0, 1].item(), bad[0, 0].item()
    c2 = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
    c2.idx_full_k.copy_(bad.cuda())
    with pytest.raises(fa.FaError) as e:
        fa.fa_validate(layout, c2)
    assert e.value.status == fa.FA_ERR_INDEX


def test_snapshot_restore():
    """The cache is plain caller-owned memory: copying it back restores the outputs."""
    shape = SMALL_BF16.with_(B=1, L=400, T=512, M=32)
    pair, stream = make_pair(shape, seed=10, P=16, max_mid=512)
    q = synth.queries(shape, seed=10).cuda()
    out0, out1 = torch.empty_like(q), torch.empty_like(q)
    fa.fa_decode_attention(pair.layout, pair.gpu, q, out0, pair.ws)
    names = ("k_init", "v_init", "k_local", "v_local", "k_mid", "v_mid", "coef_k", "coef_v", "state")
    snap = {n: getattr(pair.gpu, n).clone() for n in names}
    K, V = stream.tokens(400, 416)
    for t in range(16):
        fa.fa_append(pair.layout, pair.gpu, K[:, t].cuda().contiguous(), V[:, t].cuda().contiguous())
    for n in names:
        getattr(pair.gpu, n).copy_(snap[n])
    fa.fa_decode_attention(pair.layout, pair.gpu, q, out1, pair.ws)
    assert torch.equal(out0, out1)


@pytest.mark.parametrize("algo", ALGOS)
def test_many_classes_per_cta(algo):
    """Several residue classes per CTA and per transform batch (B * H_kv large, 64 classes of 64 slots):
    the producer and the consumers must walk the tiles of a batch in the same order."""
    shape = synth.Shape("many_classes", B=2, layers=1, Hq=32, Hkv=8, d=128, L=3600, dtype="bf16", n_full_k=32,
                        n_full_v=32, M=128, T=4096, L_init=4, L_local=128)
    pair, stream = make_pair(shape, seed=11, algo=algo, P=64, max_mid=4096)
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=11))
    K, V = stream.tokens(shape.L, shape.L + 3)
    for t in range(3):
        pair.append(K[:, t], V[:, t])
    pair.check_decode(synth.queries(shape, seed=11, step=1, peak=4.0))


@pytest.mark.parametrize("algo", ALGOS)
def test_mha_48_kept_dims(algo):
    """The MHA serving shape in small: G = 1, 48 kept / 80 compressed dims, M = 256, batch 3."""
    shape = synth.Shape("mha48", B=3, layers=1, Hq=4, Hkv=4, d=128, L=2500, dtype="bf16", n_full_k=48, n_full_v=48,
                        M=256, T=4096, L_init=4, L_local=256)
    pair, stream = make_pair(shape, seed=12, algo=algo, P=32, max_mid=4096)
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=12))
    K, V = stream.tokens(shape.L, shape.L + 2)
    for t in range(2):
        pair.append(K[:, t], V[:, t])
    pair.check_state()
    pair.check_decode(synth.queries(shape, seed=12, step=1))


@pytest.mark.parametrize("kw,P", [
    (dict(B=3, Hq=7, Hkv=7, L=3000, T=4096, M=128), 32),      # 21 heads: 4 or 5 classes per CTA, the last transform of a batch half empty
    (dict(B=2, Hq=3, Hkv=3, L=1700, T=2048, M=128), 8),       # more CTAs per head than classes: one class per CTA, slot 1 never used
    (dict(B=1, Hq=40, Hkv=40, L=2300, T=4096, M=256), 16),    # lone CTAs, two per SM: all 16 classes and the windows in one CTA
])
def test_mha_two_classes_per_packed_transform(kw, P):
    """One query head per KV head: the transform kernel packs two residue classes into a complex transform (the two
    slots are one head: own maxima, sums, outputs and z per slot, folded before the partial results).  Ragged class
    lengths, odd class counts per batch, decode call and fused steps (the pending middle token lands in either slot)."""
    shape = SMALL_BF16.with_(d=128, n_full_k=48, n_full_v=32, L_init=4, L_local=64, decode_steps=3, **kw)
    pair, stream = make_pair(shape, seed=33, algo=fa.FA_DECODE_FFT, P=P, max_mid=shape.T)
    pair.check_decode(synth.queries(shape, seed=33))
    K, V = stream.tokens(shape.L, shape.L + 3)
    for t in range(3):
        pair.check_step(synth.queries(shape, seed=33, step=t + 1), K[:, t], V[:, t])
    pair.check_state()


@pytest.mark.parametrize("algo", ALGOS)
def test_decode_step_from_empty_through_eviction(algo):
    """fa_decode_step token by token: init fills, local fills, then every step evicts a row into the middle;
    outputs against append + decode of the oracle, the cache against the oracle's at the end."""
    shape = SMALL_BF16.with_(B=1, Hq=4, Hkv=1, L=0, L_init=3, L_local=8, T=256, M=32, n_full_k=16, n_full_v=8)
    layout = layout_of(shape, max_mid=256, P=8, algo=algo)
    stream = synth.KVStream(shape, seed=11)
    pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    fa.fa_cache_reset(layout, pair.gpu)
    K0, V0 = stream.tokens(0, 0)
    pair.ref.compress(to64(K0), to64(V0))
    K, V = stream.tokens(0, 60)
    for t in range(60):
        pair.check_step(synth.queries(shape, seed=11, step=t), K[:, t], V[:, t])
        if t in (2, 3, 10, 11, 12, 40, 59):
            pair.check_state()
    # the same workspace keeps serving plain decode calls
    pair.check_decode(synth.queries(shape, seed=12))


def test_decode_step_after_compress_gqa_batch():
    """Prefill, then fused steps on a batch of two rows with four query heads per KV head."""
    shape = SMALL_BF16.with_(L=700, decode_steps=12)
    pair, stream = make_pair(shape, seed=13, algo=fa.FA_DECODE_FFT, P=16)
    K, V = stream.tokens(shape.L, shape.L + 12)
    for t in range(12):
        pair.check_step(synth.queries(shape, seed=13, step=t), K[:, t], V[:, t])
    pair.check_state()
    assert fa.fa_launch_count(pair.layout, 3) in (1, 2, 4)       # one launch where the decode call is the fused kernel


def test_decode_step_full_middle_reports_capacity():
    """A step whose append finds the middle full changes nothing, reports it, and still decodes."""
    shape = SMALL_BF16.with_(B=1, Hq=4, Hkv=1, L=0, L_init=2, L_local=4, T=64, M=16, n_full_k=16, n_full_v=8)
    layout = layout_of(shape, max_mid=8, P=2, algo=fa.FA_DECODE_FFT)
    stream = synth.KVStream(shape, seed=14)
    try:
        pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    except fa.FaError as e:
        if e.status == fa.FA_ERR_UNSUPPORTED:
            pytest.skip("layout outside the FFT kernel's range")
        raise
    fa.fa_cache_reset(layout, pair.gpu)
    K0, V0 = stream.tokens(0, 0)
    pair.ref.compress(to64(K0), to64(V0))
    K, V = stream.tokens(0, 15)
    for t in range(14):                                   # 2 + 4 + 8 tokens fill everything
        pair.check_step(synth.queries(shape, seed=14, step=t), K[:, t], V[:, t])
    q = synth.queries(shape, seed=14, step=99)
    out = torch.full_like(q, float("nan"), device="cuda")
    fa.fa_decode_step(layout, pair.gpu, q.cuda().contiguous(), K[:, 14].cuda().contiguous(), V[:, 14].cuda().contiguous(),
                      out, pair.ws)
    assert fa.fa_poll_status(pair.gpu) == fa.FA_ERR_CAPACITY
    want = pair.ref.decode(to64(q))                       # the oracle cache did not take the token either
    assert np.abs(to64(out) - want).max() <= 2e-2
    pair.check_state()


@pytest.mark.parametrize("pinned", [True, False])
def test_decode_step_host_buffers(pinned):
    """The host-buffer step (pinned buffers are read by a staging kernel, pageable ones copied) gives the
    same outputs and cache as the oracle's append + decode."""
    shape = SMALL_BF16.with_(L=400, decode_steps=6)
    pair, stream = make_pair(shape, seed=15, algo=fa.FA_DECODE_FFT, P=16)
    staging = torch.zeros(fa.fa_step_staging_bytes(pair.layout), dtype=torch.uint8, device="cuda")
    K, V = stream.tokens(shape.L, shape.L + 6)

    def host(t):
        t = t.contiguous().cpu()
        return t.pin_memory() if pinned else t

    for t in range(6):
        q = synth.queries(shape, seed=15, step=t)
        out_h = host(torch.zeros_like(q))
        fa.fa_decode_step_host(pair.layout, pair.gpu, host(q), host(K[:, t]), host(V[:, t]), out_h, staging, pair.ws)
        torch.cuda.synchronize()
        pair.ref.append(to64(K[:, t]), to64(V[:, t]))
        want = pair.ref.decode(to64(q))
        assert np.abs(to64(out_h) - want).max() <= 2e-2
    pair.check_state()


def test_ragged_batch_compress_append_decode():
    """Rows of one batch with different prompt lengths: each row must behave as a one-row cache of its own
    (oracle: one cache per row), through compression, steps that evict in one row and not in the other,
    and decode."""
    from oracle import fa_oracle as fo
    from tests.parity_util import oracle_cfg
    shape = SMALL_BF16.with_(B=2, L=1200, T=2048, M=128)
    layout = layout_of(shape, max_mid=2048, P=16, algo=fa.FA_DECODE_FFT)
    stream = synth.KVStream(shape, seed=16)
    K, V = stream.tokens(0, 1200)
    lengths = [1200, 37]                                    # the second row has not even filled its local window
    try:
        gpu = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
        ws = fa.new_workspace(layout)
        fa.fa_compress_ragged(layout, gpu, K.cuda(), V.cuda(), lengths, ws)
    except fa.FaError as e:
        if e.status == fa.FA_ERR_UNSUPPORTED:
            pytest.skip("layout outside the FFT kernel's range")
        raise
    refs = []
    for b in range(2):
        import dataclasses
        cfg = dataclasses.replace(oracle_cfg(layout), B=1)
        r = fo.OracleCache(cfg, stream.idx_full_k.numpy(), stream.idx_full_v.numpy())
        r.compress(to64(K[b:b + 1, :lengths[b]]), to64(V[b:b + 1, :lengths[b]]))
        refs.append(r)
    st = gpu.state.cpu().numpy()
    for b in range(2):
        assert (st[b, 0], st[b, 1], st[b, 2]) == (refs[b].n_init[0], refs[b].n_local[0], refs[b].n_mid[0])
    Kn, Vn = stream.tokens(1200, 1240)
    for t in range(40):                                      # row 0 evicts every step, row 1 fills its window then evicts
        q = synth.queries(shape, seed=16, step=t)
        out = torch.full_like(q, float("nan"), device="cuda")
        fa.fa_decode_step(layout, gpu, q.cuda().contiguous(), Kn[:, t].cuda().contiguous(), Vn[:, t].cuda().contiguous(), out, ws)
        torch.cuda.synchronize()
        for b in range(2):
            refs[b].append(to64(Kn[b:b + 1, t]), to64(Vn[b:b + 1, t]))
            want = refs[b].decode(to64(q[b:b + 1]))
            assert np.abs(to64(out[b:b + 1]) - want).max() <= 2e-2, (t, b)
    assert fa.fa_poll_status(gpu) == fa.FA_OK
    st = gpu.state.cpu().numpy()
    for b in range(2):
        assert (st[b, 0], st[b, 1], st[b, 2]) == (refs[b].n_init[0], refs[b].n_local[0], refs[b].n_mid[0])
        den = np.abs(refs[b].coef_k[0]).max()
        assert np.abs(to64(gpu.coef_k[b]) - refs[b].coef_k[0]).max() / max(den, 1e-30) <= 1e-3


@pytest.mark.parametrize("B", [2, 4, 8])
def test_fused_decode_with_row_chunks(B):
    """Batches whose parts hold more coefficient rows than the staging buffers take at once (the fused
    kernel then walks its slice in chunks), through fused steps and plain decode."""
    shape = SMALL_BF16.with_(B=B, Hq=16, Hkv=4, L=1300, T=2048, M=1024, n_full_k=32, n_full_v=32, decode_steps=4)
    pair, stream = make_pair(shape, seed=17, algo=fa.FA_DECODE_FFT, P=4)
    pair.check_decode(synth.queries(shape, seed=17))
    K, V = stream.tokens(shape.L, shape.L + 4)
    for t in range(4):
        pair.check_step(synth.queries(shape, seed=17, step=t + 1), K[:, t], V[:, t])
    pair.check_state()


def test_fused_decode_one_cta_per_head():
    """As many (batch row, KV head) pairs as SMs allow one CTA each: the fused kernel with a single part."""
    shape = SMALL_BF16.with_(B=16, Hq=16, Hkv=8, L=600, T=1024, M=128, n_full_k=32, n_full_v=48, decode_steps=2)
    pair, stream = make_pair(shape, seed=18, algo=fa.FA_DECODE_FFT, P=8)
    assert fa.fa_launch_count(pair.layout, 2) == 1
    pair.check_decode(synth.queries(shape, seed=18))
    K, V = stream.tokens(shape.L, shape.L + 2)
    for t in range(2):
        pair.check_step(synth.queries(shape, seed=18, step=t + 1), K[:, t], V[:, t])
    pair.check_state()


@pytest.mark.parametrize("T,P,M", [(1024, 8, 128), (2048, 4, 512)])
def test_fused_decode_more_heads_than_sms(T, P, M):
    """More (batch row, KV head) pairs than SMs: still one launch, one CTA per pair running in waves and
    waiting for nobody (no counters, plain launch).  Transform length 128: two CTAs share an SM (shorter
    ring, register cap); 512: one per SM."""
    shape = SMALL_BF16.with_(B=20, Hq=16, Hkv=8, L=700, T=T, M=M, n_full_k=32, n_full_v=48, decode_steps=2)
    pair, stream = make_pair(shape, seed=23, algo=fa.FA_DECODE_FFT, P=P)
    assert fa.fa_launch_count(pair.layout, 2) == 1 and fa.fa_launch_count(pair.layout, 3) == 2      # one part per head: append kernel + fused decode
    pair.check_decode(synth.queries(shape, seed=23))
    K, V = stream.tokens(shape.L, shape.L + 2)
    for t in range(2):
        pair.check_step(synth.queries(shape, seed=23, step=t + 1), K[:, t], V[:, t])
    pair.check_state()


def test_fused_decode_split_build_long_transforms():
    """Transform length 1024 with several class batches per CTA takes the split build of the fused kernel (a tile group
    of warps forms the kept-dim products of a batch beside the transform group's phases on it, handshakes on four
    shared-memory barriers), in the decode call and in the one-launch step.  Here GH = 2 and two classes per batch;
    the 128K configuration of the full-size tests runs it with GH = 4 and one class per batch."""
    shape = SMALL_BF16.with_(B=4, Hq=16, Hkv=8, L=4200, T=16384, M=512, n_full_k=32, n_full_v=48, decode_steps=2)
    pair, stream = make_pair(shape, seed=27, algo=fa.FA_DECODE_FFT, P=16, max_mid=16384)
    assert fa.fa_launch_count(pair.layout, 2) == 1 and fa.fa_launch_count(pair.layout, 4) == 1
    pair.check_decode(synth.queries(shape, seed=27))
    K, V = stream.tokens(shape.L, shape.L + 2)
    for t in range(2):
        pair.check_step(synth.queries(shape, seed=27, step=t + 1), K[:, t], V[:, t])
    pair.check_state()


@pytest.mark.parametrize("B", [1, 3])
def test_fused_decode_two_ctas_per_sm_cooperative(B):
    """Short transforms with fewer heads than SMs: a head's parts are two to an SM and still wait for one
    another (cooperative launch over 2 x SMs resident CTAs)."""
    shape = SMALL_BF16.with_(B=B, Hq=32, Hkv=16, L=1800, T=2048, M=256, n_full_k=48, n_full_v=32, decode_steps=3)
    pair, stream = make_pair(shape, seed=24, algo=fa.FA_DECODE_FFT, P=16)
    assert fa.fa_launch_count(pair.layout, 2) == 1
    pair.check_decode(synth.queries(shape, seed=24))
    K, V = stream.tokens(shape.L, shape.L + 3)
    for t in range(3):
        pair.check_step(synth.queries(shape, seed=24, step=t + 1), K[:, t], V[:, t])
    pair.check_state()


def test_workspace_counters_must_start_at_zero_and_init_restores_them():
    """A workspace full of garbage is made usable by fa_workspace_init."""
    shape = SMALL_BF16.with_(B=1, Hq=4, Hkv=1, L=500, T=1024, M=64)
    pair, _ = make_pair(shape, seed=19, algo=fa.FA_DECODE_FFT, P=8)
    pair.ws = torch.full((pair.ws.numel(),), 0, dtype=torch.uint8, device="cuda")
    pair.ws[4096:] = 0xAB                                   # scratch beyond the counters may hold anything
    pair.check_decode(synth.queries(shape, seed=19))
    dirty = torch.full((pair.ws.numel(),), 0x5A, dtype=torch.uint8, device="cuda")
    fa.fa_workspace_init(dirty)
    assert not dirty[:4096].any() and bool((dirty[4096:] == 0x5A).all())
    pair.ws = dirty
    pair.check_decode(synth.queries(shape, seed=19, step=1))


def test_bounded_wait_runs_out_reports_timeout_and_workspace_init_recovers():
    """Failure path of the cooperative decode kernel, without faulting or hanging anything: one barrier
    counter of a caller workspace is preset so that the arrivals of the head's parts can never reach the
    number the waiting parts poll for.  Every poll loop is bounded (2^22 polls of ~0.1 us with back-off,
    well under a second per CTA, all CTAs polling at the same time), so the kernel gives up, records
    FA_ERR_TIMEOUT in the cache's status word and returns; the output of that call is undefined.
    fa_workspace_init then restores the workspace and the next call matches the oracle."""
    import time
    shape = SMALL_BF16.with_(B=1, Hq=8, Hkv=2, L=1800, T=2048, M=256, n_full_k=32, n_full_v=32)
    pair, _ = make_pair(shape, seed=31, algo=fa.FA_DECODE_FFT, P=16)
    assert fa.fa_launch_count(pair.layout, 2) == 1            # the fused, cooperative form: its parts wait for one another
    q = synth.queries(shape, seed=31)
    pair.check_decode(q)                                      # a good call first
    counters = pair.ws[:4096].view(torch.int32)
    assert not counters.any()                                 # a good call leaves every counter at zero
    counters[0] = -(1 << 20)                                  # first barrier of (row 0, KV head 0): arrivals cannot reach n
    out = torch.zeros_like(q, device="cuda")
    t0 = time.perf_counter()
    fa.fa_decode_attention(pair.layout, pair.gpu, q.cuda(), out, pair.ws)
    st = fa.fa_poll_status(pair.gpu)                          # synchronises
    waited = time.perf_counter() - t0
    assert st == fa.FA_ERR_TIMEOUT
    assert waited < 20.0, waited
    assert fa.fa_poll_status(pair.gpu) == fa.FA_OK            # the status word is cleared by the poll
    fa.fa_workspace_init(pair.ws)
    pair.check_decode(synth.queries(shape, seed=31, step=1))
    pair.check_decode(q)
    assert not pair.ws[:4096].any()


def test_full_row_in_a_batch_is_refused_alone():
    """Batch of two rows, one whose middle is full and one with room: the push changes nothing in the
    full row (FA_ERR_CAPACITY in the status word) and goes through in the other (oracle: one cache per
    row, since a row is a cache of its own)."""
    import dataclasses
    from oracle import fa_oracle as fo
    from tests.parity_util import oracle_cfg
    shape = SMALL_BF16.with_(B=2, Hq=4, Hkv=1, L=0, L_init=2, L_local=4, T=64, M=16, n_full_k=16, n_full_v=8)
    layout = layout_of(shape, max_mid=8, P=2, algo=fa.FA_DECODE_AUTO)
    stream = synth.KVStream(shape, seed=32)
    K, V = stream.tokens(0, 20)
    lengths = [14, 9]                                         # row 0: 2 + 4 + 8 = full; row 1: three middle tokens
    gpu = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
    ws = fa.new_workspace(layout)
    fa.fa_compress_ragged(layout, gpu, K.cuda(), V.cuda(), lengths, ws)
    refs = []
    for b in range(2):
        r = fo.OracleCache(dataclasses.replace(oracle_cfg(layout), B=1), stream.idx_full_k.numpy(), stream.idx_full_v.numpy())
        r.compress(to64(K[b:b + 1, :lengths[b]]), to64(V[b:b + 1, :lengths[b]]))
        refs.append(r)
    for step, use_step in enumerate((False, True)):
        k_new, v_new = K[:, 15 + step].contiguous(), V[:, 15 + step].contiguous()
        q = synth.queries(shape, seed=32, step=step)
        out = torch.full_like(q, float("nan"), device="cuda")
        if use_step:
            fa.fa_decode_step(layout, gpu, q.cuda(), k_new.cuda(), v_new.cuda(), out, ws)
        else:
            fa.fa_append(layout, gpu, k_new.cuda(), v_new.cuda())
            fa.fa_decode_attention(layout, gpu, q.cuda(), out, ws)
        assert fa.fa_poll_status(gpu) == fa.FA_ERR_CAPACITY   # from row 0
        refs[1].append(to64(k_new[1:2]), to64(v_new[1:2]))    # row 0's oracle cache is left alone: the push was refused
        st = gpu.state.cpu().numpy()
        for b in range(2):
            assert (st[b, 0], st[b, 1], st[b, 2]) == (refs[b].n_init[0], refs[b].n_local[0], refs[b].n_mid[0]), (step, b)
            want = refs[b].decode(to64(q[b:b + 1]))
            assert np.abs(to64(out[b:b + 1]) - want).max() <= 2e-2, (step, b)
            for name in ("coef_k", "coef_v"):
                rc = getattr(refs[b], name)[0]
                assert np.abs(to64(getattr(gpu, name)[b]) - rc).max() <= 1e-3 * max(np.abs(rc).max(), 1e-30), (step, b, name)


def test_multi_layer_step_equals_single_calls_bit_for_bit():
    """fa_decode_step_layers over layers with different schemas (kept dims per layer as in the
    inverted-pyramid schema: more compressed dims in early layers) against one fa_decode_step per
    layer on twin caches: outputs and every cache buffer identical bit for bit, and the first layer
    against the oracle."""
    base = SMALL_BF16.with_(B=2, Hq=8, Hkv=2, L=900, T=1024, M=128, decode_steps=4)
    schemas = [(16, 8), (32, 32), (32, 32), (64, 40)]          # (n_full_k, n_full_v) per layer
    n_layers, steps = len(schemas), 4
    layouts, twins, streams, pair0 = [], [], [], None
    for i, (nfk, nfv) in enumerate(schemas):
        shape = base.with_(n_full_k=nfk, n_full_v=nfv)
        layout = layout_of(shape, max_mid=1024, P=8, algo=fa.FA_DECODE_AUTO)
        stream = synth.KVStream(shape, seed=40 + i, layer=i)
        K, V = stream.tokens(0, shape.L)
        pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
        pair.compress(K, V)
        twin = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)       # a bitwise copy (two compress calls may differ in the last bit)
        for name in ("k_init", "v_init", "k_local", "v_local", "k_mid", "v_mid", "coef_k", "coef_v", "state"):
            getattr(twin, name).copy_(getattr(pair.gpu, name))
        layouts.append(layout); twins.append((pair.gpu, twin)); streams.append((shape, stream))
        if i == 0:
            pair0 = pair
    ws = fa.new_workspace(max(layouts, key=fa.fa_workspace_bytes))
    qs = [torch.empty((2, 8, 128), dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)]
    ks = [torch.empty((2, 2, 128), dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)]
    vs = [torch.empty_like(k) for k in ks]
    outs_a = [torch.full_like(q, float("nan")) for q in qs]
    outs_b = [torch.full_like(q, float("nan")) for q in qs]
    args = fa.LayerStep(layouts, [a for a, _ in twins], qs, ks, vs, outs_a)
    for t in range(steps):
        for i, (shape, stream) in enumerate(streams):
            k_new, v_new = stream.tokens(shape.L + t, shape.L + t + 1)
            qs[i].copy_(synth.queries(shape, seed=40 + i, step=t, layer=i)); ks[i].copy_(k_new[:, 0]); vs[i].copy_(v_new[:, 0])
        fa.fa_decode_step_layers(args, ws)
        for i in range(n_layers):
            fa.fa_decode_step(layouts[i], twins[i][1], qs[i], ks[i], vs[i], outs_b[i], ws)
        torch.cuda.synchronize()
        for i in range(n_layers):
            assert torch.equal(outs_a[i].view(torch.int16), outs_b[i].view(torch.int16)), (t, i)
        pair0.ref.append(to64(ks[0]), to64(vs[0]))
        assert np.abs(to64(outs_a[0]) - pair0.ref.decode(to64(qs[0]))).max() <= 2e-2
    for i, (a, b) in enumerate(twins):
        for name in ("k_init", "v_init", "k_local", "v_local", "k_mid", "v_mid", "coef_k", "coef_v", "state"):
            assert torch.equal(getattr(a, name), getattr(b, name)), (i, name)
    pair0.check_state()


@pytest.mark.parametrize("kw,P", [
    (dict(B=1, Hq=8, Hkv=2, d=128, L=3000, T=4096, M=256, n_full_k=32, n_full_v=32), 16),     # two heads per CTA, two row tiles
    (dict(B=2, Hq=6, Hkv=3, d=128, L=2300, T=4096, M=512, n_full_k=16, n_full_v=48), 32),     # odd head count: one head per CTA; 6-chunk V rows
    (dict(B=1, Hq=4, Hkv=4, d=64, L=1500, T=2048, M=128, n_full_k=8, n_full_v=16), 8),        # one row tile: every token of a block in one CTA
    (dict(B=1, Hq=2, Hkv=2, d=128, L=1400, T=2048, M=128, n_full_k=64, n_full_v=64), 4),      # more chunks than the gather warps hold: partition kernel writes the rows
    (dict(B=1, Hq=2, Hkv=2, d=128, L=1100 + 37, T=2048, M=1024, n_full_k=0, n_full_v=8), 16), # nothing kept of K; ragged last block; idle row-tile CTAs
    (dict(B=6, Hq=4, Hkv=4, d=128, L=1300, T=4096, M=2048, n_full_k=32, n_full_v=16), 16),    # more (batch, head group) units than teams of pairs: a team's blocks run through two or three units
])
def test_tensor_compress_with_its_gather(kw, P):
    """Middles of 1024 tokens and more take the tcgen05 kernel, which also writes the kept-dim rows of the middle
    from the boxes it loads (every row_tiles-th token per CTA): windows, K^mu / V^mu (with V's chunk permutation) and
    counters bit-exact, coefficients within 1e-3, decode on top within the output tolerance."""
    shape = SMALL_BF16.with_(L_init=4, L_local=32, **kw)
    layout = layout_of(shape, max_mid=shape.T, P=P)
    stream = synth.KVStream(shape, seed=61, freq="offgrid")
    pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    K, V = stream.tokens(0, shape.L)
    pair.compress(K, V)
    worst = pair.check_state()
    assert worst <= 1e-3, worst
    pair.check_decode(synth.queries(shape, seed=61))


@pytest.mark.parametrize("kw,P,one_launch", [
    (dict(B=1, Hq=8, Hkv=2, L=1500, T=2048, M=128), 16, True),                       # the fused one-launch step
    (dict(B=4, Hq=16, Hkv=8, L=4200, T=16384, M=512, n_full_k=32, n_full_v=48), 16, False),   # split build; append + decode
])
def test_decode_steps_replay_from_a_cuda_graph(kw, P, one_launch):
    """Three token steps captured in a CUDA graph after an eager pass and replayed (the same three tokens once more):
    every output of the replay and the cache afterwards against the oracle, which takes the six steps in turn."""
    shape = SMALL_BF16.with_(decode_steps=8, **kw)
    pair, stream = make_pair(shape, seed=44, algo=fa.FA_DECODE_FFT, P=P, max_mid=shape.T)
    assert (fa.fa_launch_count(pair.layout, 3) == 1) == one_launch
    K, V = stream.tokens(shape.L, shape.L + 3)
    qs = [synth.queries(shape, seed=44, step=t + 1) for t in range(3)]
    q_dev = [q.cuda().contiguous() for q in qs]
    k_dev = [K[:, t].cuda().contiguous() for t in range(3)]
    v_dev = [V[:, t].cuda().contiguous() for t in range(3)]
    outs = [torch.empty_like(q) for q in q_dev]

    def body():
        for t in range(3):
            fa.fa_decode_step(pair.layout, pair.gpu, q_dev[t], k_dev[t], v_dev[t], outs[t], pair.ws)

    def oracle_pass():
        for t in range(3):
            pair.ref.append(to64(K[:, t]), to64(V[:, t]))
            want = pair.ref.decode(to64(qs[t]))
            assert np.abs(to64(outs[t]) - want).max() <= 2e-2 * max(1.0, float(np.abs(want).max())), t

    body()
    torch.cuda.synchronize()
    oracle_pass()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        body()
    for o in outs:
        o.zero_()
    g.replay()
    torch.cuda.synchronize()
    oracle_pass()
    pair.check_state()


def test_compress_layers_and_decode_replay_from_a_cuda_graph():
    """The call over several layers and a decode call behind it, captured in one CUDA graph after an eager call (which
    sets the kernels' attributes) and replayed: the caches and the output of the replay against the oracle."""
    shape = SMALL_BF16.with_(B=2, Hq=8, Hkv=4, d=128, L=2600, T=4096, M=512, n_full_k=32, n_full_v=16, L_init=4, L_local=64)
    layout = layout_of(shape, max_mid=shape.T, P=16)
    n = 3
    pairs, Ks, Vs = [], [], []
    for i in range(n):
        stream = synth.KVStream(shape, seed=80 + i, freq="offgrid")
        pairs.append(Pair(layout, stream.idx_full_k, stream.idx_full_v))
        K, V = stream.tokens(0, shape.L)
        Ks.append(K)
        Vs.append(V)
    Kc, Vc = [K.cuda() for K in Ks], [V.cuda() for V in Vs]
    qs = synth.queries(shape, seed=80)
    q_dev = qs.cuda().contiguous()
    out = torch.empty_like(q_dev)
    caches, ws = [p.gpu for p in pairs], pairs[0].ws

    def body():
        fa.fa_compress_layers([layout] * n, caches, Kc, Vc, ws)
        fa.fa_decode_attention(layout, caches[n - 1], q_dev, out, ws)

    body()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        body()
    for p in pairs:                                               # the replay has to produce everything again
        p.gpu.coef_k.fill_(7.0)
        p.gpu.k_mid.zero_()
    out.zero_()
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    for i, p in enumerate(pairs):
        p.ref.compress(to64(Ks[i]), to64(Vs[i]))
        worst = p.check_state()
        assert worst <= 1e-3, (i, worst)
    want = pairs[n - 1].ref.decode(to64(qs))
    assert np.abs(to64(out) - want).max() <= 2e-2 * max(1.0, float(np.abs(want).max()))


@pytest.mark.parametrize("kw,P,flags,n_layers", [
    (dict(B=3, Hkv=4, d=64, M=1536, L=1214, n_full_k=8, n_full_v=16, L_init=7, L_local=16), 8, fa.FA_COMPRESS_ORDERED, 2),   # six pairs per team, ordered halves
    (dict(B=2, Hkv=6, d=64, M=256, L=2679, n_full_k=48, n_full_v=8, L_init=0, L_local=16), 8, 0, 2),                         # one pair per team: 74 teams over 6 units
    (dict(B=5, Hkv=2, d=128, M=768, L=3100, n_full_k=16, n_full_v=48, L_init=4, L_local=100), 16, 0, 3),                     # three pairs per team
    (dict(B=1, Hkv=1, d=64, M=256, L=2955, n_full_k=0, n_full_v=32, L_init=0, L_local=64), 8, fa.FA_COMPRESS_ORDERED, 1),    # one head alone (one head per pair)
])
def test_pair_compress_team_cuts(kw, P, flags, n_layers):
    """Shapes that cut the token blocks between teams of CTA pairs in different ways (pairs per team, units per
    team, the order-fixed halves, several layers in one call): every layer's cache against the oracle."""
    shape = SMALL_BF16.with_(Hq=kw["Hkv"], T=8192, **kw)
    layout = layout_of(shape, max_mid=shape.T, P=P)
    pairs, Ks, Vs = [], [], []
    for i in range(n_layers):
        stream = synth.KVStream(shape, seed=90 + i, freq="offgrid")
        pairs.append(Pair(layout, stream.idx_full_k, stream.idx_full_v))
        K, V = stream.tokens(0, shape.L)
        Ks.append(K)
        Vs.append(V)
    if n_layers == 1:
        fa.fa_compress(layout, pairs[0].gpu, Ks[0].cuda(), Vs[0].cuda(), pairs[0].ws, flags=flags)
    else:
        fa.fa_compress_layers([layout] * n_layers, [p.gpu for p in pairs], [K.cuda() for K in Ks], [V.cuda() for V in Vs],
                              pairs[0].ws, flags=flags)
    for i, p in enumerate(pairs):
        p.ref.compress(to64(Ks[i]), to64(Vs[i]))
        worst = p.check_state()
        assert worst <= 1e-3, (i, worst)
    pairs[-1].check_decode(synth.queries(shape, seed=90))


@pytest.mark.parametrize("kw,pair_form", [
    (dict(B=2, Hq=8, Hkv=4, d=128, L=2600, T=4096, M=512, n_full_k=32, n_full_v=16), True),    # partition kernels, then contractions, overlapped
    (dict(B=1, Hq=4, Hkv=2, d=128, L=900, T=2048, M=256, n_full_k=32, n_full_v=32), False),    # short middle: layer after layer
])
def test_compress_layers_against_oracle_and_single_calls(kw, pair_form):
    """fa_compress_layers on four layers with their own inputs and index sets: every layer's cache against the oracle
    (windows, kept-dim rows and counters bit-exact, coefficients within 1e-3), bit-equal in everything but the
    coefficients to a single fa_compress of that layer, the same over repeated calls (the kernels of neighbouring
    layers overlap), and usable by a decode call enqueued right behind it."""
    shape = SMALL_BF16.with_(L_init=4, L_local=64, **kw)
    layout = layout_of(shape, max_mid=shape.T, P=16)
    n = 4
    pairs, Ks, Vs, idx = [], [], [], []
    for i in range(n):
        stream = synth.KVStream(shape, seed=70 + i, freq="offgrid")
        pairs.append(Pair(layout, stream.idx_full_k, stream.idx_full_v))
        idx.append((stream.idx_full_k, stream.idx_full_v))
        K, V = stream.tokens(0, shape.L)
        Ks.append(K)
        Vs.append(V)
    Kc, Vc = [K.cuda() for K in Ks], [V.cuda() for V in Vs]
    qs = synth.queries(shape, seed=70)
    out = torch.empty_like(qs.cuda())
    for rep in range(4):
        fa.fa_compress_layers([layout] * n, [p.gpu for p in pairs], Kc, Vc, pairs[0].ws)
        fa.fa_decode_attention(layout, pairs[n - 1].gpu, qs.cuda(), out, pairs[0].ws)       # right behind the last contraction
        torch.cuda.synchronize()
        if rep == 0:
            first = [(p.gpu.k_mid.clone(), p.gpu.v_mid.clone(), p.gpu.coef_k.clone(), p.gpu.coef_v.clone()) for p in pairs]
            out0 = out.clone()
        else:
            for p, f in zip(pairs, first):
                assert torch.equal(p.gpu.k_mid, f[0]) and torch.equal(p.gpu.v_mid, f[1])
                assert (p.gpu.coef_k - f[2]).abs().max() <= 1e-3 and (p.gpu.coef_v - f[3]).abs().max() <= 1e-3
            assert (out.float() - out0.float()).abs().max() <= 2e-2
    for i, p in enumerate(pairs):
        p.ref.compress(to64(Ks[i]), to64(Vs[i]))
        worst = p.check_state()
        assert worst <= 1e-3, (i, worst)
        single = Pair(layout, *idx[i])
        fa.fa_compress(layout, single.gpu, Kc[i], Vc[i], single.ws)
        for name in ("k_init", "v_init", "k_local", "v_local", "k_mid", "v_mid", "state"):
            assert torch.equal(getattr(single.gpu, name), getattr(p.gpu, name)), (i, name)
    pairs[n - 1].check_decode(qs)
    assert fa.fa_launch_count(layout, 0) == 2 and pair_form == (shape.L - 68 >= 1024)


@pytest.mark.parametrize("shape,P", [(SMALL_BF16, 16), (SMALL_BF16.with_(L=2040, T=2048, M=256), 8), (CFG0, 32),
                                      (CFG0.with_(L_init=4, L_local=64, L=700), 16)])
def test_compress_by_transform_matches_oracle(shape, P):
    """FA_COMPRESS_FFT: the coefficients as the lowest bins of per-class transforms (fp32, no rounded basis):
    windows, kept dims and counters bit-exact as always, coefficients far inside the 1e-3 bar, and the decode
    on top of them within the output tolerance."""
    layout = layout_of(shape, max_mid=shape.T, P=P)
    stream = synth.KVStream(shape, seed=51, freq="offgrid")
    pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    K, V = stream.tokens(0, shape.L)
    fa.fa_compress(layout, pair.gpu, K.cuda(), V.cuda(), pair.ws, flags=fa.FA_COMPRESS_FFT)
    pair.ref.compress(to64(K), to64(V))
    worst = pair.check_state()
    assert worst <= 2e-5, worst
    pair.check_decode(synth.queries(shape, seed=51))


@pytest.mark.parametrize("kw", [dict(B=1, Hq=8, Hkv=2, L=3000, M=256), dict(B=3, Hq=8, Hkv=4, L=3500, M=512)])
def test_ordered_compress_is_bit_reproducible(kw):
    """FA_COMPRESS_ORDERED (the tensor path cuts the tokens of a head in two halves only: a coefficient is zero plus
    two terms, whose sum does not depend on the order of arrival) and FA_COMPRESS_FFT give the same bits on every
    call; both stay within the coefficient tolerance of the oracle."""
    shape = SMALL_BF16.with_(T=4096, n_full_k=32, n_full_v=32, **kw)
    layout = layout_of(shape, max_mid=4096, P=16)
    stream = synth.KVStream(shape, seed=52)
    K, V = stream.tokens(0, shape.L)
    Kc, Vc = K.cuda(), V.cuda()
    for flags in (fa.FA_COMPRESS_ORDERED, fa.FA_COMPRESS_FFT, fa.FA_COMPRESS_ORDERED | fa.FA_COMPRESS_FFT):
        pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
        runs = []
        for _ in range(12):                                   # (also a watch on the barriers across the CTA pairs of the tensor path)
            fa.fa_compress(layout, pair.gpu, Kc, Vc, pair.ws, flags=flags)
            torch.cuda.synchronize()
            runs.append((pair.gpu.coef_k.clone(), pair.gpu.coef_v.clone()))
        for ck, cv in runs[1:]:
            assert torch.equal(ck, runs[0][0]) and torch.equal(cv, runs[0][1]), flags
        pair.ref.compress(to64(K), to64(V))
        pair.check_state()
