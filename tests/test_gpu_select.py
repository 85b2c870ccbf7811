"""Sec. 3.4 on the GPU (fa_select_dims) against the oracle: index sets bit-exact, errors within tolerance.

The synthetic K / V streams hold, per KV head, in-band sinusoid dims (rebuilt almost exactly from the
coefficients) and white-noise dims (not rebuilt): the error gap between the two groups is many
orders of magnitude, so fp32 / bf16 arithmetic cannot change the ranking across the groups; the number
of kept dims equals the number of noise dims, so the selection is unique."""
import numpy as np
import pytest
import torch

from oracle import fa_oracle as fo
from paper_2506_11886_b200 import fa, synth
from tests.parity_util import layout_of, oracle_cfg, to64

pytestmark = pytest.mark.gpu


def _oracle_selection(layout, K, V):
    cfg = oracle_cfg(layout)
    B, L, H, d = K.shape
    mse = np.zeros((B, H, 2, d))
    for side, X in enumerate((to64(K), to64(V))):
        for b in range(B):
            for h in range(H):
                mse[b, h, side] = fo.dim_mse(cfg, X, b, h)
    sets = []
    for side, n_full in enumerate((layout.n_full_k, layout.n_full_v)):
        full, comp = zip(*(fo.select_dims(mse[:, h, side].mean(axis=0), n_full) for h in range(H)))
        sets += [np.stack(full), np.stack(comp)]
    return sets, mse


@pytest.mark.parametrize("dtype,d,L", [("bf16", 128, 900), ("bf16", 64, 333), ("f32", 128, 300)])
def test_select_dims_matches_oracle(dtype, d, L):
    shape = synth.Shape("sel", B=2, layers=1, Hq=4, Hkv=2, d=d, L=L, dtype=dtype, n_full_k=d // 4, n_full_v=3 * d // 8,
                        M=64, T=1024, L_init=4, L_local=32)
    layout = layout_of(shape, max_mid=1024, P=16)
    stream = synth.KVStream(shape, seed=21)
    K, V = stream.tokens(0, L)
    got = fa.fa_select_dims(layout, K.cuda().contiguous(), V.cuda().contiguous())
    torch.cuda.synchronize()
    want_sets, want_mse = _oracle_selection(layout, K, V)
    names = ("idx_full_k", "idx_comp_k", "idx_full_v", "idx_comp_v")
    for name, g, w in zip(names, got[:4], want_sets):
        np.testing.assert_array_equal(g.cpu().numpy(), w, err_msg=name)
    # the generator's own index sets are what the selection must find
    np.testing.assert_array_equal(got[0].cpu().numpy(), stream.idx_full_k.numpy())
    np.testing.assert_array_equal(got[2].cpu().numpy(), stream.idx_full_v.numpy())
    # errors: relative to the largest error of the row (the well-rebuilt dims sit at the arithmetic's floor)
    g_mse = to64(got[4])
    scale = want_mse.max(axis=-1, keepdims=True)
    assert np.abs(g_mse - want_mse).max() <= 5e-3 * scale.max()
    assert (np.abs(g_mse - want_mse) <= 2e-2 * scale + 1e-6).all()


@pytest.mark.parametrize("Hkv,d,M,L", [(3, 128, 256, 1500), (4, 64, 512, 2000), (2, 128, 128, 129 + 36)])
def test_tensor_core_reconstruction_against_oracle_and_fp32_path(Hkv, d, M, L):
    """bf16 prefill tensors take the tcgen05 reconstruction (several pipeline rounds, a ragged last token tile,
    one or two heads per CTA); the same values handed over as fp32 take the fp32 kernel: both against the oracle."""
    shape = synth.Shape("selt", B=2, layers=1, Hq=Hkv, Hkv=Hkv, d=d, L=L, dtype="bf16", n_full_k=d // 4, n_full_v=d // 2,
                        M=M, T=2048, L_init=4, L_local=32)
    layout = layout_of(shape, max_mid=2048, P=16)
    stream = synth.KVStream(shape, seed=23)
    K, V = stream.tokens(0, L)
    got = fa.fa_select_dims(layout, K.cuda().contiguous(), V.cuda().contiguous())
    shape32 = shape.with_(dtype="f32")
    layout32 = layout_of(shape32, max_mid=2048, P=16)
    got32 = fa.fa_select_dims(layout32, K.float().cuda().contiguous(), V.float().cuda().contiguous())
    torch.cuda.synchronize()
    want_sets, want_mse = _oracle_selection(layout, K, V)
    for g, g32, w in zip(got[:4], got32[:4], want_sets):
        np.testing.assert_array_equal(g.cpu().numpy(), w)
        np.testing.assert_array_equal(g32.cpu().numpy(), w)
    scale = want_mse.max(axis=-1, keepdims=True)
    for g_mse in (to64(got[4]), to64(got32[4])):
        assert (np.abs(g_mse - want_mse) <= 2e-2 * scale + 1e-6).all()
    # the noise dims (errors of the order of the signal) agree closely between the two paths
    big = want_mse > 0.1 * scale
    np.testing.assert_allclose(to64(got[4])[big], to64(got32[4])[big], rtol=5e-3)


def test_select_dims_empty_middle_and_workspace_check():
    shape = synth.Shape("sel0", B=1, layers=1, Hq=2, Hkv=2, d=64, L=20, dtype="bf16", n_full_k=16, n_full_v=8, M=16,
                        T=256, L_init=4, L_local=32)
    layout = layout_of(shape, max_mid=256, P=8)
    stream = synth.KVStream(shape, seed=22)
    K, V = stream.tokens(0, 20)
    got = fa.fa_select_dims(layout, K.cuda().contiguous(), V.cuda().contiguous())
    torch.cuda.synchronize()
    assert not got[4].any()                                                   # no middle: zero errors
    np.testing.assert_array_equal(got[1].cpu().numpy(), np.tile(np.arange(48), (2, 1)))   # lowest indices compressed
    np.testing.assert_array_equal(got[0].cpu().numpy(), np.tile(np.arange(48, 64), (2, 1)))
    assert fa.fa_workspace_bytes(layout) > 0
    import ctypes as C
    out = C.c_size_t(0)
    assert fa.lib().fa_select_workspace_bytes(C.byref(layout.c()), C.byref(out)) == fa.FA_OK and out.value > 0
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    idx = [torch.zeros((2, n), dtype=torch.int32, device="cuda") for n in (16, 48, 8, 56)]
    st = fa.lib().fa_select_dims(C.byref(layout.c()), K.cuda().data_ptr(), V.cuda().data_ptr(), K.stride(0), K.stride(1),
                                 K.stride(2), 20, *[t.data_ptr() for t in idx], None, small.data_ptr(), small.numel(), None)
    assert st == fa.FA_ERR_WORKSPACE
