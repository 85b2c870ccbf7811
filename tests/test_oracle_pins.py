"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

None of these checks re-types the oracle's own formula: they compare it with
the hand-written Eq.4 fixture, numpy's FFT, closed forms, textbook softmax
attention (torch), brute force through a different route, and invariants.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import fa_oracle as fo

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _cfg(**kw):
    base = dict(B=1, Hq=2, Hkv=1, d=8, n_full_k=2, n_full_v=2, k=4, T=32, L_init=0, L_local=0,
                cap_mid=32, scale=1.0, norm=0)
    base.update(kw)
    return fo.OracleConfig(**base)


def _idx(rng, Hkv, d, n_full):
    return np.stack([np.sort(rng.permutation(d)[:n_full]) for _ in range(Hkv)]).astype(np.int32).reshape(Hkv, n_full)


def _F(T, k, L):
    """Eq.4 as a matrix [2k][L] assembled from oracle columns."""
    return np.stack([fo.basis_column(T, k, j) for j in range(L)], axis=1)


# ------------------------------------------------------------------ basis
def test_eq4_fixture():
    gold = np.loadtxt(os.path.join(GOLD, "eq4_T8_k3.txt"))
    assert gold.shape == (6, 8)
    np.testing.assert_allclose(_F(8, 3, 8), gold, atol=1e-15)


@pytest.mark.parametrize("T,k", [(64, 32), (64, 5), (96, 17), (1024, 32)])
def test_gram_over_full_period(T, k):
    """Rows of F over a full period are orthogonal with squared norms T, 0, T/2, T/2, ..."""
    F = _F(T, k, T)
    gram = F @ F.T
    diag = np.full(2 * k, T / 2.0)
    diag[0], diag[1] = T, 0.0
    np.testing.assert_allclose(gram, np.diag(diag), atol=1e-10 * T)


def test_basis_addition_theorem_at_large_positions():
    """Column j1 + j2 is column j1 rotated by column j2 (angle addition), also where
    n * j overflows 32 bits and exceeds many periods."""
    T, k = 131072, 1024
    for j1, j2 in [(129019, 2052), (65536, 65535), (100003, 31068)]:
        a, b, c = (fo.basis_column(T, k, j) for j in (j1, j2, j1 + j2))
        cos_sum = a[0::2] * b[0::2] - a[1::2] * b[1::2]
        sin_sum = a[1::2] * b[0::2] + a[0::2] * b[1::2]
        np.testing.assert_allclose(c[0::2], cos_sum, atol=1e-12)
        np.testing.assert_allclose(c[1::2], sin_sum, atol=1e-12)
    np.testing.assert_allclose(fo.basis_column(T, k, 7)[0::2] ** 2 + fo.basis_column(T, k, 7)[1::2] ** 2, 1.0, atol=1e-14)
    # periodicity: position j and j + T give the same column
    np.testing.assert_allclose(fo.basis_column(T, k, 5), fo.basis_column(T, k, 5 + T), atol=1e-12)


def test_weights():
    w = fo.weights(_cfg(k=4, T=32))
    np.testing.assert_allclose(w, [1 / 32, 0, 2 / 32, 2 / 32, 2 / 32, 2 / 32, 2 / 32, 2 / 32])
    np.testing.assert_allclose(fo.weights(_cfg(k=4, T=32, norm=1)), np.full(8, 0.25))


# ------------------------------------------------------------ compression
def _compress_case(rng, B=2, Hkv=2, d=8, nfk=3, nfv=2, k=5, T=64, L=50, L_init=2, L_local=7, cap=64, norm=0, Hq=4):
    cfg = _cfg(B=B, Hq=Hq, Hkv=Hkv, d=d, n_full_k=nfk, n_full_v=nfv, k=k, T=T, L_init=L_init,
               L_local=L_local, cap_mid=cap, norm=norm, scale=1.0 / math.sqrt(d))
    cache = fo.OracleCache(cfg, _idx(rng, Hkv, d, nfk), _idx(rng, Hkv, d, nfv))
    K = rng.standard_normal((B, L, Hkv, d))
    V = rng.standard_normal((B, L, Hkv, d))
    cache.compress(K, V)
    return cfg, cache, K, V


def test_partition_and_gather_are_slices():
    """Eq.1-2: windows and kept dims are plain slices of K, V."""
    rng = np.random.default_rng(1)
    cfg, c, K, V = _compress_case(rng)
    L, n_mid = K.shape[1], K.shape[1] - 2 - 7
    assert (c.n_init == 2).all() and (c.n_local == 7).all() and (c.n_mid == n_mid).all()
    for b in range(cfg.B):
        for h in range(cfg.Hkv):
            np.testing.assert_array_equal(c.k_init[b, h], K[b, :2, h])
            np.testing.assert_array_equal(c.v_local[b, h], V[b, L - 7:, h])
            np.testing.assert_array_equal(c.k_mid[b, h, :n_mid], K[b, 2:L - 7, h][:, c.idx_full_k[h]])
            np.testing.assert_array_equal(c.v_mid[b, h, :n_mid], V[b, 2:L - 7, h][:, c.idx_full_v[h]])
    # index sets: disjoint cover, ascending
    for h in range(cfg.Hkv):
        both = np.concatenate([c.idx_full_k[h], c.idx_comp_k[h]])
        assert sorted(both.tolist()) == list(range(cfg.d))
        assert (np.diff(c.idx_comp_k[h]) > 0).all()


def test_coefficients_equal_rfft_of_zero_padded_column():
    """Eq.3: C[2n] = Re rfft(x (+) 0_T)[n], C[2n+1] = -Im rfft(...)[n]."""
    rng = np.random.default_rng(2)
    cfg, c, K, V = _compress_case(rng)
    L = K.shape[1]
    for X, coef, idc in ((K, c.coef_k, c.idx_comp_k), (V, c.coef_v, c.idx_comp_v)):
        for b in range(cfg.B):
            for h in range(cfg.Hkv):
                mid = X[b, 2:L - 7, h][:, idc[h]]                       # [n_mid][d_c]
                spec = np.fft.rfft(mid, n=cfg.T, axis=0)[:cfg.k]        # zero-padded to T
                np.testing.assert_allclose(coef[b, h, 0::2], spec.real, atol=1e-11)
                np.testing.assert_allclose(coef[b, h, 1::2], -spec.imag, atol=1e-11)


def test_coefficients_brute_force_non_power_of_two_period():
    rng = np.random.default_rng(3)
    cfg, c, K, V = _compress_case(rng, T=45, k=7, L=40, L_init=1, L_local=3, cap=45)
    mid = K[0, 1:37, 1][:, c.idx_comp_k[1]]
    want = np.zeros((14, mid.shape[1]))
    for n in range(7):
        for j in range(mid.shape[0]):
            want[2 * n] += math.cos(2 * math.pi * n * j / 45) * mid[j]
            want[2 * n + 1] += math.sin(2 * math.pi * n * j / 45) * mid[j]
    np.testing.assert_allclose(c.coef_k[0, 1], want, atol=1e-11)


def test_short_prompts_fill_init_then_local():
    rng = np.random.default_rng(4)
    for L, want in [(0, (0, 0, 0)), (1, (1, 0, 0)), (2, (2, 0, 0)), (5, (2, 3, 0)), (9, (2, 7, 0)), (10, (2, 7, 1))]:
        cfg, c, K, V = _compress_case(rng, L=L)
        assert (int(c.n_init[0]), int(c.n_local[0]), int(c.n_mid[0])) == want
        if want[2] == 0:
            assert not c.coef_k.any() and not c.coef_v.any()


def test_capacity_error():
    rng = np.random.default_rng(5)
    with pytest.raises(ValueError):
        _compress_case(rng, L=50, cap=10)


# ---------------------------------------------------------- reconstruction
def test_exact_recovery_of_in_span_signal():
    """A signal built from the basis functions over a full period comes back exactly."""
    rng = np.random.default_rng(6)
    T, k, d = 64, 9, 6
    cfg = _cfg(B=1, Hq=1, Hkv=1, d=d, n_full_k=0, n_full_v=0, k=k, T=T, cap_mid=T)
    a = rng.standard_normal((2 * k, d))
    a[1] = 0.0
    X = (_F(T, k, T).T @ a).reshape(1, T, 1, d)
    cache = fo.OracleCache(cfg, np.zeros((1, 0), np.int32), np.zeros((1, 0), np.int32))
    cache.compress(X, 2.0 * X)
    np.testing.assert_allclose(cache.reconstruct(0, 0, 0), X[0, :, 0], atol=1e-12)
    np.testing.assert_allclose(cache.reconstruct(0, 0, 1), 2 * X[0, :, 0], atol=1e-12)


def test_reconstruction_is_truncated_irfft():
    """For n_mid < T the rebuilt column is irfft of the k lowest bins of the zero-padded column."""
    rng = np.random.default_rng(7)
    cfg, c, K, V = _compress_case(rng, T=64, k=11, L=50, L_init=2, L_local=7)
    n_mid = 41
    for side, X, idc, idf in ((0, K, c.idx_comp_k, c.idx_full_k), (1, V, c.idx_comp_v, c.idx_full_v)):
        rec = c.reconstruct(1, 0, side)
        mid = X[1, 2:43, 0]
        spec = np.fft.rfft(mid[:, idc[0]], n=64, axis=0)
        spec[11:] = 0.0
        low = np.fft.irfft(spec, n=64, axis=0)[:n_mid]
        np.testing.assert_allclose(rec[:, idc[0]], low, atol=1e-12)
        np.testing.assert_array_equal(rec[:, idf[0]], mid[:, idf[0]])


def test_full_rank_is_identity_without_nyquist():
    """k = T/2: every signal with no Nyquist component is reproduced."""
    rng = np.random.default_rng(8)
    T, d = 32, 4
    cfg = _cfg(B=1, Hq=1, Hkv=1, d=d, n_full_k=0, n_full_v=0, k=T // 2, T=T, cap_mid=T)
    x = rng.standard_normal((T, d))
    alt = ((-1.0) ** np.arange(T))[:, None]
    x -= alt * (alt * x).mean(axis=0)                       # remove the Nyquist component
    cache = fo.OracleCache(cfg, np.zeros((1, 0), np.int32), np.zeros((1, 0), np.int32))
    cache.compress(x.reshape(1, T, 1, d), x.reshape(1, T, 1, d))
    np.testing.assert_allclose(cache.reconstruct(0, 0, 0), x, atol=1e-12)


def test_paper_scale_is_a_fixed_multiple_of_the_orthogonal_one():
    """1/k instead of (1/T, 2/T): non-constant part scaled by T/2k, constant part by T/k."""
    rng = np.random.default_rng(9)
    outs = {}
    for norm in (0, 1):
        cfg, c, K, V = _compress_case(np.random.default_rng(9), T=64, k=8, norm=norm)
        outs[norm] = (c.reconstruct(0, 1, 0)[:, c.idx_comp_k[1]], c.coef_k[0, 1].copy())
    ortho, coef = outs[0]
    const_part = coef[0] / 64.0
    want = (ortho - const_part) * (64 / 16.0) + const_part * (64 / 8.0)
    np.testing.assert_allclose(outs[1][0], want, atol=1e-12)


# ------------------------------------------------------------------ append
@pytest.mark.parametrize("L0,steps", [(0, 30), (5, 20), (20, 25)])
def test_append_equals_recompress(L0, steps):
    """Eq.5 is exactly additive: compress(L0) + s appends == compress(L0 + s)."""
    rng = np.random.default_rng(10)
    B, Hkv, d, T = 2, 2, 8, 64
    cfg = _cfg(B=B, Hq=4, Hkv=Hkv, d=d, n_full_k=3, n_full_v=2, k=6, T=T, L_init=2, L_local=7, cap_mid=T)
    ik, iv = _idx(rng, Hkv, d, 3), _idx(rng, Hkv, d, 2)
    K = rng.standard_normal((B, L0 + steps, Hkv, d))
    V = rng.standard_normal((B, L0 + steps, Hkv, d))
    a = fo.OracleCache(cfg, ik, iv)
    a.compress(K[:, :L0], V[:, :L0])
    for s in range(steps):
        a.append(K[:, L0 + s], V[:, L0 + s])
    b = fo.OracleCache(cfg, ik, iv)
    b.compress(K, V)
    for name in ("n_init", "n_local", "n_mid", "k_init", "v_init", "k_local", "v_local", "k_mid", "v_mid"):
        np.testing.assert_array_equal(getattr(a, name), getattr(b, name), err_msg=name)
    np.testing.assert_allclose(a.coef_k, b.coef_k, atol=1e-12)
    np.testing.assert_allclose(a.coef_v, b.coef_v, atol=1e-12)


def test_append_without_local_window_and_overflow():
    rng = np.random.default_rng(11)
    cfg = _cfg(B=1, Hq=1, Hkv=1, d=4, n_full_k=1, n_full_v=1, k=2, T=8, L_init=0, L_local=0, cap_mid=8)
    ik = iv = np.array([[2]], np.int32)
    K = rng.standard_normal((1, 8, 1, 4))
    a, b = fo.OracleCache(cfg, ik, iv), fo.OracleCache(cfg, ik, iv)
    a.compress(K[:, :0], K[:, :0])
    for s in range(8):
        a.append(K[:, s], K[:, s])
    b.compress(K, K)
    np.testing.assert_allclose(a.coef_k, b.coef_k, atol=1e-13)
    np.testing.assert_array_equal(a.k_mid, b.k_mid)
    with pytest.raises(ValueError):
        a.append(K[:, 0], K[:, 0])


# --------------------------------------------------------------- attention
def _sdpa(q, K, V, scale):
    """Textbook softmax attention through torch (fp64): q [Hq][d], K, V [Hq][n][d]."""
    out = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[:, None, :], torch.from_numpy(K), torch.from_numpy(V), scale=scale)
    return out[:, 0].numpy()


def test_no_compressed_dims_is_standard_attention():
    rng = np.random.default_rng(12)
    B, Hq, Hkv, d, L = 2, 4, 2, 8, 40
    cfg = _cfg(B=B, Hq=Hq, Hkv=Hkv, d=d, n_full_k=d, n_full_v=d, k=4, T=64, L_init=3, L_local=5,
               cap_mid=64, scale=0.37)
    full = np.tile(np.arange(d, dtype=np.int32), (Hkv, 1))
    cache = fo.OracleCache(cfg, full, full)
    K, V = rng.standard_normal((B, L, Hkv, d)), rng.standard_normal((B, L, Hkv, d))
    q = rng.standard_normal((B, Hq, d))
    cache.compress(K, V)
    out = cache.decode(q)
    for b in range(B):
        Kh = np.repeat(K[b].transpose(1, 0, 2), Hq // Hkv, axis=0)      # GQA: head g -> g // G
        Vh = np.repeat(V[b].transpose(1, 0, 2), Hq // Hkv, axis=0)
        np.testing.assert_allclose(out[b], _sdpa(q[b], Kh, Vh, 0.37), atol=1e-12)


def test_hybrid_attention_against_fft_rebuilt_cache():
    """Whole path (compress, some appends, decode) == textbook attention on a K~, V~ rebuilt
    independently with numpy's rfft/irfft from the ORIGINAL tokens."""
    rng = np.random.default_rng(13)
    B, Hq, Hkv, d, L0, steps, T, k = 2, 6, 2, 8, 30, 12, 64, 7
    L_init, L_local = 2, 5
    cfg = _cfg(B=B, Hq=Hq, Hkv=Hkv, d=d, n_full_k=3, n_full_v=2, k=k, T=T, L_init=L_init, L_local=L_local,
               cap_mid=T, scale=0.5)
    ik, iv = _idx(rng, Hkv, d, 3), _idx(rng, Hkv, d, 2)
    L = L0 + steps
    K, V = rng.standard_normal((B, L, Hkv, d)), rng.standard_normal((B, L, Hkv, d))
    q = rng.standard_normal((B, Hq, d))
    cache = fo.OracleCache(cfg, ik, iv)
    cache.compress(K[:, :L0], V[:, :L0])
    for s in range(steps):
        cache.append(K[:, L0 + s], V[:, L0 + s])
    out = cache.decode(q)

    def rebuilt(X, idx_comp):
        Y = X.copy()                                               # [L][d] of one (b, h)
        mid = X[L_init:L - L_local]
        spec = np.fft.rfft(mid[:, idx_comp], n=T, axis=0)
        spec[k:] = 0.0
        Y[L_init:L - L_local, idx_comp] = np.fft.irfft(spec, n=T, axis=0)[:mid.shape[0]]
        return Y

    G = Hq // Hkv
    for b in range(B):
        Kt = np.stack([rebuilt(K[b, :, g // G], cache.idx_comp_k[g // G]) for g in range(Hq)])
        Vt = np.stack([rebuilt(V[b, :, g // G], cache.idx_comp_v[g // G]) for g in range(Hq)])
        np.testing.assert_allclose(out[b], _sdpa(q[b], Kt, Vt, 0.5), atol=1e-12)


def test_full_rank_hybrid_is_dense_attention_on_original_cache():
    rng = np.random.default_rng(14)
    T, d, Hq = 32, 4, 2
    cfg = _cfg(B=1, Hq=Hq, Hkv=1, d=d, n_full_k=1, n_full_v=1, k=T // 2, T=T, cap_mid=T, scale=0.5)
    x = rng.standard_normal((2, T, d))
    alt = ((-1.0) ** np.arange(T))[None, :, None]
    x -= alt * (alt * x).mean(axis=1, keepdims=True)
    K, V = x[0].reshape(1, T, 1, d), x[1].reshape(1, T, 1, d)
    cache = fo.OracleCache(cfg, np.array([[1]], np.int32), np.array([[3]], np.int32))
    cache.compress(K, V)
    q = rng.standard_normal((1, Hq, d))
    want = _sdpa(q[0], np.repeat(K[0].transpose(1, 0, 2), Hq, 0), np.repeat(V[0].transpose(1, 0, 2), Hq, 0), 0.5)
    np.testing.assert_allclose(cache.decode(q)[0], want, atol=1e-12)


def test_attention_invariants():
    """Outputs are convex combinations of V~ rows; a positive rescale of q with the inverse
    rescale of the softmax scale changes nothing; sampling KV heads leaves the others untouched."""
    rng = np.random.default_rng(15)
    cfg, c, K, V = _compress_case(rng, Hq=4)
    q = rng.standard_normal((cfg.B, cfg.Hq, cfg.d))
    out = c.decode(q)
    G = cfg.Hq // cfg.Hkv
    for b in range(cfg.B):
        for g in range(cfg.Hq):
            h = g // G
            Vt = np.concatenate([c.v_init[b, h], c.reconstruct(b, h, 1), c.v_local[b, h]])
            assert (out[b, g] <= Vt.max(axis=0) + 1e-12).all() and (out[b, g] >= Vt.min(axis=0) - 1e-12).all()
    c2 = fo.OracleCache(fo.OracleConfig(**{**cfg.__dict__, "scale": cfg.scale / 4.0}), c.idx_full_k, c.idx_full_v)
    c2.compress(K, V)
    np.testing.assert_allclose(c2.decode(4.0 * q), out, atol=1e-12)
    part = c.decode(q, heads=(1, 2))
    assert np.isnan(part[:, :G]).all()
    np.testing.assert_array_equal(part[:, G:], out[:, G:])


def test_empty_cache_decodes_to_zero():
    rng = np.random.default_rng(16)
    cfg, c, K, V = _compress_case(rng, L=0)
    assert not c.decode(rng.standard_normal((cfg.B, cfg.Hq, cfg.d))).any()


# --------------------------------------------------------------- selection
def test_dimension_selection_by_reconstruction_error():
    """Sec. 3.4: in-band sinusoid dims rebuild almost exactly, white-noise dims do not."""
    rng = np.random.default_rng(17)
    T, k, d, L = 128, 16, 12, 128
    cfg = _cfg(B=1, Hq=1, Hkv=1, d=d, n_full_k=0, n_full_v=0, k=k, T=T, cap_mid=T)
    smooth = np.sort(rng.permutation(d)[:7])
    t = np.arange(L)[:, None]
    X = rng.standard_normal((L, d))
    for e in smooth:
        X[:, e] = sum(rng.uniform(0.25, 0.75) * np.cos(2 * np.pi * rng.integers(1, k) * t[:, 0] / T + rng.uniform(0, 6.28))
                      for _ in range(4))
    mse = fo.dim_mse(cfg, X.reshape(1, L, 1, d), 0, 0)
    # closed form: the error of a column is its energy outside the k lowest bins (Parseval)
    spec = np.fft.rfft(X, axis=0)
    spec[:k] = 0.0
    np.testing.assert_allclose(mse, (np.fft.irfft(spec, n=T, axis=0) ** 2).mean(axis=0), atol=1e-12)
    idx_full, idx_comp = fo.select_dims(mse, d - 7)
    np.testing.assert_array_equal(idx_comp, smooth)
    assert sorted(np.concatenate([idx_full, idx_comp]).tolist()) == list(range(d))
    # ties: equal errors -> the lower index is compressed first
    f, c_ = fo.select_dims(np.array([1.0, 0.5, 0.5, 0.5, 2.0]), 3)
    np.testing.assert_array_equal(c_, [1, 2])
    np.testing.assert_array_equal(f, [0, 3, 4])
