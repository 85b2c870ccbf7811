"""Helpers of the GPU parity tests: feed the same seeded bits to the CUDA
library (through its C ABI binding) and to the fp64 oracle, and compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import fa_oracle as fo
from paper_2506_11886_b200 import fa, synth

# Tolerances of the parity bar.
COEF_REL = 1e-3          # max|C - C_ref| / max|C_ref| per (b, h, K|V) coefficient matrix
OUT_ABS_BF16 = 2e-2      # max abs error of outputs, bf16 I/O, fp32 accumulation, unit-scale inputs
OUT_ABS_F32 = 5e-4       # fp32 I/O: fp32 sums over up to ~1e5 unit-scale terms (see design notes)


def layout_of(shape: synth.Shape, max_mid=None, P=None, algo=fa.FA_DECODE_AUTO, norm=0) -> fa.Layout:
    if P is None:
        P = shape.mid_classes or max(1, shape.T // shape.k)
    if max_mid is None:
        max_mid = min(shape.T, max(0, shape.L - shape.L_init - shape.L_local) + shape.decode_steps + 8)
    return fa.Layout(batch=shape.B, n_q_heads=shape.Hq, n_kv_heads=shape.Hkv, head_dim=shape.d,
                     n_full_k=shape.n_full_k, n_full_v=shape.n_full_v, n_coef=shape.M, period=shape.T,
                     l_init=shape.L_init, l_local=shape.L_local, max_mid=max_mid, mid_classes=P,
                     kv_dtype=fa.FA_F32 if shape.dtype == "f32" else fa.FA_BF16, norm=norm, decode_algo=algo,
                     softmax_scale=shape.softmax_scale)


def oracle_cfg(layout: fa.Layout, heads=None) -> fo.OracleConfig:
    return fo.OracleConfig(B=layout.batch, Hq=layout.n_q_heads, Hkv=layout.n_kv_heads, d=layout.head_dim,
                           n_full_k=layout.n_full_k, n_full_v=layout.n_full_v, k=layout.n_coef // 2, T=layout.period,
                           L_init=layout.l_init, L_local=layout.l_local, cap_mid=max(1, layout.max_mid),
                           scale=layout.softmax_scale, norm=layout.norm)


def unswizzle_v_rows(rows: np.ndarray, slots: np.ndarray, layout: fa.Layout) -> np.ndarray:
    """V^mu rows of bf16 caches are stored with their 16-byte chunks (8 dims) XOR-permuted by a
    function of the slot index (include/fa.h); returns the rows in logical dim order.
    rows: [H][n][n_full_v] in stored order, slots: [n] slot index of each row."""
    nfv = layout.n_full_v
    nch = nfv // 8
    if layout.kv_dtype != fa.FA_BF16 or nch not in (2, 4, 6, 8):
        return rows
    x = {2: (slots >> 2) & 1, 4: (slots >> 1) & 3, 6: (slots >> 2) & 1, 8: slots & 7}[nch]
    out = np.empty_like(rows)
    for c in range(nch):
        pc = c ^ x                                              # physical chunk of logical chunk c, per row
        for val in np.unique(pc):
            sel = pc == val
            out[:, sel, 8 * c:8 * c + 8] = rows[:, sel, 8 * val:8 * val + 8]
    return out


def to64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


class Pair:
    """One CUDA cache and one oracle cache fed with identical inputs."""

    def __init__(self, layout: fa.Layout, idx_full_k, idx_full_v, device="cuda"):
        self.layout = layout
        self.gpu = fa.Cache(layout, idx_full_k, idx_full_v, device=device)
        self.ws = fa.new_workspace(layout, device=device)
        self.ref = fo.OracleCache(oracle_cfg(layout), idx_full_k.numpy(), idx_full_v.numpy())
        fa.fa_validate(layout, self.gpu)

    def compress(self, K: torch.Tensor, V: torch.Tensor):
        fa.fa_compress(self.layout, self.gpu, K.cuda(), V.cuda(), self.ws)
        self.ref.compress(to64(K), to64(V))

    def append(self, k_new: torch.Tensor, v_new: torch.Tensor):
        fa.fa_append(self.layout, self.gpu, k_new.cuda().contiguous(), v_new.cuda().contiguous())
        self.ref.append(to64(k_new), to64(v_new))

    def step(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, heads=None):
        """One fa_decode_step on the CUDA side; append then decode on the oracle side."""
        out = torch.full_like(q, float("nan"), device="cuda")
        fa.fa_decode_step(self.layout, self.gpu, q.cuda().contiguous(), k_new.cuda().contiguous(),
                          v_new.cuda().contiguous(), out, self.ws)
        torch.cuda.synchronize()
        self.ref.append(to64(k_new), to64(v_new))
        return to64(out), self.ref.decode(to64(q), heads=heads)

    def check_step(self, q, k_new, v_new, heads=None, tol=None):
        got, want = self.step(q, k_new, v_new, heads=heads)
        if tol is None:
            tol = OUT_ABS_F32 if self.layout.kv_dtype == fa.FA_F32 else OUT_ABS_BF16
        mask = ~np.isnan(want)
        assert mask.any()
        assert not np.isnan(got[mask]).any()
        err = np.abs(got[mask] - want[mask]).max()
        assert err <= tol, f"output error {err:.3e} > {tol}"
        return err

    def decode(self, q: torch.Tensor, heads=None):
        out = torch.full_like(q, float("nan"), device="cuda")
        fa.fa_decode_attention(self.layout, self.gpu, q.cuda().contiguous(), out, self.ws)
        torch.cuda.synchronize()
        return to64(out), self.ref.decode(to64(q), heads=heads)

    # ---- comparisons ---------------------------------------------------
    def check_state(self):
        """Counters, windows and kept dims bit-exact; coefficients within COEF_REL."""
        L, g, r = self.layout, self.gpu, self.ref
        assert fa.fa_poll_status(g) == fa.FA_OK
        st = g.state.cpu().numpy()
        np.testing.assert_array_equal(st[:, 0], r.n_init)
        np.testing.assert_array_equal(st[:, 1], r.n_local)
        np.testing.assert_array_equal(st[:, 2], r.n_mid)
        assert (st[:, 4] == 0).all()
        for b in range(L.batch):
            ni, nl, nm, head = (int(x) for x in st[b, :4])
            for name in ("k", "v"):
                gi, gl, gm = (to64(getattr(g, f"{name}_{w}")[b]) for w in ("init", "local", "mid"))
                ri, rl, rm = (getattr(r, f"{name}_{w}")[b] for w in ("init", "local", "mid"))
                np.testing.assert_array_equal(gi[:, :ni], ri[:, :ni], err_msg=f"{name}_init")
                if nl:
                    order = (head + np.arange(nl)) % L.l_local
                    np.testing.assert_array_equal(gl[:, order], rl[:, :nl], err_msg=f"{name}_local")
                j = np.arange(nm)
                got_mid = gm[:, j % L.mid_classes, j // L.mid_classes]          # [H][nm][n_full], stored order
                if name == "v":
                    got_mid = unswizzle_v_rows(got_mid, j // L.mid_classes, L)
                np.testing.assert_array_equal(got_mid, rm[:, :nm], err_msg=f"{name}_mid")
        worst = 0.0
        for name in ("coef_k", "coef_v"):
            gc, rc = to64(getattr(g, name)), getattr(r, name)
            if rc.size == 0:
                continue
            for b in range(L.batch):
                for h in range(L.n_kv_heads):
                    den = max(np.abs(rc[b, h]).max(), 1e-30)
                    worst = max(worst, np.abs(gc[b, h] - rc[b, h]).max() / den)
        assert worst <= COEF_REL, f"coefficient error {worst:.3e} > {COEF_REL}"
        return worst

    def check_decode(self, q, heads=None, tol=None):
        got, want = self.decode(q, heads=heads)
        if tol is None:
            tol = OUT_ABS_F32 if self.layout.kv_dtype == fa.FA_F32 else OUT_ABS_BF16
        mask = ~np.isnan(want)
        assert mask.any()
        assert not np.isnan(got[mask]).any()
        err = np.abs(got[mask] - want[mask]).max()
        assert err <= tol, f"output error {err:.3e} > {tol}"
        return err


def make_pair(shape: synth.Shape, seed: int, L=None, algo=fa.FA_DECODE_AUTO, P=None, max_mid=None, freq="grid", norm=0):
    """Stream + compressed pair for a shape (prefill of L tokens)."""
    layout = layout_of(shape, max_mid=max_mid, P=P, algo=algo, norm=norm)
    stream = synth.KVStream(shape, seed=seed, freq=freq)
    pair = Pair(layout, stream.idx_full_k, stream.idx_full_v)
    L = shape.L if L is None else L
    K, V = stream.tokens(0, L)
    pair.compress(K, V)
    return pair, stream
