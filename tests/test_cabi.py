"""The C-ABI library loads on a machine without a GPU and exports every symbol
that include/fa.h declares; host-only entry points behave (no compute calls)."""
import ctypes as C
import os
import re

import pytest

from paper_2506_11886_b200 import build, fa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "fa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fa_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert {"fa_compress", "fa_append", "fa_decode_attention"} <= set(names)
    lib = fa.lib()
    for n in names:
        assert hasattr(lib, n), n


def test_binding_mirrors_the_struct_layouts():
    assert C.sizeof(fa.fa_layout) == 16 * 4
    assert C.sizeof(fa.fa_cache) == 14 * C.sizeof(C.c_void_p)
    assert fa.fa_version() >= 100


def _layout(**kw):
    base = dict(batch=1, n_q_heads=32, n_kv_heads=8, head_dim=128, n_full_k=32, n_full_v=32, n_coef=1024,
                period=32768, l_init=4, l_local=1024, max_mid=32768, mid_classes=64)
    base.update(kw)
    return fa.Layout(**base)


def test_cache_sizes_of_the_32k_configuration():
    sz = fa.fa_cache_sizes_of(_layout())
    assert sz["k_mid"] == 8 * 32768 * 32 * 2 and sz["v_mid"] == sz["k_mid"]
    assert sz["coef_k"] == 8 * 1024 * 96 * 4
    assert sz["k_local"] == 8 * 1024 * 128 * 2 and sz["k_init"] == 8 * 4 * 128 * 2
    assert sz["idx_full_k"] == 8 * 32 * 4 and sz["idx_comp_v"] == 8 * 96 * 4
    assert fa.fa_workspace_bytes(_layout()) > 0


@pytest.mark.parametrize("kw,status", [
    (dict(n_kv_heads=5), fa.FA_ERR_INVALID_ARG),
    (dict(n_coef=1023), fa.FA_ERR_INVALID_ARG),
    (dict(n_coef=65538, period=65536), fa.FA_ERR_INVALID_ARG),
    (dict(max_mid=40000), fa.FA_ERR_INVALID_ARG),
    (dict(mid_classes=0), fa.FA_ERR_INVALID_ARG),
    (dict(softmax_scale=0.0), fa.FA_ERR_INVALID_ARG),
    (dict(kv_dtype=7), fa.FA_ERR_INVALID_ARG),
    (dict(n_full_k=33), fa.FA_ERR_UNSUPPORTED),
    (dict(head_dim=512, n_full_k=32), fa.FA_ERR_UNSUPPORTED),
    (dict(n_q_heads=8 * 32), fa.FA_ERR_UNSUPPORTED),
])
def test_bad_layouts_are_refused_on_the_host(kw, status):
    with pytest.raises(fa.FaError) as e:
        fa.fa_cache_sizes_of(_layout(**kw))
    assert e.value.status == status
    assert fa.status_string(status)


def test_null_arguments():
    lib = fa.lib()
    assert lib.fa_cache_sizes_of(None, None) == fa.FA_ERR_INVALID_ARG
    assert lib.fa_poll_status(None, None) == fa.FA_ERR_INVALID_ARG
    lay = _layout().c()
    assert lib.fa_decode_attention(C.byref(lay), None, None, None, None, 0, None) == fa.FA_ERR_INVALID_ARG
    assert lib.fa_append(C.byref(lay), None, None, None, None) == fa.FA_ERR_INVALID_ARG
    assert lib.fa_compress_layers(-1, None, None, None, None, 0, 0, 0, 0, 0, None, 0, None) == fa.FA_ERR_INVALID_ARG
    assert lib.fa_compress_layers(2, None, None, None, None, 0, 0, 0, 0, 0, None, 0, None) == fa.FA_ERR_INVALID_ARG
    assert lib.fa_compress_layers(0, None, None, None, None, 0, 0, 0, 0, 0, None, 0, None) == fa.FA_OK      # no layers: nothing to do


def test_launch_plan_is_host_logic():
    """Which form a decode call takes is decided on the host from the layout alone: one fused
    kernel (cooperative while a head has several CTAs; with more heads than SMs, one CTA per head in
    waves), three kernels when asked for or when the fused kernel's staging does not fit; the fused
    step (the push riding on the decode launch) needs the fused kernel."""
    lib = fa.lib()

    def launches(what, **kw):
        return lib.fa_launch_count(C.byref(_layout(**kw).c()), what)

    assert launches(0) == 2 and launches(1) == 1
    assert launches(2) == 1 and launches(3) == 1                                   # 8 KV heads: 18 CTAs each; the step is one launch
    assert launches(2, decode_algo=fa.FA_DECODE_FFT_SPLIT) == 3 and launches(3, decode_algo=fa.FA_DECODE_FFT_SPLIT) == 4
    assert launches(2, decode_algo=fa.FA_DECODE_DIRECT) == 3
    assert launches(2, batch=8) == 1                                               # 64 (b, head) pairs: two CTAs each
    assert launches(2, batch=16) == 1                                              # 128 pairs: one CTA each
    assert launches(2, batch=32) == 1                                              # more pairs than SMs: still one CTA each, in waves
    assert launches(2, kv_dtype=fa.FA_F32) == 3                                    # fp32 caches take the direct kernel
    assert launches(3, n_q_heads=64) in (2, 4)                                      # 8 query heads per KV head: two passes
    assert launches(99) == 0
    # plan queries: split build, classes per batch, CTAs per (batch row, KV head)
    assert launches(4) == 0 and launches(5) == 4 and launches(6) == 18             # 32K context: 16 class CTAs of 4 classes + 2 window CTAs
    mha = dict(n_q_heads=32, n_kv_heads=32, batch=8, n_coef=256, period=4096, max_mid=4096, mid_classes=32, l_local=1024, n_full_k=48, n_full_v=48)
    assert launches(2, **mha) == 1 and launches(6, **mha) == 1                     # 256 heads: lone CTAs, two to an SM, still one fused launch
    assert launches(5, **mha) == 32                                                # one query head per KV head: two classes per transform, all 32 in one batch
    assert launches(2, **dict(mha, batch=5)) == 1                                  # 160 heads, all resident at once: stays fused
    long_ctx = dict(batch=4, n_coef=2048, period=131072, max_mid=131072, mid_classes=128, l_local=2048)
    assert launches(4, **long_ctx) == 1 and launches(5, **long_ctx) == 2           # longest transforms: split build, two classes per batch
    # the workspace grows with the number of partial results but stays far below the static limit's order
    small, big = fa.fa_workspace_bytes(_layout()), fa.fa_workspace_bytes(_layout(batch=8))
    assert 0 < small < big


def test_select_workspace_and_null_arguments():
    lib = fa.lib()
    out = C.c_size_t(0)
    lay = _layout().c()
    assert lib.fa_select_workspace_bytes(C.byref(lay), C.byref(out)) == fa.FA_OK
    # coefficients of all 128 dims of K and V: 2 * 8 heads * 1024 rows * 128 dims * 4 bytes, plus windows and scratch
    assert out.value >= 2 * 8 * 1024 * 128 * 4
    assert lib.fa_select_workspace_bytes(C.byref(lay), None) == fa.FA_ERR_INVALID_ARG
    odd = _layout(head_dim=96, n_full_k=32, n_full_v=32).c()
    assert lib.fa_select_workspace_bytes(C.byref(odd), C.byref(out)) == fa.FA_ERR_UNSUPPORTED
    assert lib.fa_select_dims(C.byref(lay), None, None, 0, 0, 0, 5, None, None, None, None, None, None, 0, None) == fa.FA_ERR_INVALID_ARG
    assert lib.fa_decode_step(C.byref(lay), None, None, None, None, None, None, 0, None) == fa.FA_ERR_INVALID_ARG
    assert lib.fa_workspace_init(None, 1 << 20, None) == fa.FA_ERR_WORKSPACE
