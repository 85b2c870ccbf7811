"""The allocation-free decode entry point (fixed scratch array inside the library) must give
what fa_decode_attention gives with a caller workspace, and what the oracle computes.  It exists for callers that cannot
allocate device memory at that point: engines whose HBM is fully handed to their own pools,
or decode loops where cudaMalloc (a device-wide synchronisation) is off limits.

Collected last on purpose (file name), so a run that stops at the first failure has already
run every other test.  Passes alone in a fresh process and after the rest of the suite."""
import numpy as np
import pytest
import torch

from paper_2506_11886_b200 import fa, synth
from tests.parity_util import OUT_ABS_BF16, make_pair, to64


def test_layouts_beyond_the_fixed_scratch_are_refused_on_the_host():
    """Host-side check only: nothing is launched for a layout that needs more than the limit."""
    limit = fa.fa_static_workspace_limit()
    assert limit == 8 << 20
    big = fa.Layout(batch=8, n_q_heads=32, n_kv_heads=32, head_dim=128, n_full_k=48, n_full_v=48, n_coef=4096,
                    period=65536, l_init=4, l_local=1024, max_mid=65536, mid_classes=32)
    assert fa.fa_workspace_bytes(big) > limit
    lay = big.c()
    import ctypes as C
    f = fa.lib().fa_decode_attention_static
    f.restype = C.c_int
    assert f(C.byref(lay), None, None, None, None) == fa.FA_ERR_WORKSPACE


@pytest.mark.gpu
def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    shape = synth.Shape("no_alloc_bf16", B=2, layers=1, Hq=8, Hkv=2, d=128, L=1500, dtype="bf16", n_full_k=32,
                        n_full_v=48, M=128, T=2048, L_init=4, L_local=64)
    pair, stream = make_pair(shape, seed=77, max_mid=2048)
    assert fa.fa_workspace_bytes(pair.layout) <= fa.fa_static_workspace_limit()
    for call in range(2):                                    # the second call meets the first one's leftovers
        q = synth.queries(shape, seed=77, step=call).cuda()
        want = torch.full_like(q, float("nan"))
        got = torch.full_like(q, float("nan"))
        fa.fa_decode_attention(pair.layout, pair.gpu, q, want, pair.ws)
        fa.fa_decode_attention_static(pair.layout, pair.gpu, q, got)
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all()
        err = (got.float() - want.float()).abs().max().item()
        assert err <= OUT_ABS_BF16, f"call {call}: {err}"
        ref = pair.ref.decode(to64(q))                       # and against the fp64 oracle on the same cache
        err_ref = np.abs(to64(got) - ref).max()
        assert err_ref <= OUT_ABS_BF16, f"call {call} vs oracle: {err_ref}"
        k_new, v_new = stream.tokens(shape.L + call, shape.L + call + 1)
        pair.append(k_new[:, 0], v_new[:, 0])                # the cache changes between the two calls
    assert fa.fa_poll_status(pair.gpu) == fa.FA_OK


@pytest.mark.gpu
def test_static_scratch_call_clears_stale_barrier_counters():
    """A layout whose decode call is the cooperative kernel, i.e. one that uses the barrier counters in
    the first 4 KiB of the library's array.  The caller has no pointer to that array, so it could not
    re-zero the counters after a call that gave up on a wait: every static call clears them itself in
    front of its kernels.  Two static calls in a row must both match the oracle."""
    shape = synth.Shape("no_alloc_coop", B=1, Hq=8, Hkv=2, layers=1, d=128, L=1800, dtype="bf16", n_full_k=32,
                        n_full_v=32, M=256, T=2048, L_init=4, L_local=64)
    pair, _ = make_pair(shape, seed=78, max_mid=2048, algo=fa.FA_DECODE_FFT, P=16)
    for call in range(2):
        q = synth.queries(shape, seed=78, step=call).cuda()
        got = torch.full_like(q, float("nan"))
        fa.fa_decode_attention_static(pair.layout, pair.gpu, q, got)
        torch.cuda.synchronize()
        assert np.abs(to64(got) - pair.ref.decode(to64(q))).max() <= OUT_ABS_BF16
    assert fa.fa_poll_status(pair.gpu) == fa.FA_OK
