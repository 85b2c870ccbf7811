"""Per-phase timeline of the decode kernel (debug aid, not part of the hot path).

Needs a timeline build of the library::

    FA_NVCC_EXTRA="-DFA_TIMELINE" python -m paper_2506_11886_b200.build
    python -m paper_2506_11886_b200.timeline [config]

In such a build lane 0 of every consumer warp of the first and of the last CTA of (batch row 0, KV head 0)
stores the SM clock at the phase boundaries of `decode_fft_kernel`; this script runs a few decode calls on a
synthetic cache of the chosen configuration and prints, per stamped warp, the cycles from the CTA's first
stamp to each boundary.  Stamps: 0 entry, 1 set-up done, 2 own u rows written, 3 arrived at the u barrier,
4 q.K of the kept dims done, 5 u of all CTAs visible, 6 u loaded, 7 window tokens done, 8 spectra of the
first class group built, 9 score transform done, 10 softmax done, 11 p.V of the kept dims done, 12 probability
transform done, 13 all class groups folded, 14 output fragments and softmax sums reduced, 15 partial results
written, 16 arrived at the merge barrier, 17 merge barrier passed, 18 merge slice done, 19 ticket taken,
20 (last CTA of the head only) output rows written.  The default build has no stamps and no `fa_debug_timeline` symbol.

With ``--spans`` the script replays a CUDA graph of decode calls instead and prints, per launch, how long the CTAs
ran (entry to exit, in cycles of their SM's clock), how long after entry the wait for the previous kernel returned,
and the gap on one SM between the exit of a CTA of one launch and the entry of a CTA of the next.
"""
import ctypes
import sys

import numpy as np
import torch

from . import fa, synth


def main(cfg: int = 1, calls: int = 6) -> None:
    lib = fa.lib()
    if not hasattr(lib, "fa_debug_timeline"):
        raise SystemExit("this is not a timeline build: rebuild with FA_NVCC_EXTRA=-DFA_TIMELINE")
    shape = synth.CONFIGS[cfg]
    layout = fa.Layout(batch=shape.B, n_q_heads=shape.Hq, n_kv_heads=shape.Hkv, head_dim=shape.d,
                       n_full_k=shape.n_full_k, n_full_v=shape.n_full_v, n_coef=shape.M, period=shape.T,
                       l_init=shape.L_init, l_local=shape.L_local, max_mid=shape.T,
                       mid_classes=shape.T // shape.k, softmax_scale=shape.softmax_scale)
    stream = synth.KVStream(shape, seed=1000, device="cuda")
    K, V = stream.tokens(0, shape.L, work_dtype=torch.float32)
    ws = fa.new_workspace(layout)
    caches = []
    for _ in range(3):                                   # more than one instance: no call finds its cache in L2
        c = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
        fa.fa_compress(layout, c, K, V, ws)
        caches.append(c)
    q = synth.queries(shape, seed=1000, device="cuda")
    out = torch.empty_like(q)
    for i in range(calls):
        fa.fa_decode_attention(layout, caches[i % 3], q, out, ws)
    torch.cuda.synchronize()
    buf = (ctypes.c_longlong * (2 * 8 * 32))()
    lib.fa_debug_timeline.argtypes = [ctypes.c_void_p]
    rc = lib.fa_debug_timeline(buf)
    if rc != 0:
        raise SystemExit(f"fa_debug_timeline: CUDA error {rc}")
    stamps = np.array(buf, dtype=np.int64).reshape(2, 8, 32)
    for cta, name in enumerate(("first CTA of the head", "last CTA of the head")):
        seen = stamps[cta][stamps[cta] > 0]
        if seen.size == 0:
            continue
        t0 = seen.min()
        print(name)
        for w in range(8):
            row = stamps[cta, w]
            print("  warp %d:" % w, " ".join("%d:%d" % (i, row[i] - t0) for i in range(32) if row[i] > 0))


def spans(cfg: int = 1, calls: int = 12) -> None:
    lib = fa.lib()
    if not hasattr(lib, "fa_debug_spans"):
        raise SystemExit("this is not a timeline build: rebuild with FA_NVCC_EXTRA=-DFA_TIMELINE")
    shape = synth.CONFIGS[cfg]
    layout = fa.Layout(batch=shape.B, n_q_heads=shape.Hq, n_kv_heads=shape.Hkv, head_dim=shape.d,
                       n_full_k=shape.n_full_k, n_full_v=shape.n_full_v, n_coef=shape.M, period=shape.T,
                       l_init=shape.L_init, l_local=shape.L_local, max_mid=shape.T,
                       mid_classes=shape.T // shape.k, softmax_scale=shape.softmax_scale)
    stream = synth.KVStream(shape, seed=1000, device="cuda")
    K, V = stream.tokens(0, shape.L, work_dtype=torch.float32)
    ws = fa.new_workspace(layout)
    caches = []
    for _ in range(4):
        c = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v)
        fa.fa_compress(layout, c, K, V, ws)
        caches.append(c)
    q = synth.queries(shape, seed=1000, device="cuda")
    out = torch.empty_like(q)
    for i in range(3):
        fa.fa_decode_attention(layout, caches[i % 4], q, out, ws)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(calls):
            fa.fa_decode_attention(layout, caches[i % 4], q, out, ws)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    print("us per call: %.2f" % (e0.elapsed_time(e1) * 1000 / calls))
    buf = (ctypes.c_longlong * (32 * 160 * 4))()
    lib.fa_debug_spans.argtypes = [ctypes.c_void_p]
    if lib.fa_debug_spans(buf) != 0:
        raise SystemExit("fa_debug_spans failed")
    a = np.array(buf, dtype=np.int64).reshape(32, 160, 4)
    n_cta = int((a[:, :, 1] > 0).any(axis=0).sum())
    order = [slot for slot in np.argsort(a[:, 0, 1]) if a[slot, 0, 1] > 0][-8:]
    prev = None
    for slot in order:
        sm, t_in, t_wait, t_out = (a[slot, :n_cta, i] for i in range(4))
        dur, wait = t_out - t_in, t_wait - t_in
        line = "launch: CTA cycles median %d, wait for the previous kernel returned after median %d" % (np.median(dur), np.median(wait))
        if prev is not None:
            gaps = [t_in[i] - prev[1][np.where(prev[0] == sm[i])[0][0]] for i in range(n_cta) if (prev[0] == sm[i]).any()]
            line += ", same-SM gap exit -> entry median %d" % np.median(gaps)
        print(line)
        prev = (sm, t_out)


if __name__ == "__main__":
    args = [a for a in sys.argv[1:] if a != "--spans"]
    cfg_arg = int(args[0]) if args else 1
    if "--spans" in sys.argv:
        spans(cfg_arg)
    else:
        main(cfg_arg)
