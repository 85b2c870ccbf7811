// fa_decode_attention, main kernel for bf16 caches (Eq.6 re-associated): residue-class (FFT)
// evaluation of the compressed dims, tensor-core dot products for the kept dims.
//
// With theta = 2 pi / T, u~_n = u[2n] - i u[2n+1] and the middle tokens of class c,
// j = c + P a (a = 0..S-1, S = T / P >= k):
//   scores   sum_m F[m][j] u[m]  = Re sum_n (u~_n e^{i theta n c}) e^{2 pi i n a / S}
//   outputs  z_n = sum_j p_j e^{i theta n j} = sum_c e^{i theta n c} sum_a p_{c+Pa} e^{2 pi i n a / S}
// so a class costs one length-S transform per side instead of S * k basis terms.  Two query
// heads share one complex transform (real-pair packing); with GH = 4 heads a point holds two
// complex numbers stored (re0, re1, im0, im1) and the transform arithmetic runs on packed fp32
// pairs (add/mul/fma.f32x2).  The score transform is decimation-in-frequency (natural in,
// digit-reversed out), the probability transform decimation-in-time (digit-reversed in, natural
// out), both in place: softmax is pointwise, nothing is reordered.
//
// How a CTA is organised.  All warps are workers; there is no producer warp and no CTA-wide
// barrier inside the token loop.
//   * Every warp owns a private ring of 2 KB shared-memory stages with one mbarrier each and
//     feeds itself: lane 0 issues a bulk (TMA) copy for the next piece of the warp's own work
//     list as soon as the warp has consumed a stage.  The list is static: the warp's rows of C^K
//     (for u), its share of the window rows, then for every class of its team the warp's token
//     range of K^mu and of V^mu, and at the end its rows of C^V.  Loads therefore run ahead of
//     the arithmetic across all phase boundaries.
//   * The warps form teams; a team takes one class at a time through all phases (spectrum,
//     transform, scores, softmax, p^T V, transform, fold) with barriers of its own, so teams
//     drift apart and one team's transform passes fill the issue slots another leaves empty
//     while it waits for memory.  A team keeps its own running maximum, sum, output fragments
//     and z accumulator; the CTA combines them once, in a fixed order.
//   * Scores, probabilities and the p^T V product stay in registers: q . K^T is computed with
//     the heads in the M dimension of mma.sync.m16n8k16, whose accumulator fragment is exactly
//     the B fragment (tokens x heads) that the next product V^T p needs.  Only the transform
//     input / output goes through shared memory.
//   * Window rows (init + local ring) come as [16 rows x 64 dims] TMA boxes with the 128-byte
//     swizzle and are handled warp by warp with an online softmax per warp.
//
// Forms, chosen by the host plan.  Fused (one launch per call): the parts (CTAs) of a (batch
// row, KV head) each form a slice of the rows of u and exchange it through the workspace behind
// a counter barrier, and after a second barrier every part contracts its slice of rows of every
// part's z with its rows of C^V; the last part to take a ticket adds the slices in a fixed
// order and writes the output rows.  A (b, KV head) served by a single part meets nobody: a
// plain launch that may run in waves.  Otherwise three kernels: a prologue kernel forms u, this
// kernel writes per-part partial results (m, l, o, z), an epilogue kernel merges them.
// As the second half of fa_decode_step the fused kernel also adds the pending rank-1 update of
// Eq.5 to the coefficient rows it streams and writes them back.  Every wait is bounded.
//
// "Slot" below is the position of a head inside a point / an mma row: slot s holds head
// hperm(s) = {0, 2, 1, 3}[s] (GH = 4) so that the packed real parts are slots 0, 1 and the
// packed imaginary parts slots 2, 3.
#include <mutex>

#include "fa_decode_ws.cuh"
#include "fa_tmap.cuh"

namespace fa {
namespace {

constexpr int kStageBytes = 2048;          // one piece of a warp's work list
constexpr int kMaxStages = 4;
constexpr int kMaxWarps = 16;
constexpr int kMaxGroups = 8;              // 16-token groups of a class whose scores one warp keeps in registers
constexpr int kWinRows = 16;               // window rows per piece (one [16 x 64] box per 64 dims)
constexpr uint32_t kSpinLimit = 1u << 21;   // polls of a copy's barrier, ~0.1 us apart once backed off: a fraction of a second
using bf16 = __nv_bfloat16;
typedef unsigned long long u64;

// ---- PTX wrappers -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls, records the failure, never hangs.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __noinline__ void mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* fail, int32_t* status) {
    if (*fail) return;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_test_wait(bar, parity)) return;
        if (i > 256) __nanosleep(64);
    }
    *fail = 1;
    atomicExch(status, (int)FA_ERR_TIMEOUT);
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* fail, int32_t* status) {
    if (mbar_try_wait(bar, parity)) return;
    mbar_wait_slow(bar, parity, fail, status);
}
// Eq.4 for one (row, column).
__device__ __noinline__ float basis_value(int m, int j, int T) {
    float cs, sn;
    basis_cs(m >> 1, j, T, &cs, &sn);
    return (m & 1) ? sn : cs;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(bar)
                 : "memory");
}
// One box of a window tensor map: dims x0.., rows y0.., (batch, KV head) z.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int x0, int y0, int z, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(x0), "r"(y0), "r"(z), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void team_sync(int id, int threads) {
    if (threads == 32) __syncwarp();
    else asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Barrier among the CTAs of one (b, KV head, pass) on a global counter (fused kernel only: a
// cooperative launch makes all of them resident).  Arrive: the CTA meets, then one thread fences
// (cumulative over what the others wrote before the meeting) and adds 1 with release semantics.
// Wait: one thread polls with acquire loads, bounded like every other wait of this kernel.
__device__ __forceinline__ void part_arrive(int32_t* cnt, int n, int tid) {
    __syncthreads();
    if (n > 1 && tid == 0) {                              // a part on its own meets nobody: no counter
        __threadfence();
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(cnt) : "memory");
    }
}
__device__ __forceinline__ void part_wait(const int32_t* cnt, int n, int tid, volatile int* fail, int32_t* status) {
    if (n > 1 && tid == 0 && !*fail) {
        bool ok = false;
        for (uint32_t i = 0; i < (1u << 21); ++i) {
            int v;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(cnt) : "memory");
            if (v >= n) { ok = true; break; }
            if (i > 64) __nanosleep(32);
        }
        if (!ok) { *fail = 1; atomicExch(status, (int)FA_ERR_TIMEOUT); }
    }
    __syncthreads();
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t pack_bf16(bf16 lo, bf16 hi) {
    return (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
}
__device__ __forceinline__ uint32_t pack_f2bf(float lo, float hi) {
    return pack_bf16(__float2bfloat16_rn(lo), __float2bfloat16_rn(hi));
}
// cos and sin of 2 pi * frac, frac in [0, 1): hardware approximations on an angle folded into
// [-pi, pi) (absolute error ~5e-7, far below what bf16 operands carry)
__device__ __forceinline__ float2 cis_frac(float frac) {
    const float a = 6.283185307179586f * (frac - (frac >= 0.5f ? 1.0f : 0.0f));
    return make_float2(__cosf(a), __sinf(a));
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- packed reals: N = 2 is an fp32 pair in one 64-bit register, N = 1 a float ---------------
template <int N> struct PR;
template <> struct PR<2> { u64 v; };
template <> struct PR<1> { float v; };
__device__ __forceinline__ PR<2> pk(float a, float b) { PR<2> r; asm("mov.b64 %0, {%1,%2};" : "=l"(r.v) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ void unpk(PR<2> x, float& a, float& b) { asm("mov.b64 {%0,%1}, %2;" : "=f"(a), "=f"(b) : "l"(x.v)); }
__device__ __forceinline__ PR<2> operator+(PR<2> a, PR<2> b) { PR<2> r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ PR<2> operator-(PR<2> a, PR<2> b) { PR<2> r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ PR<2> operator*(PR<2> a, PR<2> b) { PR<2> r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ PR<2> pfma(PR<2> a, PR<2> b, PR<2> c) { PR<2> r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v)); return r; }
__device__ __forceinline__ PR<1> operator+(PR<1> a, PR<1> b) { return PR<1>{a.v + b.v}; }
__device__ __forceinline__ PR<1> operator-(PR<1> a, PR<1> b) { return PR<1>{a.v - b.v}; }
__device__ __forceinline__ PR<1> operator*(PR<1> a, PR<1> b) { return PR<1>{a.v * b.v}; }
__device__ __forceinline__ PR<1> pfma(PR<1> a, PR<1> b, PR<1> c) { return PR<1>{fmaf(a.v, b.v, c.v)}; }
template <int N> __device__ __forceinline__ PR<N> splat(float x);
template <> __device__ __forceinline__ PR<2> splat<2>(float x) { return pk(x, x); }
template <> __device__ __forceinline__ PR<1> splat<1>(float x) { return PR<1>{x}; }

// N complex numbers side by side.
template <int N> struct PC { PR<N> re, im; };
template <int N> __device__ __forceinline__ PC<N> operator+(PC<N> a, PC<N> b) { return PC<N>{a.re + b.re, a.im + b.im}; }
template <int N> __device__ __forceinline__ PC<N> operator-(PC<N> a, PC<N> b) { return PC<N>{a.re - b.re, a.im - b.im}; }
template <int N> __device__ __forceinline__ PC<N> cconj_add(PC<N> a, PC<N> b) { return PC<N>{a.re + b.re, a.im - b.im}; }   // a + conj(b)
// product with one scalar complex w given as splats (wr, wi)
template <int N> __device__ __forceinline__ PC<N> cmulw(PC<N> a, PR<N> wr, PR<N> wi) {
    return PC<N>{(a.re * wr) - (a.im * wi), pfma(a.re, wi, a.im * wr)};
}

// A point of a transform buffer: N = 2 -> float4 (re0, re1, im0, im1), N = 1 -> float2 (re, im).
template <int N> __device__ __forceinline__ PC<N> ld_pt(const float* p);
template <> __device__ __forceinline__ PC<2> ld_pt<2>(const float* p) {
    PC<2> r;
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(r.re.v), "=l"(r.im.v) : "r"(smem_addr(p)) : "memory");
    return r;
}
template <> __device__ __forceinline__ PC<1> ld_pt<1>(const float* p) {
    const float2 x = *reinterpret_cast<const float2*>(p);
    return PC<1>{PR<1>{x.x}, PR<1>{x.y}};
}
__device__ __forceinline__ void st_pt(float* p, PC<2> v) {
    asm volatile("st.shared.v2.b64 [%0], {%1,%2};" ::"r"(smem_addr(p)), "l"(v.re.v), "l"(v.im.v) : "memory");
}
__device__ __forceinline__ void st_pt(float* p, PC<1> v) { *reinterpret_cast<float2*>(p) = make_float2(v.re.v, v.im.v); }

// In-place DFTs with exponent +2 pi i / R, natural order in and out.
template <int N>
__device__ __forceinline__ void dft4(PC<N>& a0, PC<N>& a1, PC<N>& a2, PC<N>& a3) {
    const PC<N> t0 = a0 + a2, t1 = a0 - a2, t2 = a1 + a3, d = a1 - a3;        // i * d = (-d.im, d.re)
    a0 = t0 + t2;
    a2 = t0 - t2;
    a1 = PC<N>{t1.re - d.im, t1.im + d.re};
    a3 = PC<N>{t1.re + d.im, t1.im - d.re};
}
template <int R, int N>
__device__ __forceinline__ void dft(PC<N> (&v)[R]) {
    if constexpr (R == 2) {
        const PC<N> t = v[0];
        v[0] = t + v[1];
        v[1] = t - v[1];
    } else if constexpr (R == 4) {
        dft4(v[0], v[1], v[2], v[3]);
    } else {
        const PR<N> h = splat<N>(0.70710678118654752440f);
        dft4(v[0], v[2], v[4], v[6]);     // even part -> E0..E3
        dft4(v[1], v[3], v[5], v[7]);     // odd part  -> O0..O3
        const PC<N> o1 = PC<N>{(v[3].re - v[3].im) * h, (v[3].re + v[3].im) * h};     // w   O1, w = e^{i pi / 4}
        const PC<N> e0 = v[0], e1 = v[2], e2 = v[4], e3 = v[6], o0 = v[1], o2 = v[5], o3 = v[7];
        v[0] = e0 + o0; v[4] = e0 - o0;
        v[1] = e1 + o1; v[5] = e1 - o1;
        v[2] = PC<N>{e2.re - o2.im, e2.im + o2.re};                                    // + i O2
        v[6] = PC<N>{e2.re + o2.im, e2.im - o2.re};
        const PC<N> w3 = PC<N>{(o3.re + o3.im) * h, (o3.re - o3.im) * h};            // w^3 O3 = (-w3.re, w3.im)
        v[3] = PC<N>{e3.re - w3.re, e3.im + w3.im};
        v[7] = PC<N>{e3.re + w3.re, e3.im - w3.im};
    }
}

// Shared-memory float index of float f of a transform buffer: 16 bytes of padding after every
// 128 bytes, every 1 KB and every 8 KB.  Points stay 16-byte aligned; the strided point accesses
// of the passes and the digit-reversed accesses of token-ordered code all spread over the banks.
__host__ __device__ constexpr int pf(int f) { return f + ((f >> 5) << 2) + ((f >> 8) << 2) + ((f >> 11) << 2); }
__host__ __device__ constexpr int pf_size(int floats) { return pf(floats) + 8; }

// Radix of the pass that handles a sub-transform of length 2^l (8 where possible, two 4s for 16).
__host__ __device__ constexpr int radix_log2(int l) { return (l >= 3 && l != 4) ? 3 : (l >= 2 ? 2 : 1); }

// One in-place pass of radix R = 2^RL over the sub-transforms of length 2^LL of one transform of
// length 2^LS, by the `nthr` threads of a team.  DIF: butterfly, then twiddle the outputs; DIT:
// twiddle the inputs, then butterfly.  The twiddle e^{2 pi i q j / 2^LL} is entry (q j) 2^(LS-LL)
// of the table tws[t] = e^{2 pi i t / S}.
template <int GH, int RL, bool DIT>
__device__ __forceinline__ void fft_pass(float* base, const float2* __restrict__ tws, int LS, int LL, int t, int nthr) {
    constexpr int N = GH / 2;
    constexpr int R = 1 << RL;
    const int STL = LL - RL, PERL = LS - RL;
    const int sh = LS - LL, smask = (1 << LS) - 1;
#pragma unroll 1
    for (int item = t; item < (1 << PERL); item += nthr) {
        const int blk = item >> STL, j = item & ((1 << STL) - 1);
        const int e0 = (blk << LL) + j;
        PC<N> v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = ld_pt<N>(base + pf((e0 + (r << STL)) * GH));
        if (STL > 0 && DIT) {
#pragma unroll
            for (int qq = 1; qq < R; ++qq) {
                const float2 w = tws[((qq * j) << sh) & smask];
                v[qq] = cmulw(v[qq], splat<N>(w.x), splat<N>(w.y));
            }
        }
        dft<R, N>(v);
        if (STL > 0 && !DIT) {
#pragma unroll
            for (int qq = 1; qq < R; ++qq) {
                const float2 w = tws[((qq * j) << sh) & smask];
                v[qq] = cmulw(v[qq], splat<N>(w.x), splat<N>(w.y));
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) st_pt(base + pf((e0 + (r << STL)) * GH), v[r]);
    }
}
// All passes of one transform by a team, a team barrier after each.
template <int GH, bool DIT>
__device__ __forceinline__ void fft_run(float* base, const float2* tws, int LS, int t, int nthr, int bar_id) {
    if (!DIT) {
#pragma unroll 1
        for (int ll = LS; ll > 0;) {
            const int rl = radix_log2(ll);
            if (rl == 3) fft_pass<GH, 3, false>(base, tws, LS, ll, t, nthr);
            else if (rl == 2) fft_pass<GH, 2, false>(base, tws, LS, ll, t, nthr);
            else fft_pass<GH, 1, false>(base, tws, LS, ll, t, nthr);
            team_sync(bar_id, nthr);
            ll -= rl;
        }
    } else {
        // the same radices in reverse order: sub-transform lengths grow from the last DIF length up to 2^LS
        int n = 0;
#pragma unroll 1
        for (int ll = LS; ll > 0; ll -= radix_log2(ll)) ++n;
#pragma unroll 1
        for (int i = n - 1; i >= 0; --i) {
            int ll = LS;
#pragma unroll 1
            for (int j = 0; j < i; ++j) ll -= radix_log2(ll);
            const int rl = radix_log2(ll);
            if (rl == 3) fft_pass<GH, 3, true>(base, tws, LS, ll, t, nthr);
            else if (rl == 2) fft_pass<GH, 2, true>(base, tws, LS, ll, t, nthr);
            else fft_pass<GH, 1, true>(base, tws, LS, ll, t, nthr);
            team_sync(bar_id, nthr);
        }
    }
}

// Position of output index a after the decimation-in-frequency passes of a length-2^LS transform.
__host__ __device__ inline int dif_pos(int LS, int a) {
    int pos = 0;
    for (int cur = LS; cur > 0;) {
        const int rl = radix_log2(cur);
        cur -= rl;
        pos += (a & ((1 << rl) - 1)) << cur;
        a >>= rl;
    }
    return pos;
}

// Physical row ranges of the logical window tokens [t0, t1): init rows, then up to two ring pieces.
struct WinSegs {
    int n;
    int buf[3];      // 0 init, 1 local
    int row[3];      // first physical row
    int cnt[3];      // rows
};
__device__ __forceinline__ WinSegs win_segments(int t0, int t1, int n_init, int n_local, int head, int l_local) {
    WinSegs w;
    w.n = 0;
#pragma unroll
    for (int i = 0; i < 3; ++i) { w.buf[i] = 0; w.row[i] = 0; w.cnt[i] = 0; }
    int a0 = t0, a1 = min(t1, n_init);
    if (a1 > a0) { w.buf[w.n] = 0; w.row[w.n] = a0; w.cnt[w.n] = a1 - a0; ++w.n; }
    int u0 = max(t0 - n_init, 0), u1 = min(t1 - n_init, n_local);
    if (u1 > u0) {
        int ps = (head + u0) % l_local;
        int len1 = min(u1 - u0, l_local - ps);
        w.buf[w.n] = 1; w.row[w.n] = ps; w.cnt[w.n] = len1; ++w.n;
        if (u1 - u0 > len1) { w.buf[w.n] = 1; w.row[w.n] = 0; w.cnt[w.n] = u1 - u0 - len1; ++w.n; }
    }
    return w;
}

// Shared-memory plan of one CTA.
constexpr int kMaxParts = 64;              // parts of one (b, KV head, pass) the merge tables hold
struct TeamSmem {
    int stages_off, tws_off, rev_off, ut_off, team_off, qc_off, xp_off, os_off, red_off, al_off, inv_off, total;
    int fb_floats, team_bytes, zt_off_in_team;
};
__host__ __device__ inline TeamSmem team_smem_layout(int log2S, int k, int GH, int d, int nt, int tw, int nsg) {
    const int S = 1 << log2S;
    TeamSmem L;
    L.fb_floats = pf_size(S * GH);
    int off = 1024;                                        // control page: mbarriers, flags, window segments
    L.stages_off = off; off += nt * tw * nsg * kStageBytes;            // 1024-byte aligned (swizzled window boxes)
    L.tws_off = off; off += 8 * S;
    L.rev_off = off; off += 2 * S;
    off = (off + 15) / 16 * 16;
    L.ut_off = off; off += (8 * k * GH + 15) / 16 * 16;               // (1/2) u~, later w z of the merge
    // a team's area: the transform buffer (also the per-warp slabs [d][GH] of the order-fixed sums), then the team's z
    const int slab_bytes = tw * d * GH * 4;
    L.zt_off_in_team = ((4 * L.fb_floats > slab_bytes ? 4 * L.fb_floats : slab_bytes) + 15) / 16 * 16;
    L.team_bytes = L.zt_off_in_team + (8 * k * GH + 15) / 16 * 16;
    L.team_off = off; off += nt * L.team_bytes;
    L.qc_off = off; off += 4 * GH * d;                     // gathered query of the compressed K dims
    L.xp_off = off; off += 8 * d;                          // fused step: compressed dims of the leaving row
    L.os_off = off; off += 4 * GH * d;                     // o of the windows, then of the whole part
    L.red_off = off; off += 4 * (2 * kMaxWarps * GH + 4 * GH + (kMaxWarps + 8) * GH);
    L.al_off = off; off += 4 * GH * kMaxParts;
    L.inv_off = off; off += 4 * d;
    L.total = (off + 127) / 128 * 128 + 1024;              // slack to align the base to 1024 bytes at run time
    return L;
}

template <int GH> __host__ __device__ constexpr int hperm(int s) { return GH == 4 ? (((s & 1) << 1) | (s >> 1)) : s; }

// ---------------------------------------------------------------------------------------------
// A warp's self-fed ring of stages.  issue() is called by all lanes with the same arguments; lane 0
// acts.  The k-th piece issued lands in stage k % nsg and completes phase (k / nsg) & 1 of its barrier.
struct Ring {
    uint32_t stage0, bar0;     // shared-memory addresses of this warp's first stage / first barrier
    int nsg, issued, taken;
    volatile int* fail;
    int32_t* status;
    __device__ __forceinline__ uint32_t stage_of(int kth) const { return stage0 + (uint32_t)(kth % nsg) * kStageBytes; }
    __device__ __forceinline__ uint32_t bar_of(int kth) const { return bar0 + (uint32_t)(kth % nsg) * 8; }
    __device__ __forceinline__ bool room() const { return issued - taken < nsg; }
    __device__ __forceinline__ void issue_bulk(const void* src, uint32_t bytes, int lane) {
        if (lane == 0) {
            mbar_expect_tx(bar_of(issued), bytes);
            bulk_g2s(stage_of(issued), src, bytes, bar_of(issued));
        }
        ++issued;
    }
    __device__ __forceinline__ void issue_box(const CUtensorMap* tm, int x0, int y0, int z, int lane) {
        if (lane == 0) {
            mbar_expect_tx(bar_of(issued), kStageBytes);
            tma_load_3d(stage_of(issued), tm, x0, y0, z, bar_of(issued));
        }
        ++issued;
    }
    // waits for the oldest piece not yet taken and returns its stage address
    __device__ __forceinline__ uint32_t take() {
        mbar_wait(bar_of(taken), (uint32_t)(taken / nsg) & 1u, fail, status);
        return stage_of(taken);
    }
    __device__ __forceinline__ void done() { __syncwarp(); ++taken; }
};

// The static work list of one warp, walked by the issuing side (all lanes keep the same cursor).
struct Cursor {
    int ph;          // 0 rows of C^K, 1 window rows, 2 classes, 3 rows of C^V, 4 end
    int a, b, c;     // phase-specific position
};

// GH query heads per CTA (2 or 4); OCC CTAs per SM the build is meant for (register cap).
template <int GH, int OCC>
__global__ void __launch_bounds__(OCC == 2 ? 256 : 512, OCC) decode_teams_kernel(
    const __grid_constant__ CUtensorMap tm_ki, const __grid_constant__ CUtensorMap tm_vi,
    const __grid_constant__ CUtensorMap tm_kl, const __grid_constant__ CUtensorMap tm_vl, Dims s, CacheDev c, DecodePlan p,
    const bf16* __restrict__ q, bf16* __restrict__ out, char* wsp, int step) {
    constexpr int N = GH / 2;
    extern __shared__ __align__(128) unsigned char smem_unaligned[];
    unsigned char* sm = smem_unaligned + ((1024u - (smem_addr(smem_unaligned) & 1023u)) & 1023u);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    Ws ws = ws_view(wsp, p);
    const int LS = p.fft_log2, S = 1 << LS;
    const int NT = p.nt, TW = p.tw, NSG = p.nsg;
    const int nwarps = NT * TW, nthreads = nwarps * 32;
    const TeamSmem L = team_smem_layout(LS, s.k, GH, s.d, NT, TW, NSG);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int team = warp / TW, wt = warp - team * TW;
    const int tthreads = TW * 32, ttid = tid - team * tthreads, bar_id = 1 + team;
    const int gq = lane >> 2, tq = lane & 3;              // mma fragment coordinates

    volatile int* fail = reinterpret_cast<volatile int*>(sm + 512);
    volatile int* last_s = fail + 1;
    float2* tws = reinterpret_cast<float2*>(sm + L.tws_off);
    uint16_t* rev = reinterpret_cast<uint16_t*>(sm + L.rev_off);
    float* ut = reinterpret_cast<float*>(sm + L.ut_off);                 // [k] (A.re, A.im, B.re, B.im) x N: (1/2) u~
    float* fbuf = reinterpret_cast<float*>(sm + L.team_off + team * L.team_bytes);      // this team's transform buffer
    float* zt = reinterpret_cast<float*>(sm + L.team_off + team * L.team_bytes + L.zt_off_in_team);   // [k] same packing as ut
    float* qc = reinterpret_cast<float*>(sm + L.qc_off);                 // [GH slots][dck]
    float* xp_s = reinterpret_cast<float*>(sm + L.xp_off);               // [dck + dcv]
    float* o_s = reinterpret_cast<float*>(sm + L.os_off);                // [GH heads][d]
    float* red_m = reinterpret_cast<float*>(sm + L.red_off);             // [warps][GH slots]
    float* red_l = red_m + kMaxWarps * GH;                               // [warps][GH slots]
    float* win_ml = red_l + kMaxWarps * GH;                              // [2][GH slots]: m, l of the windows
    float* cta_ml = win_ml + 2 * GH;                                     // [2][GH slots]: m, l of the part
    float* tred = cta_ml + 2 * GH;                                       // [teams][GH] team maxima, then alpha
    int* inv_s = reinterpret_cast<int*>(sm + L.inv_off);                 // [d]

    const int part = blockIdx.x;                          // partial-result index: class CTAs, then window CTAs
    const bool is_win = part >= p.n_split;
    const int h = blockIdx.y / p.n_pass, pass = blockIdx.y % p.n_pass;
    const int b = blockIdx.z;
    const int g_first = h * s.G + pass * GH;
    const int ng = min(GH, s.G - pass * GH);
    const int log2P = 31 - __clz(s.P);
    const int np = p.n_part;
    const float sl2 = s.scale * kLog2e;

    // ---- set-up that does not depend on the cache: it may overlap the tail of the previous kernel ----
#pragma unroll 1
    for (int i = tid; i < S; i += nthreads) {
        tws[i] = cis_frac((float)i / (float)S);
        rev[i] = (uint16_t)dif_pos(LS, i);
    }
    if (tid == 0) {
        for (int i = 0; i < nwarps * NSG; ++i) mbar_init(smem_addr(sm) + 8 * i, 1);
        *fail = 0;
        *last_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    Ring ring;
    ring.stage0 = smem_addr(sm + L.stages_off) + (uint32_t)(warp * NSG) * kStageBytes;
    ring.bar0 = smem_addr(sm) + 8u * (uint32_t)(warp * NSG);
    ring.nsg = NSG; ring.issued = 0; ring.taken = 0; ring.fail = fail; ring.status = c.status;
    __syncthreads();

    // ---- this warp's work list --------------------------------------------------------------------
    // rows of C^K / C^V of this part, split over the warps (multiples of 4 rows)
    const int m0 = part * (s.M >> 2) / np * 4, m1 = (part + 1) * (s.M >> 2) / np * 4;
    const int rows_w = (((m1 - m0 + nwarps - 1) / nwarps) + 3) & ~3;
    const int ur0 = min(m1, m0 + warp * rows_w), ur1 = min(m1, ur0 + rows_w);
    const int rpp_k = s.dck > 0 ? max(1, kStageBytes / (s.dck * 4)) : 1;      // rows of C^K per piece
    const int rpp_v = s.dcv > 0 ? max(1, kStageBytes / (s.dcv * 4)) : 1;
    const bool do_u = p.fused && s.dck > 0;
    const bool do_cv = p.fused && s.dcv > 0;
    float* ckg = s.dck > 0 ? coef_rows(c.coef_k, s, b, h, s.dck) : nullptr;
    float* cvg = s.dcv > 0 ? coef_rows(c.coef_v, s, b, h, s.dcv) : nullptr;
    const int rowb_k = s.nfk * 2, rowb_v = s.nfv * 2;
    const int pt_k = rowb_k ? min(128, (kStageBytes / rowb_k) & ~15) : 0;     // tokens per piece of K^mu / V^mu
    const int pt_v = rowb_v ? min(128, (kStageBytes / rowb_v) & ~15) : 0;
    const int nhalf = (s.d + 63) >> 6;                                         // 64-dim boxes per window row
    const int R = S / TW;                                                      // tokens of a class per warp

    // Fused step: C^K rows set off before the wait on the previous kernel (the light append kernel, which
    // does not touch the coefficients and triggers this launch only after its own wait).
    Cursor cur;
    cur.ph = do_u ? 0 : 1; cur.a = do_u ? ur0 : 0; cur.b = 0; cur.c = 0;
    int n_init = 0, n_local = 0, n_mid = 0, head = 0, c0 = 0, c1 = 0, wt0 = 0, wt1 = 0;
    bool state_known = false;
    auto n_of_class = [&](int cls) { return cls < n_mid ? (n_mid - cls + s.P - 1) >> log2P : 0; };
    // class of this team in round r, or -1
    auto class_of_round = [&](int r) { const int cls = c0 + team + NT * r; return cls < c1 ? cls : -1; };

    // Issues pieces while the ring has room; `limit_ph`: phases beyond it are not started yet.
    auto feed = [&](int limit_ph) {
#pragma unroll 1
        while (ring.room() && cur.ph <= limit_ph) {
            if (cur.ph == 0) {                                         // rows [a, ..) of C^K
                if (cur.a >= ur1) { cur.ph = 1; cur.a = 0; cur.b = 0; cur.c = 0; continue; }
                const int nr = min(rpp_k, ur1 - cur.a);
                ring.issue_bulk(ckg + (size_t)cur.a * s.dck, (uint32_t)(nr * s.dck * 4), lane);
                cur.a += nr;
            } else if (cur.ph == 1) {                                  // window rows: a = segment, b = row offset, c = sub-piece
                if (!state_known) return;
                const WinSegs sg = win_segments(wt0, wt1, n_init, n_local, head, s.l_local);
                if (cur.a >= sg.n) { cur.ph = 2; cur.a = 0; cur.b = 0; cur.c = 0; continue; }
                const int side = cur.c / nhalf, hf = cur.c - side * nhalf;
                const CUtensorMap* tm = sg.buf[cur.a] == 0 ? (side == 0 ? &tm_ki : &tm_vi) : (side == 0 ? &tm_kl : &tm_vl);
                ring.issue_box(tm, hf * 64, sg.row[cur.a] + cur.b, b * s.Hkv + h, lane);
                if (++cur.c == 2 * nhalf) {
                    cur.c = 0;
                    cur.b += kWinRows;
                    if (cur.b >= sg.cnt[cur.a]) { cur.b = 0; ++cur.a; }
                }
            } else if (cur.ph == 2) {                                  // classes: a = round, b = side, c = token offset in my range
                if (!state_known) return;
                const int cls = is_win ? -1 : class_of_round(cur.a);
                const int n_c = cls >= 0 ? n_of_class(cls) : 0;
                const int lo = wt * R, hi = min(n_c, lo + R);
                if (cls < 0 || n_c == 0) { cur.ph = 3; cur.a = ur0; cur.b = 0; cur.c = 0; continue; }
                const int ptk = cur.b == 0 ? pt_k : pt_v, rowb = cur.b == 0 ? rowb_k : rowb_v;
                if (ptk == 0 || lo + cur.c >= hi) {                    // this side has nothing (more) for me
                    cur.c = 0;
                    if (++cur.b == 2) { cur.b = 0; ++cur.a; }
                    continue;
                }
                const int a0 = lo + cur.c, nt = min(ptk, hi - a0);
                const bf16* src = cur.b == 0 ? mid_row<bf16>(c.k_mid, s, b, h, cls, a0, s.nfk) : mid_row<bf16>(c.v_mid, s, b, h, cls, a0, s.nfv);
                ring.issue_bulk(src, (uint32_t)(nt * rowb), lane);
                cur.c += ptk;
            } else if (cur.ph == 3) {                                  // rows of C^V
                if (!do_cv || cur.a >= ur1) { cur.ph = 4; continue; }
                const int nr = min(rpp_v, ur1 - cur.a);
                ring.issue_bulk(cvg + (size_t)cur.a * s.dcv, (uint32_t)(nr * s.dcv * 4), lane);
                cur.a += nr;
            } else {
                return;
            }
        }
    };
    if (p.fused && step) feed(0);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.fused && !step) feed(0);

    n_init = c.state[kStateStride * b + 0]; n_local = c.state[kStateStride * b + 1];
    n_mid = min(c.state[kStateStride * b + 2], s.max_mid); head = c.state[kStateStride * b + 3];
    c0 = is_win ? 0 : part * s.P / p.n_split;
    c1 = is_win ? 0 : (part + 1) * s.P / p.n_split;
    {
        const int n_win = n_init + n_local;
        // window tokens: spread over the class CTAs, or over CTAs of their own; inside a CTA over its warps in
        // runs of whole pieces
        const int wi = p.n_wsplit ? part - p.n_split : part, wn = p.n_wsplit ? p.n_wsplit : p.n_split;
        const bool has_win = p.n_wsplit ? is_win : true;
        const int w0 = has_win ? wi * n_win / wn : 0, w1 = has_win ? (wi + 1) * n_win / wn : 0;
        const int per = ((((w1 - w0) + nwarps - 1) / nwarps) + kWinRows - 1) / kWinRows * kWinRows;
        wt0 = min(w1, w0 + warp * per);
        wt1 = min(w1, wt0 + per);
    }
    state_known = true;
    const int j_pend = step ? ws.pend_j[b] : -1;

    // gathered query of the compressed K dims, the leaving row of a fused step, dim -> slot of D^vu
    if (do_u) {
        const int32_t* idc_k = c.idx_comp_k + (size_t)h * s.dck;
#pragma unroll 1
        for (int i = tid; i < GH * s.dck; i += nthreads) {
            const int g = i / s.dck, e = i - g * s.dck;
            qc[i] = g < ng ? __bfloat162float(q[((size_t)b * s.Hq + g_first + g) * s.d + idc_k[e]]) : 0.f;
        }
    }
    if (j_pend >= 0) {
        const float* xp = ws.pend + ((size_t)b * s.Hkv + h) * (s.dck + s.dcv);
#pragma unroll 1
        for (int i = tid; i < s.dck + s.dcv; i += nthreads) xp_s[i] = __ldcg(xp + i);
    }
#pragma unroll 1
    for (int i = tid; i < GH * s.d; i += nthreads) o_s[i] = 0.f;
#pragma unroll 1
    for (int e = tid; e < s.d; e += nthreads) inv_s[e] = -1;
    if (tid < 2 * GH) { win_ml[tid] = tid < GH ? kNegBig : 0.f; }
    __syncthreads();
#pragma unroll 1
    for (int e = tid; e < s.nfv; e += nthreads) inv_s[c.idx_full_v[(size_t)h * s.nfv + e]] = e;

    // A fragments of q for the kept K dims (heads in the M dimension: row gq = slot gq = head hperm(gq)).
    // With the contraction index permuted, k-step ks of the 16-byte piece 4 rd + tq of a K row pairs
    // elements (e0, e0 + 1) with a0 and (e0 + 2, e0 + 3) with a2, e0 = 8 piece + 4 ks.
    const int my_head = hperm<GH>(gq & (GH - 1));
    const bool row_on = gq < GH && my_head < ng;
    const bf16* qrow = q + ((size_t)b * s.Hq + g_first + my_head) * s.d;
    const int npk = s.nfk >> 3, nchv = s.nfv >> 3, npw = s.d >> 3;
    uint32_t qk[2][2][2];
    {
        const int32_t* idf_k = c.idx_full_k + (size_t)h * s.nfk;
#pragma unroll
        for (int rd = 0; rd < 2; ++rd)
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const int piece = 4 * rd + tq, e0 = 8 * piece + 4 * ks;
                const bool on = row_on && piece < npk;
                qk[rd][ks][0] = on ? pack_bf16(qrow[idf_k[e0]], qrow[idf_k[e0 + 1]]) : 0u;
                qk[rd][ks][1] = on ? pack_bf16(qrow[idf_k[e0 + 2]], qrow[idf_k[e0 + 3]]) : 0u;
            }
    }
    feed(3);

    // ================================ u = W C^K q, this part's rows ================================
    // u_g[m] = scale * log2(e) * w_m * sum_e C^K[m][e] q_g[D^kc[e]]: eight lanes per row, four rows at a time.
    if (do_u) {
        const int l8 = lane & 7, rg = lane >> 3, nv = s.dck >> 2;
#pragma unroll 1
        for (int r0 = ur0; r0 < ur1; r0 += rpp_k) {
            const int nr = min(rpp_k, ur1 - r0);
            const uint32_t st = ring.take();
#pragma unroll 1
            for (int rr = 0; rr < nr; rr += 4) {
                const int r = r0 + rr + rg;
                const bool on = rr + rg < nr;
                float a[GH];
#pragma unroll
                for (int g = 0; g < GH; ++g) a[g] = 0.f;
                if (on) {
                    const float f = j_pend >= 0 ? basis_value(r, j_pend, s.T) : 0.f;
                    const uint32_t rowa = st + (uint32_t)((rr + rg) * s.dck) * 4;
#pragma unroll 1
                    for (int v = l8; v < nv; v += 8) {
                        uint4 raw = lds128(rowa + 16 * v);
                        float4 x = make_float4(__uint_as_float(raw.x), __uint_as_float(raw.y), __uint_as_float(raw.z), __uint_as_float(raw.w));
                        if (j_pend >= 0) {                 // fused step: rank-1 update of Eq.5 on the way through, written back
                            const float4 y = *reinterpret_cast<const float4*>(xp_s + 4 * v);
                            x.x = fmaf(f, y.x, x.x); x.y = fmaf(f, y.y, x.y); x.z = fmaf(f, y.z, x.z); x.w = fmaf(f, y.w, x.w);
                            *reinterpret_cast<float4*>(ckg + (size_t)r * s.dck + 4 * v) = x;
                        }
#pragma unroll
                        for (int g = 0; g < GH; ++g) {
                            const float4 y = *reinterpret_cast<const float4*>(qc + g * s.dck + 4 * v);
                            a[g] = fmaf(x.x, y.x, fmaf(x.y, y.y, fmaf(x.z, y.z, fmaf(x.w, y.w, a[g]))));
                        }
                    }
                }
#pragma unroll
                for (int g = 0; g < GH; ++g) {
                    a[g] += __shfl_xor_sync(0xffffffffu, a[g], 1);
                    a[g] += __shfl_xor_sync(0xffffffffu, a[g], 2);
                    a[g] += __shfl_xor_sync(0xffffffffu, a[g], 4);
                }
                float mine = a[0];
#pragma unroll
                for (int g = 1; g < GH; ++g) if (l8 == g) mine = a[g];
                if (on && l8 < ng)
                    ws.u[((size_t)b * s.Hq + g_first + l8) * s.M + r] = recon_weight(s.norm, r, s.k, s.T) * sl2 * mine;
            }
            ring.done();
            feed(3);
        }
        part_arrive(ws.bar + 4 * (((size_t)b * s.Hkv + h) * p.n_pass + pass) + 0, np, tid);
    }
    int32_t* bar = ws.bar + 4 * (((size_t)b * s.Hkv + h) * p.n_pass + pass);

    // ================================ window rows, warp by warp ================================
    // Online softmax per warp over its rows; heads in the M dimension for q . K^T, dims in the M dimension
    // for V^T p, whose B fragment is the score fragment itself.
    const uint32_t zero_u = smem_addr(sm + 544);           // 16 bytes of zeros (a chunk past the end of a row)
    if (tid < 4) reinterpret_cast<uint32_t*>(sm + 544)[tid] = 0u;
    float m_run = kNegBig, l_lane = 0.f;                  // of this lane's slot gq (window phase: per warp; classes: per team)
    // per-warp slabs [rows][GH] for order-fixed sums over the warps, in the transform-buffer part of each team's area
    float* slab = reinterpret_cast<float*>(sm + L.team_off + team * L.team_bytes) + (size_t)wt * (s.d * GH);
    const bool cta_has_win = p.n_wsplit ? is_win : (n_init + n_local) > 0;
    if (wt1 > wt0) {
        uint32_t qw[2][2][2][2];                          // [half][chunk of the lane's pair][k-step][a0 / a2]
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
#pragma unroll
            for (int rd = 0; rd < 2; ++rd)
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
                    const int piece = 8 * hf + 2 * tq + rd, e0 = 8 * piece + 4 * ks;
                    const bool on = row_on && piece < npw;
                    qw[hf][rd][ks][0] = on ? pack_bf16(qrow[e0], qrow[e0 + 1]) : 0u;
                    qw[hf][rd][ks][1] = on ? pack_bf16(qrow[e0 + 2], qrow[e0 + 3]) : 0u;
                }
        float accw[8][4];
#pragma unroll
        for (int mt = 0; mt < 8; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) accw[mt][i] = 0.f;
        const WinSegs sg = win_segments(wt0, wt1, n_init, n_local, head, s.l_local);
#pragma unroll 1
        for (int si = 0; si < sg.n; ++si)
#pragma unroll 1
            for (int r0 = 0; r0 < sg.cnt[si]; r0 += kWinRows) {
                const int nt = min(kWinRows, sg.cnt[si] - r0);
                float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};       // tokens 0-7, 8-15
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    if (hf < nhalf) {
                        const uint32_t st = ring.take();
                        // token gq of each octet, chunks 2 tq and 2 tq + 1 of this half (128-byte swizzle: chunk ^ (row & 7))
#pragma unroll
                        for (int rd = 0; rd < 2; ++rd) {
                            const int cj = 2 * tq + rd;
                            {
                                uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
                                if (8 * hf + cj < npw) {
                                    const uint32_t a_lo = st + (uint32_t)gq * 128 + (uint32_t)((cj ^ gq) << 4);
                                    lo = lds128(a_lo);
                                    hi = lds128(a_lo + 8 * 128);
                                }
                                mma_bf16(d0, qw[hf][rd][0][0], 0u, qw[hf][rd][0][1], 0u, lo.x, lo.y);
                                mma_bf16(d0, qw[hf][rd][1][0], 0u, qw[hf][rd][1][1], 0u, lo.z, lo.w);
                                mma_bf16(d1, qw[hf][rd][0][0], 0u, qw[hf][rd][0][1], 0u, hi.x, hi.y);
                                mma_bf16(d1, qw[hf][rd][1][0], 0u, qw[hf][rd][1][1], 0u, hi.z, hi.w);
                            }
                        }
                        ring.done();
                        feed(3);
                    }
                }
                // scores of tokens 2 tq, 2 tq + 1 (octet 0) and 8 + 2 tq, 9 + 2 tq (octet 1) for slot gq
                float sc[4] = {d0[0] * sl2, d0[1] * sl2, d1[0] * sl2, d1[1] * sl2};
                float mx = kNegBig;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tk = (i >> 1) * 8 + 2 * tq + (i & 1);
                    if (tk >= nt) sc[i] = kNegBig;
                    mx = fmaxf(mx, sc[i]);
                }
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);
                const float alpha = ex2(m_run - m_new);
                m_run = m_new;
                float pr[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tk = (i >> 1) * 8 + 2 * tq + (i & 1);
                    pr[i] = (tk < nt && gq < GH) ? ex2(sc[i] - m_new) : 0.f;
                }
                l_lane = l_lane * alpha + (pr[0] + pr[1]) + (pr[2] + pr[3]);
                const uint32_t b0 = pack_f2bf(pr[0], pr[1]), b1 = pack_f2bf(pr[2], pr[3]);
                // rescale the output fragments (slots 2 tq, 2 tq + 1 in the N dimension) when a maximum moved
                const float al = __shfl_sync(0xffffffffu, alpha, ((2 * tq) & 7) * 4), ah = __shfl_sync(0xffffffffu, alpha, ((2 * tq + 1) & 7) * 4);
                if (__any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
                    for (int mt = 0; mt < 8; ++mt) { accw[mt][0] *= al; accw[mt][1] *= ah; accw[mt][2] *= al; accw[mt][3] *= ah; }
                }
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    if (hf < nhalf) {
                        const uint32_t st = ring.take();
                        if (nt < kWinRows) {
                            // rows past the end of the segment hold what follows it in the buffer: zero them (p = 0 does not stop a NaN)
#pragma unroll 1
                            for (int i = lane; i < (kWinRows - nt) * 8; i += 32) {
                                const int rr = nt + (i >> 3);
                                asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(st + (uint32_t)rr * 128 + (uint32_t)((i & 7) << 4)), "r"(0u) : "memory");
                            }
                            __syncwarp();
                        }
                        const int mi = lane >> 3, tok = ((mi >> 1) << 3) + (lane & 7);
#pragma unroll
                        for (int mt = 0; mt < 4; ++mt) {
                            const int chunk = 2 * mt + (mi & 1);                            // of this half
                            if (8 * hf + 2 * mt < npw) {
                                uint32_t af[4];
                                ldmatrix_x4_trans(af, (8 * hf + chunk < npw) ? st + (uint32_t)tok * 128 + (uint32_t)((chunk ^ (tok & 7)) << 4) : zero_u);
                                mma_bf16(accw[4 * hf + mt], af[0], af[1], af[2], af[3], b0, b1);
                            }
                        }
                        if (nt < kWinRows) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        ring.done();
                        feed(3);
                    }
                }
            }
        // this warp's (m, l) per slot and its output fragments [d][GH], unscaled, for the combine below
        l_lane += __shfl_xor_sync(0xffffffffu, l_lane, 1);
        l_lane += __shfl_xor_sync(0xffffffffu, l_lane, 2);
        if (tq == 0 && gq < GH) { red_m[warp * GH + gq] = m_run; red_l[warp * GH + gq] = l_lane; }
        if (2 * tq < GH) {
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                const int e_lo = 16 * mt + gq, e_hi = e_lo + 8;
                if (e_lo < s.d) *reinterpret_cast<float2*>(slab + e_lo * GH + 2 * tq) = make_float2(accw[mt][0], accw[mt][1]);
                if (e_hi < s.d) *reinterpret_cast<float2*>(slab + e_hi * GH + 2 * tq) = make_float2(accw[mt][2], accw[mt][3]);
            }
        }
    } else if (tq == 0 && gq < GH) {
        red_m[warp * GH + gq] = kNegBig;
        red_l[warp * GH + gq] = 0.f;
    }
    const bool has_classes = !is_win && c0 < c1 && n_of_class(c0) > 0;
    // all of u is needed from here on (the window rows above covered the exchange latency)
    if (do_u && !is_win) part_wait(bar + 0, np, tid, fail, c.status);
    else __syncthreads();
    if (cta_has_win) {
        // order-fixed combine of the warps' window results into o_s [GH heads][d] and (m, l) per slot
#pragma unroll 1
        for (int i = tid; i < GH * s.d; i += nthreads) {
            const int g = i / s.d, e = i - g * s.d, sl = hperm<GH>(g);
            float mw = kNegBig;
#pragma unroll 1
            for (int w = 0; w < nwarps; ++w) mw = fmaxf(mw, red_m[w * GH + sl]);
            float v = 0.f;
#pragma unroll 1
            for (int w = 0; w < nwarps; ++w) {
                const float mwv = red_m[w * GH + sl];
                if (mwv > 0.5f * kNegBig) {
                    const float* sw = reinterpret_cast<const float*>(sm + L.team_off + (w / TW) * L.team_bytes) + (size_t)(w % TW) * (s.d * GH);
                    v = fmaf(sw[e * GH + sl], ex2(mwv - mw), v);
                }
            }
            o_s[i] = v;
        }
        if (tid < GH) {
            float mw = kNegBig, lw = 0.f;
#pragma unroll 1
            for (int w = 0; w < nwarps; ++w) mw = fmaxf(mw, red_m[w * GH + tid]);
#pragma unroll 1
            for (int w = 0; w < nwarps; ++w) lw = fmaf(red_l[w * GH + tid], ex2(red_m[w * GH + tid] - mw), lw);
            win_ml[tid] = mw;
            win_ml[GH + tid] = lw;
        }
        __syncthreads();
    }

    // ut[n] = (A.re, A.im, B.re, B.im), A = heads of the real slots, B = heads of the imaginary slots
#pragma unroll 1
    for (int n = tid; n < s.k; n += nthreads) {
        float2 uv[GH];
#pragma unroll
        for (int sl = 0; sl < GH; ++sl) {
            const int g = hperm<GH>(sl);
            uv[sl] = make_float2(0.f, 0.f);
            if (g < ng && s.dck > 0 && has_classes) uv[sl] = __ldcg(reinterpret_cast<const float2*>(ws.u + ((size_t)b * s.Hq + g_first + g) * s.M + 2 * n));
        }
        float* e = ut + n * 2 * GH;
#pragma unroll
        for (int sl = 0; sl < GH; ++sl) {
            const int ab = sl / N, ln = sl - ab * N;
            e[(2 * ab) * N + ln] = 0.5f * uv[sl].x;
            e[(2 * ab + 1) * N + ln] = -0.5f * uv[sl].y;
        }
    }
#pragma unroll 1
    for (int i = ttid; i < 2 * GH * s.k; i += tthreads) zt[i] = 0.f;
    __syncthreads();

    // ================================ middle classes, team by team ================================
    m_run = kNegBig;
    l_lane = 0.f;
    float acc[4][4];                                      // [m-tile of 16 dims][mma D fragment]: dims x slots
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
    {
        const int nmt = (s.nfv + 15) >> 4;
        // per-lane constants of the V product: a group of 16 tokens starts at a multiple of 16, so the chunk
        // swizzle of a lane's row depends on the lane alone.  A chunk past the end of the row reads the zero block.
        uint32_t v_off[4], v_mul[4];
        {
            const int mi = lane >> 3, tok = ((mi >> 1) << 3) + (lane & 7), sw = v_swz(tok, nchv);
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const int chunk = 2 * mt + (mi & 1);
                v_mul[mt] = chunk < nchv ? 1u : 0u;
                v_off[mt] = chunk < nchv ? (uint32_t)(tok * rowb_v + 16 * (chunk ^ sw)) : zero_u;
            }
        }
        float* tmax = tred + team * (TW + 1) * GH;              // [TW][GH] maxima of the team's warps, then [GH] alpha
        float* talpha = tmax + TW * GH;
        const int lo = wt * R;
        const PC<N> czero = PC<N>{splat<N>(0.f), splat<N>(0.f)};
        auto ld_entry = [&](const float* tab, int n, PC<N>& A, PC<N>& B) {
            if constexpr (N == 2) {
                const float4 x = *reinterpret_cast<const float4*>(tab + n * 8), y = *reinterpret_cast<const float4*>(tab + n * 8 + 4);
                A = PC<N>{pk(x.x, x.y), pk(x.z, x.w)};
                B = PC<N>{pk(y.x, y.y), pk(y.z, y.w)};
            } else {
                const float4 x = *reinterpret_cast<const float4*>(tab + n * 4);
                A = PC<N>{PR<1>{x.x}, PR<1>{x.y}};
                B = PC<N>{PR<1>{x.z}, PR<1>{x.w}};
            }
        };
        auto st_entry = [&](float* tab, int n, const PC<N>& A, const PC<N>& B) {
            if constexpr (N == 2) {
                float a0, a1, a2, a3, b0, b1, b2, b3;
                unpk(A.re, a0, a1); unpk(A.im, a2, a3); unpk(B.re, b0, b1); unpk(B.im, b2, b3);
                *reinterpret_cast<float4*>(tab + n * 8) = make_float4(a0, a1, a2, a3);
                *reinterpret_cast<float4*>(tab + n * 8 + 4) = make_float4(b0, b1, b2, b3);
            } else {
                *reinterpret_cast<float4*>(tab + n * 4) = make_float4(A.re.v, A.im.v, B.re.v, B.im.v);
            }
        };
        auto tw_class = [&](int n, int cls) -> float2 { return cis_frac((float)((n * cls) & (s.T - 1)) / (float)s.T); };

#pragma unroll 1
        for (int round = 0;; ++round) {
            const int cls = is_win ? -1 : class_of_round(round);
            if (cls < 0) break;
            const int n_c = n_of_class(cls);
            if (n_c == 0) break;                           // classes are filled in order: nothing further on
            const int hi = min(n_c, lo + R);

            // ---- kept dims: kd[group][i] = scale log2(e) (q_u . K^mu) of tokens lo + 16 group + {2 tq, 2 tq + 1, 8 + 2 tq, 9 + 2 tq}, slot gq
            float kd[kMaxGroups][4];
            {
                uint32_t st = 0;
#pragma unroll
                for (int gi = 0; gi < kMaxGroups; ++gi) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) kd[gi][i] = 0.f;
                    const int a = lo + 16 * gi;
                    if (pt_k && a < hi) {
                        const int in_piece = (16 * gi) % pt_k;
                        if (in_piece == 0) st = ring.take();
                        float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
                        const uint32_t row_lo = st + (uint32_t)((in_piece + gq) * rowb_k) + 16u * tq;
#pragma unroll
                        for (int rd = 0; rd < 2; ++rd) {
                            if (4 * rd < npk) {
                                uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
                                if (4 * rd + tq < npk) {
                                    x0 = lds128(row_lo + 64u * rd);
                                    x1 = lds128(row_lo + 64u * rd + 8u * rowb_k);
                                }
                                mma_bf16(d0, qk[rd][0][0], 0u, qk[rd][0][1], 0u, x0.x, x0.y);
                                mma_bf16(d0, qk[rd][1][0], 0u, qk[rd][1][1], 0u, x0.z, x0.w);
                                mma_bf16(d1, qk[rd][0][0], 0u, qk[rd][0][1], 0u, x1.x, x1.y);
                                mma_bf16(d1, qk[rd][1][0], 0u, qk[rd][1][1], 0u, x1.z, x1.w);
                            }
                        }
                        kd[gi][0] = d0[0] * sl2; kd[gi][1] = d0[1] * sl2; kd[gi][2] = d1[0] * sl2; kd[gi][3] = d1[1] * sl2;
                        if (in_piece + 16 >= pt_k || a + 16 >= hi) { ring.done(); feed(3); }
                    }
                }
            }

            // ---- packed Hermitian spectrum of the class: X_m = V^A_m + i V^B_m per complex lane,
            // V_m = v_m + conj(v_{S-m}), v_n = (1/2) u~_n e^{i theta n c}.  Pair 0 is bins (0, S/2).
            team_sync(bar_id, tthreads);                   // the fold of the previous class has read the buffer
            if (s.dck > 0) {
#pragma unroll 1
                for (int pr = ttid; pr < S / 2; pr += tthreads) {
                    const int m = pr, mc = pr == 0 ? S / 2 : S - pr;
                    PC<N> Am = czero, Bm = czero, Ac = czero, Bc = czero;
                    if (m < s.k) ld_entry(ut, m, Am, Bm);
                    if (mc < s.k) ld_entry(ut, mc, Ac, Bc);
                    const float2 twm = tw_class(m, cls), twc = tw_class(mc, cls);
                    const PR<N> wmr = splat<N>(twm.x), wmi = splat<N>(twm.y), wcr = splat<N>(twc.x), wci = splat<N>(twc.y);
                    const PC<N> vAm = cmulw(Am, wmr, wmi), vBm = cmulw(Bm, wmr, wmi);
                    const PC<N> vAc = cmulw(Ac, wcr, wci), vBc = cmulw(Bc, wcr, wci);
                    if (pr != 0) {
                        const PC<N> VA = cconj_add(vAm, vAc), VB = cconj_add(vBm, vBc);
                        st_pt(fbuf + pf(m * GH), PC<N>{VA.re - VB.im, VA.im + VB.re});        // V^A + i V^B
                        st_pt(fbuf + pf(mc * GH), PC<N>{VA.re + VB.im, VB.re - VA.im});       // conj(V^A) + i conj(V^B)
                    } else {                                                                   // self-conjugate bins
                        const PC<N> VA0 = cconj_add(vAm, vAm), VB0 = cconj_add(vBm, vBm);
                        const PC<N> VA1 = cconj_add(vAc, vAc), VB1 = cconj_add(vBc, vBc);
                        st_pt(fbuf + pf(0), PC<N>{VA0.re - VB0.im, VA0.im + VB0.re});
                        st_pt(fbuf + pf((S / 2) * GH), PC<N>{VA1.re - VB1.im, VA1.im + VB1.re});
                    }
                }
                team_sync(bar_id, tthreads);
                fft_run<GH, false>(fbuf, tws, LS, ttid, tthreads, bar_id);            // score of slot a at point rev[a]
            } else {
#pragma unroll 1
                for (int i = ttid; i < L.fb_floats; i += tthreads) fbuf[i] = 0.f;
                team_sync(bar_id, tthreads);
            }

            // ---- full scores of my tokens (compressed part from the transform + kept part), team maximum
            float mx = kNegBig;
#pragma unroll
            for (int gi = 0; gi < kMaxGroups; ++gi) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tok = lo + 16 * gi + (i >> 1) * 8 + 2 * tq + (i & 1);
                    if (16 * gi < R) {
                        if (tok < hi && gq < GH) {
                            kd[gi][i] += fbuf[pf(rev[tok] * GH + gq)];
                            mx = fmaxf(mx, kd[gi][i]);
                        } else {
                            kd[gi][i] = kNegBig;
                        }
                    }
                }
            }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            if (tq == 0 && gq < GH) tmax[wt * GH + gq] = mx;
            team_sync(bar_id, tthreads);
            if (gq < GH) {
#pragma unroll 1
                for (int w = 0; w < TW; ++w) mx = fmaxf(mx, tmax[w * GH + gq]);
            }
            const float m_new = fmaxf(m_run, mx);
            const float alpha = ex2(m_run - m_new);
            m_run = m_new;
            l_lane *= alpha;
            if (wt == 0 && tq == 0 && gq < GH) talpha[gq] = alpha;
            // ---- probabilities: fp32 into the transform buffer (every point of it, zeros past the class's end), kept in kd for the V product
#pragma unroll
            for (int gi = 0; gi < kMaxGroups; ++gi) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tok = lo + 16 * gi + (i >> 1) * 8 + 2 * tq + (i & 1);
                    if (16 * gi < R) {
                        const float pv = (tok < hi && gq < GH) ? ex2(kd[gi][i] - m_new) : 0.f;
                        kd[gi][i] = pv;
                        l_lane += pv;
                        if (gq < GH) fbuf[pf(rev[tok] * GH + gq)] = pv;
                    }
                }
            }
            {
                const float al = __shfl_sync(0xffffffffu, alpha, ((2 * tq) & 7) * 4), ah = __shfl_sync(0xffffffffu, alpha, ((2 * tq + 1) & 7) * 4);
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) { acc[mt][0] *= al; acc[mt][1] *= ah; acc[mt][2] *= al; acc[mt][3] *= ah; }
            }
            team_sync(bar_id, tthreads);

            // ---- z_n = alpha z_n + e^{i theta n c} Y_n, Y = transform of the packed probabilities
            if (s.dcv > 0) {
                fft_run<GH, true>(fbuf, tws, LS, ttid, tthreads, bar_id);
                PR<N> alA, alB;
                if constexpr (N == 2) { alA = pk(talpha[0], talpha[1]); alB = pk(talpha[2], talpha[3]); }
                else { alA = PR<1>{talpha[0]}; alB = PR<1>{talpha[1]}; }
                const PR<N> half = splat<N>(0.5f);
#pragma unroll 1
                for (int pr = ttid; pr < S / 2; pr += tthreads) {
                    const int m = pr, mc = pr == 0 ? S / 2 : S - pr;
                    if (m >= s.k && mc >= s.k) continue;
                    const float2 twm = tw_class(m, cls), twc = tw_class(mc, cls);
                    const PC<N> ya = ld_pt<N>(fbuf + pf(m * GH)), yb = ld_pt<N>(fbuf + pf(mc * GH));
                    const PR<N> wmr = splat<N>(twm.x), wmi = splat<N>(twm.y), wcr = splat<N>(twc.x), wci = splat<N>(twc.y);
                    PC<N> zAm, zBm, zAc, zBc;
                    if (pr != 0) {
                        // real slots: y0 = (ya + conj(yb)) / 2, imaginary slots: y1 = (ya - conj(yb)) / (2 i); bin mc holds the conjugates
                        const PC<N> y0 = PC<N>{(ya.re + yb.re) * half, (ya.im - yb.im) * half};
                        const PC<N> y1 = PC<N>{(ya.im + yb.im) * half, (yb.re - ya.re) * half};
                        zAm = cmulw(y0, wmr, wmi);
                        zBm = cmulw(y1, wmr, wmi);
                        zAc = cmulw(PC<N>{y0.re, splat<N>(0.f) - y0.im}, wcr, wci);
                        zBc = cmulw(PC<N>{y1.re, splat<N>(0.f) - y1.im}, wcr, wci);
                    } else {
                        // bins 0 and S/2 are real for each real sequence: (re, im) of the packed value are the two heads
                        zAm = cmulw(PC<N>{ya.re, splat<N>(0.f)}, wmr, wmi);
                        zBm = cmulw(PC<N>{ya.im, splat<N>(0.f)}, wmr, wmi);
                        zAc = cmulw(PC<N>{yb.re, splat<N>(0.f)}, wcr, wci);
                        zBc = cmulw(PC<N>{yb.im, splat<N>(0.f)}, wcr, wci);
                    }
                    if (m < s.k) {
                        PC<N> A, B;
                        ld_entry(zt, m, A, B);
                        st_entry(zt, m, PC<N>{pfma(A.re, alA, zAm.re), pfma(A.im, alA, zAm.im)},
                                 PC<N>{pfma(B.re, alB, zBm.re), pfma(B.im, alB, zBm.im)});
                    }
                    if (mc < s.k) {
                        PC<N> A, B;
                        ld_entry(zt, mc, A, B);
                        st_entry(zt, mc, PC<N>{pfma(A.re, alA, zAc.re), pfma(A.im, alA, zAc.im)},
                                 PC<N>{pfma(B.re, alB, zBc.re), pfma(B.im, alB, zBc.im)});
                    }
                }
            }

            // ---- o^u[dim][slot] += V^mu^T p, 16 tokens per mma, p straight from the registers
            if (pt_v) {
                uint32_t st = 0;
#pragma unroll
                for (int gi = 0; gi < kMaxGroups; ++gi) {
                    const int a = lo + 16 * gi;
                    if (a < hi) {
                        const int in_piece = (16 * gi) % pt_v;
                        if (in_piece == 0) st = ring.take();
                        const int rem = hi - a;
                        if (rem < 16) {
                            // rows past the end of the class hold stale bytes: zero them (p = 0 does not stop a NaN)
#pragma unroll 1
                            for (int i = lane; i < (16 - rem) * nchv; i += 32) {
                                const int rr = in_piece + rem + i / nchv;
                                asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(st + (uint32_t)(rr * rowb_v) + (uint32_t)((i % nchv) << 4)), "r"(0u) : "memory");
                            }
                            __syncwarp();
                        }
                        const uint32_t gbase = st + (uint32_t)(in_piece * rowb_v);
                        const uint32_t b0 = gq < GH ? pack_f2bf(kd[gi][0], kd[gi][1]) : 0u, b1 = gq < GH ? pack_f2bf(kd[gi][2], kd[gi][3]) : 0u;
#pragma unroll
                        for (int mt = 0; mt < 4; ++mt) {
                            if (mt < nmt) {
                                uint32_t af[4];
                                ldmatrix_x4_trans(af, v_off[mt] + gbase * v_mul[mt]);
                                mma_bf16(acc[mt], af[0], af[1], af[2], af[3], b0, b1);
                            }
                        }
                        if (in_piece + 16 >= pt_v || a + 16 >= hi) {
                            if (rem < 16) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            ring.done();
                            feed(3);
                        }
                    }
                }
            }
        }
    }

    // ================================ combine the teams (and the windows) ================================
    __syncthreads();                                       // every team is done with its transform buffer
    l_lane += __shfl_xor_sync(0xffffffffu, l_lane, 1);
    l_lane += __shfl_xor_sync(0xffffffffu, l_lane, 2);
    if (tq == 0 && gq < GH) { red_m[warp * GH + gq] = m_run; red_l[warp * GH + gq] = l_lane; }
    if (2 * tq < GH) {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            const int e_lo = 16 * mt + gq, e_hi = e_lo + 8;
            if (e_lo < s.nfv) *reinterpret_cast<float2*>(slab + e_lo * GH + 2 * tq) = make_float2(acc[mt][0], acc[mt][1]);
            if (e_hi < s.nfv) *reinterpret_cast<float2*>(slab + e_hi * GH + 2 * tq) = make_float2(acc[mt][2], acc[mt][3]);
        }
    }
    __syncthreads();
    if (tid < GH) {                                        // slot tid: maximum and sum of the part
        float mc = win_ml[tid];
#pragma unroll 1
        for (int w = 0; w < nwarps; ++w) mc = fmaxf(mc, red_m[w * GH + tid]);
        float lc = win_ml[GH + tid] * ex2(win_ml[tid] - mc);
#pragma unroll 1
        for (int w = 0; w < nwarps; ++w) lc = fmaf(red_l[w * GH + tid], ex2(red_m[w * GH + tid] - mc), lc);
        cta_ml[tid] = mc;
        cta_ml[GH + tid] = lc;
    }
    __syncthreads();
    const size_t qh0 = (size_t)b * s.Hq + g_first;
    // o of the part: windows (all dims) + kept dims of the classes at their natural positions, order-fixed over the warps
#pragma unroll 1
    for (int i = tid; i < GH * s.d; i += nthreads) {
        const int g = i / s.d, e = i - g * s.d, sl = hperm<GH>(g);
        const float mc = cta_ml[sl];
        float v = o_s[i] * ex2(win_ml[sl] - mc);
        const int pos = inv_s[e];
        if (pos >= 0) {
#pragma unroll 1
            for (int w = 0; w < nwarps; ++w) {
                const float mwv = red_m[w * GH + sl];
                if (mwv > 0.5f * kNegBig) {
                    const float* sw = reinterpret_cast<const float*>(sm + L.team_off + (w / TW) * L.team_bytes) + (size_t)(w % TW) * (s.d * GH);
                    v = fmaf(sw[pos * GH + sl], ex2(mwv - mc), v);
                }
            }
        }
        o_s[i] = v;
        if ((np > 1 || !p.fused) && g < ng) ws.o[((qh0 + g) * np + part) * s.d + e] = v;
    }
    // z of the part: the teams' accumulators scaled to the part's maximum.  Several parts (or the three-kernel
    // form): to the workspace; a part on its own: w z straight into the table the merge reads.
    float* zw_s = ut;                                      // [GH heads][rows of this part] (u is no longer needed)
    __syncthreads();                                       // (ut is free: every team is past its last spectrum)
#pragma unroll 1
    for (int n = tid; n < s.k; n += nthreads) {
        float zr[GH], zi[GH];                              // per slot
#pragma unroll
        for (int sl = 0; sl < GH; ++sl) { zr[sl] = 0.f; zi[sl] = 0.f; }
#pragma unroll 1
        for (int t = 0; t < NT; ++t) {
            const float* e = reinterpret_cast<const float*>(sm + L.team_off + t * L.team_bytes + L.zt_off_in_team) + n * 2 * GH;
#pragma unroll
            for (int sl = 0; sl < GH; ++sl) {
                const float mt_ = red_m[(t * TW) * GH + sl];
                if (mt_ > 0.5f * kNegBig) {
                    const float sc = ex2(mt_ - cta_ml[sl]);
                    const int ab = sl / N, ln = sl - ab * N;
                    zr[sl] = fmaf(e[(2 * ab) * N + ln], sc, zr[sl]);
                    zi[sl] = fmaf(e[(2 * ab + 1) * N + ln], sc, zi[sl]);
                }
            }
        }
#pragma unroll
        for (int sl = 0; sl < GH; ++sl) {
            const int g = hperm<GH>(sl);
            if (g >= ng) continue;
            if (np > 1 || !p.fused) {
                *reinterpret_cast<float2*>(ws.z + ((qh0 + g) * np + part) * s.M + 2 * n) = make_float2(zr[sl], zi[sl]);
            } else {
                zw_s[g * s.M + 2 * n] = zr[sl] * recon_weight(s.norm, 2 * n, s.k, s.T);
                zw_s[g * s.M + 2 * n + 1] = zi[sl] * recon_weight(s.norm, 2 * n + 1, s.k, s.T);
            }
        }
    }
    if ((np > 1 || !p.fused) && tid < GH) {
        const int g = hperm<GH>(tid);                     // slot tid holds head g
        if (g < ng) {
            float* ml = ws.ml + ((qh0 + g) * np + part) * 2;
            ml[0] = cta_ml[tid];
            ml[1] = cta_ml[GH + tid];
        }
    }
    if (!p.fused) return;

    // ================================ merge (fused kernel) ================================
    // Each part contracts its rows of the merged z with its rows of C^V (streamed through the warps' rings,
    // already on their way); the last part to finish adds the slices and the parts' o in a fixed order,
    // normalises and writes the output rows.
    float* al_s = reinterpret_cast<float*>(sm + L.al_off);                  // [GH heads][np]: exp2(m_part - max)
    float* linv_s = reinterpret_cast<float*>(sm + L.qc_off);               // [GH heads] (the gathered query is no longer needed)
    const int rows = m1 - m0;
    if (np > 1) {
        part_arrive(bar + 1, np, tid);
        part_wait(bar + 1, np, tid, fail, c.status);
#pragma unroll 1
        for (int g = warp; g < GH; g += nwarps) {          // one warp per head, lanes over the parts
            float mx = kNegBig;
#pragma unroll 1
            for (int sp = lane; sp < np; sp += 32) {
                float2 ml = make_float2(kNegBig, 0.f);
                if (g < ng) ml = __ldcg(reinterpret_cast<const float2*>(ws.ml + ((qh0 + g) * np + sp) * 2));
                mx = fmaxf(mx, ml.x);
            }
            mx = warp_max(mx);
            float Lsum = 0.f;
#pragma unroll 1
            for (int sp = lane; sp < np; sp += 32) {
                float2 ml = make_float2(kNegBig, 0.f);
                if (g < ng) ml = __ldcg(reinterpret_cast<const float2*>(ws.ml + ((qh0 + g) * np + sp) * 2));
                const float a = ex2(ml.x - mx);
                al_s[g * np + sp] = a;
                Lsum = fmaf(a, ml.y, Lsum);
            }
            Lsum = warp_sum(Lsum);
            if (lane == 0) linv_s[g] = Lsum > 0.f ? __fdividef(1.0f, Lsum) : 0.f;
        }
        __syncthreads();
        // w_m z_m of my rows, merged over the parts in a fixed order
        if (s.dcv > 0) {
#pragma unroll 1
            for (int t = tid; t < GH * rows; t += nthreads) {
                const int g = t / rows, r = t - g * rows;
                float v = 0.f;
                if (g < ng) {
                    const float* z = ws.z + (qh0 + g) * np * s.M + m0 + r;
#pragma unroll 4
                    for (int sp = 0; sp < np; ++sp) v = fmaf(al_s[g * np + sp], __ldcg(z + (size_t)sp * s.M), v);
                    v *= recon_weight(s.norm, m0 + r, s.k, s.T);
                }
                zw_s[g * s.M + r] = v;
            }
        }
    } else {
        if (tid < GH) {
            const int sl = hperm<GH>(tid);                 // head tid sits in slot sl
            const float lc = cta_ml[GH + sl];
            linv_s[tid] = lc > 0.f ? __fdividef(1.0f, lc) : 0.f;
        }
    }
    __syncthreads();
    // my rows of C^V against w z: lane v holds 16-byte chunk v of a row
    float* ocw = slab;                                     // this warp's partial o^c [GH][dcv]
    if (s.dcv > 0) {
        const int nv = s.dcv >> 2;
        float4 acc4[GH];
#pragma unroll
        for (int g = 0; g < GH; ++g) acc4[g] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
        for (int r0 = ur0; r0 < ur1; r0 += rpp_v) {
            const int nr = min(rpp_v, ur1 - r0);
            const uint32_t st = ring.take();
            if (lane < nv) {
#pragma unroll 1
                for (int rr = 0; rr < nr; ++rr) {
                    const int r = r0 + rr;
                    const uint4 raw = lds128(st + (uint32_t)(rr * s.dcv) * 4 + 16u * lane);
                    float4 x = make_float4(__uint_as_float(raw.x), __uint_as_float(raw.y), __uint_as_float(raw.z), __uint_as_float(raw.w));
                    if (j_pend >= 0) {                     // fused step: pending rank-1 update of this row of C^V
                        const float f = basis_value(r, j_pend, s.T);
                        const float4 y = *reinterpret_cast<const float4*>(xp_s + s.dck + 4 * lane);
                        x.x = fmaf(f, y.x, x.x); x.y = fmaf(f, y.y, x.y); x.z = fmaf(f, y.z, x.z); x.w = fmaf(f, y.w, x.w);
                        *reinterpret_cast<float4*>(cvg + (size_t)r * s.dcv + 4 * lane) = x;
                    }
#pragma unroll
                    for (int g = 0; g < GH; ++g) {
                        const float w = zw_s[g * s.M + (r - m0)];
                        acc4[g].x = fmaf(w, x.x, acc4[g].x);
                        acc4[g].y = fmaf(w, x.y, acc4[g].y);
                        acc4[g].z = fmaf(w, x.z, acc4[g].z);
                        acc4[g].w = fmaf(w, x.w, acc4[g].w);
                    }
                }
            }
            ring.done();
            feed(3);
        }
        if (lane < nv) {
#pragma unroll
            for (int g = 0; g < GH; ++g) *reinterpret_cast<float4*>(ocw + g * s.dcv + 4 * lane) = acc4[g];
        }
    }
    __syncthreads();
    // order-fixed sum over the warps; inv_s becomes dim -> slot in D^vc
#pragma unroll 1
    for (int e = tid; e < s.d; e += nthreads) inv_s[e] = -1;
    __syncthreads();
    if (s.dcv > 0) {
        const int32_t* idc_v = c.idx_comp_v + (size_t)h * s.dcv;
#pragma unroll 1
        for (int e = tid; e < s.dcv; e += nthreads) inv_s[idc_v[e]] = e;
#pragma unroll 1
        for (int t = tid; t < GH * s.dcv; t += nthreads) {
            const int g = t / s.dcv, e = t - g * s.dcv;
            float v = 0.f;
#pragma unroll 1
            for (int w = 0; w < nwarps; ++w) {
                const float* sw = reinterpret_cast<const float*>(sm + L.team_off + (w / TW) * L.team_bytes) + (size_t)(w % TW) * (s.d * GH);
                const int wr0 = min(m1, m0 + w * rows_w);
                if (wr0 < m1) v += sw[g * s.dcv + e];
            }
            if (np > 1) { if (g < ng) ws.oc[((qh0 + g) * np + part) * s.dcv + e] = v; }
            else zw_s[t] = v;                              // (a lone part: w z has been consumed; o^c [GH][dcv] takes its place)
        }
    }
    // ticket: the last part to get here finishes the rows
    __syncthreads();
    if (np > 1) {
        if (tid == 0) {
            int old = 0;
            __threadfence();
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(bar + 2) : "memory");
            *last_s = old == np - 1;
        }
        __syncthreads();
        if (!*last_s) return;
#pragma unroll 1
        for (int t = tid; t < ng * s.d; t += nthreads) {
            const int g = t / s.d, e = t - g * s.d;
            const float* o = ws.o + (qh0 + g) * np * s.d + e;
            float v = 0.f;
#pragma unroll 4
            for (int sp = 0; sp < np; ++sp) v = fmaf(al_s[g * np + sp], __ldcg(o + (size_t)sp * s.d), v);
            const int slot = inv_s[e];
            if (slot >= 0) {
                const float* oc = ws.oc + (qh0 + g) * np * s.dcv + slot;
                float w = 0.f;
#pragma unroll 4
                for (int x = 0; x < np; ++x) w += __ldcg(oc + (size_t)x * s.dcv);
                v += w;
            }
            out[(qh0 + g) * s.d + e] = __float2bfloat16_rn(v * linv_s[g]);
        }
        if (tid == 0) { bar[0] = 0; bar[1] = 0; bar[2] = 0; }   // the counters are zero again for the next call
    } else {
#pragma unroll 1
        for (int t = tid; t < ng * s.d; t += nthreads) {
            const int g = t / s.d, e = t - g * s.d;
            float v = o_s[t];
            const int slot = inv_s[e];
            if (slot >= 0) v += zw_s[g * s.dcv + slot];
            out[(qh0 + g) * s.d + e] = __float2bfloat16_rn(v * linv_s[g]);
        }
    }
}

// Whether the driver takes the cooperative and the programmatic-serialization launch attributes
// together, per device: -1 not probed, 0 no, 1 yes.  set = -2 reads, anything else records.
int coop_pdl_state(int set) {
    constexpr int kMaxDev = 64;
    static signed char state[kMaxDev];
    static bool init = false;
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) { cudaGetLastError(); return 0; }
    std::lock_guard<std::mutex> lock(mu);
    if (!init) { for (int i = 0; i < kMaxDev; ++i) state[i] = -1; init = true; }
    if (set != -2) state[dev] = (signed char)set;
    return state[dev];
}

template <int GH, int OCC>
cudaError_t launch_teams_t(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* q, void* out, char* ws, int step,
                           cudaStream_t st) {
    const TeamSmem L = team_smem_layout(p.fft_log2, s.k, GH, s.d, p.nt, p.tw, p.nsg);
    cudaError_t err = ensure_dynamic_smem(decode_teams_kernel<GH, OCC>, (size_t)L.total);
    if (err != cudaSuccess) return err;
    // window buffers as tensor maps (cached per buffer)
    CUtensorMap tki, tvi, tkl, tvl;
    const int n_bh = s.B * s.Hkv;
    const bool ok_i = window_map(&tki, c.k_init, s.l_init, s.d, n_bh) & window_map(&tvi, c.v_init, s.l_init, s.d, n_bh);
    const bool ok_l = window_map(&tkl, c.k_local, s.l_local, s.d, n_bh) & window_map(&tvl, c.v_local, s.l_local, s.d, n_bh);
    if ((s.l_init > 0 && !ok_i) || (s.l_local > 0 && !ok_l)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_part, s.Hkv * p.n_pass, s.B);
    cfg.blockDim = dim3(32 * p.nt * p.tw);
    cfg.dynamicSmemBytes = (size_t)L.total;
    cfg.stream = st;
    // Programmatic dependent launch: the kernel may be scheduled while its predecessor in the stream
    // still runs and waits (griddepcontrol.wait) where it first reads what the predecessor wrote.  The
    // fused kernel with several parts per head is also a cooperative launch (its CTAs wait for one
    // another); whether the driver takes both attributes together is found out on the first launch
    // outside a stream capture.
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeCooperative;
    attr[1].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (p.fused && p.n_part > 1) {                       // a head served by one CTA waits for nobody: plain launch, any grid
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        const int known = coop_pdl_state(-2);
        if (known < 0 && (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone)) {
            cfg.attrs = attr + 1;                                          // not probed yet: stay on the plain cooperative launch
        } else if (known != 0) {
            cfg.numAttrs = 2;
            cudaError_t err2 = cudaLaunchKernelEx(&cfg, decode_teams_kernel<GH, OCC>, tki, tvi, tkl, tvl, s, c, p,
                                                  static_cast<const bf16*>(q), static_cast<bf16*>(out), ws, step);
            if (err2 == cudaSuccess) { coop_pdl_state(1); return err2; }
            if (known == 1) return err2;
            cudaGetLastError();
            coop_pdl_state(0);
            cfg.attrs = attr + 1;
            cfg.numAttrs = 1;
        } else {
            cfg.attrs = attr + 1;
        }
    }
    return cudaLaunchKernelEx(&cfg, decode_teams_kernel<GH, OCC>, tki, tvi, tkl, tvl, s, c, p, static_cast<const bf16*>(q),
                              static_cast<bf16*>(out), ws, step);
}

// Resident CTAs of the kernel instance on the whole device for the plan's block and shared memory.
template <int GH, int OCC>
int resident_ctas_t(const Dims& s, const DecodePlan& p) {
    struct Entry { int dev, threads; size_t smem; int ctas; };
    static Entry table[16];
    static int used = 0;
    static std::mutex mu;
    const size_t smem = (size_t)team_smem_layout(p.fft_log2, s.k, GH, s.d, p.nt, p.tw, p.nsg).total;
    const int threads = 32 * p.nt * p.tw;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i)
        if (table[i].dev == dev && table[i].smem == smem && table[i].threads == threads) return table[i].ctas;
    if (ensure_dynamic_smem(decode_teams_kernel<GH, OCC>, smem) != cudaSuccess) { cudaGetLastError(); return 0; }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_teams_kernel<GH, OCC>, threads, smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    const int ctas = per_sm * sm_count();
    if (used < 16) table[used++] = Entry{dev, threads, smem, ctas};
    return ctas;
}

}  // namespace

// Team shape of the kernel for transform length 2^log2S with `occ` CTAs per SM: warps per team (a warp keeps
// the scores of at most kMaxGroups 16-token groups of a class in registers), teams, ring depth; false if the
// shared memory does not fit.
bool decode_teams_shape(const Dims& s, int log2S, int gh, int occ, int* nt_out, int* tw_out, int* nsg_out, size_t* smem_out) {
    const int S = 1 << log2S;
    const int max_warps = occ == 2 ? 8 : kMaxWarps;
    const size_t limit = occ == 2 ? 113 * 1024 : 227 * 1024;       // two CTAs share the SM's 228 KB, 1 KB reserved each
    int tw = S / (16 * kMaxGroups);
    if (tw < 2) tw = 2;
    if (tw > max_warps || S / tw < 16) return false;
    for (int nt = max_warps / tw; nt >= 1; --nt) {
        if (nt > 8) continue;
        for (int nsg = kMaxStages; nsg >= 2; --nsg) {
            const size_t need = (size_t)team_smem_layout(log2S, s.k, gh, s.d, nt, tw, nsg).total;
            if (need <= limit) {
                if (nt * tw < 4) return false;
                *nt_out = nt; *tw_out = tw; *nsg_out = nsg;
                if (smem_out) *smem_out = need;
                return true;
            }
        }
    }
    return false;
}

int decode_teams_max_parts() { return kMaxParts; }

// True if the fused kernel of this plan can be launched as planned: a part that waits for nobody runs in
// waves; parts that wait for one another must all be resident at once (what a cooperative launch checks),
// which depends on the registers and shared memory of the compiled instance, so the runtime is asked.
bool decode_fft_launchable(const Dims& s, const DecodePlan& p) {
    if (!p.fused) return true;
    if (p.n_part <= 1) return true;
    const long long grid = (long long)p.n_part * s.Hkv * p.n_pass * s.B;
    int resident = 0;
    if (p.gh == 4) resident = p.occ == 2 ? resident_ctas_t<4, 2>(s, p) : resident_ctas_t<4, 1>(s, p);
    else resident = p.occ == 2 ? resident_ctas_t<2, 2>(s, p) : resident_ctas_t<2, 1>(s, p);
    return grid <= resident;
}

cudaError_t launch_decode_fft(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, const void* q, void* out,
                              char* ws, bool step, cudaStream_t st) {
    if (dtype != FA_BF16) return cudaErrorInvalidValue;
    const int stp = step ? 1 : 0;
    if (p.gh == 4) return p.occ == 2 ? launch_teams_t<4, 2>(s, c, p, q, out, ws, stp, st) : launch_teams_t<4, 1>(s, c, p, q, out, ws, stp, st);
    return p.occ == 2 ? launch_teams_t<2, 2>(s, c, p, q, out, ws, stp, st) : launch_teams_t<2, 1>(s, c, p, q, out, ws, stp, st);
}

}  // namespace fa
