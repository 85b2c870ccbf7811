// fa_decode_attention, main kernel for bf16 caches: residue-class (FFT) evaluation of the
// compressed dims and tensor-core dot products for the kept dims (Eq.6 re-associated).
//
// With theta = 2 pi / T, u~_n = u[2n] - i u[2n+1] and the middle tokens of class c,
// j = c + P a (a = 0..S-1, S = T / P >= k):
//   scores   sum_m F[m][j] u[m]  = Re sum_n (u~_n e^{i theta n c}) e^{2 pi i n a / S}
//   outputs  z_n = sum_j p_j e^{i theta n j} = sum_c e^{i theta n c} sum_a p_{c+Pa} e^{2 pi i n a / S}
// so a class costs one length-S transform per side instead of S * k basis terms.  Two query
// heads share one complex transform (real-pair packing).  With GH = 4 heads a point holds two
// complex numbers stored (re0, re1, im0, im1) and all transform arithmetic runs on packed
// fp32 pairs (add/mul/fma.f32x2).  The score transform runs decimation-in-frequency (natural
// in, digit-reversed out), the probability transform decimation-in-time (digit-reversed in,
// natural out), both in place: softmax is pointwise, so nothing is ever reordered.  NB classes
// are transformed together.
//
// K^mu / V^mu are class-major, so the tokens of a class are one contiguous stream; a producer
// warp brings it in with bulk (TMA) copies through a ring of shared-memory stages.  The eight
// consumer warps feed the tiles to mma.sync (bf16 x bf16 -> fp32; exact for q . K, p rounded to
// bf16 for p . V): K fragments are read with 128-bit loads using the freedom to permute the
// contraction index, V^T fragments with transposing 8x8 matrix loads, conflict-free because
// V^mu rows are stored chunk-swizzled.  Window rows (init + local ring) arrive as tiled TMA
// boxes with the 128-byte swizzle from tensor maps of the window buffers and take the same
// route.  Every wait is bounded.
//
// Two forms, chosen by the host plan.  Three kernels: a prologue kernel forms u = W C^K q, this
// kernel writes per-part partial results (m, l, o, z), an epilogue kernel merges them and applies
// C^V.  Fused (one cooperative launch per call): the parts of a (batch row, KV head) each form a
// slice of the rows of u and exchange it through the workspace behind a counter barrier, window
// tokens have parts of their own, and after a second barrier every part merges its slice of the
// coefficient rows (its rows of every part's z against its rows of C^V); the last part to take
// a ticket adds the slices in a fixed order and writes the output rows.  As the second half of
// fa_decode_step the fused kernel also adds the pending rank-1 update of Eq.5 to the coefficient
// rows it stages and writes them back.
//
// "Slot" below is the position of a head inside a point / an mma column: slot s holds head
// hperm(s) = {0, 2, 1, 3}[s] (GH = 4) so that the packed real parts are slots 0, 1 and the
// packed imaginary parts slots 2, 3.
#include <mutex>

#include "fa_decode_ws.cuh"
#include "fa_tmap.cuh"

#ifdef FA_TIMELINE
// Timeline build (-DFA_TIMELINE): lane 0 of every consumer warp of the first and the last CTA of (batch row 0, KV
// head 0) stamps the SM clock at the phase boundaries marked TL(i); fa_debug_timeline copies the stamps out.
__device__ long long g_fa_timeline[2 * 8 * 32];
#define TL(i) do { if ((threadIdx.x & 31) == 0 && threadIdx.x < 256 && blockIdx.y == 0 && blockIdx.z == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) \
    g_fa_timeline[((blockIdx.x == 0 ? 0 : 1) * 8 + (threadIdx.x >> 5)) * 32 + (i)] = clock64(); } while (0)
extern "C" int fa_debug_timeline(long long* host_out) {
    return (int)cudaMemcpyFromSymbol(host_out, g_fa_timeline, sizeof(g_fa_timeline));
}
// Per CTA and launch (the last 32 launches): SM id, SM clock at entry, after the wait for the previous kernel, at exit.
__device__ long long g_fa_span[32 * 160 * 4];
__device__ int g_fa_span_cnt[160];
extern "C" int fa_debug_spans(long long* host_out) {
    return (int)cudaMemcpyFromSymbol(host_out, g_fa_span, sizeof(g_fa_span));
}
#define SPAN(i) do { if (threadIdx.x == 0 && blockIdx.z == 0) { const int cta_ = blockIdx.y * gridDim.x + blockIdx.x; if (cta_ < 160) { \
    const int l_ = g_fa_span_cnt[cta_] & 31; long long* p_ = g_fa_span + (l_ * 160 + cta_) * 4; \
    if ((i) == 0) { unsigned sm_; asm volatile("mov.u32 %0, %%smid;" : "=r"(sm_)); p_[0] = sm_; } \
    p_[1 + ((i) > 2 ? 2 : (i))] = clock64(); if ((i) >= 2) g_fa_span_cnt[cta_] += 1; } } } while (0)
#else
#define TL(i) do { } while (0)
#define SPAN(i) do { } while (0)
#endif

namespace fa {
namespace {

constexpr int kConsumers = 256;
constexpr int kWarps = kConsumers / 32;
constexpr int kThreads = kConsumers + 32;
// The split kernel: the eight warps above are the transform group, six more consume the ring tiles (kept-dim products).
constexpr int kSplitConsumers = kConsumers + 192;
constexpr int kSplitWarps = kSplitConsumers / 32;
__host__ __device__ constexpr int threads_of(bool split) { return (split ? kSplitConsumers : kConsumers) + 32; }
constexpr int kStageBytes = 16384;
constexpr int kStages = 5;                 // stages of the ring with one CTA per SM
constexpr int kStagesOcc2 = 3;             // with two CTAs per SM (small transforms, many heads)
// (the split build runs a ring of three as well: its tile group drains the ring steadily, and the two stages it gives
// up are what lets a batch hold two classes of the longest transforms)
__host__ __device__ constexpr int ring_stages(int occ, int split = 0) { return (occ == 2 || split) ? kStagesOcc2 : kStages; }
constexpr int kPendRows = 256;            // rows of a part whose basis values are tabulated for the fused step's update
constexpr int kWinRowsPerTile = 64;       // rows of one window tile: two [64 rows x 64 dims] TMA boxes, 128-byte swizzle
constexpr int kWinHalfBytes = kWinRowsPerTile * 128;
constexpr uint32_t kSpinLimit = 1u << 24;
using bf16 = __nv_bfloat16;
typedef unsigned long long u64;

// ---- PTX wrappers -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(b)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* b, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(smem_addr(b)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls, records the failure, never hangs.  The common case
// (the phase is already complete) is one inlined test; the polling loop is a call, so that the many
// wait sites do not bloat the kernel (its code is fetched cold: every phase runs once per CTA).
__device__ __noinline__ void mbar_wait_slow(uint64_t* b, uint32_t parity, volatile int* fail, int32_t* status) {
    if (*fail) return;
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(b, parity)) return;
    *fail = 1;
    atomicExch(status, (int)FA_ERR_TIMEOUT);
}
__device__ __forceinline__ void mbar_wait(uint64_t* b, uint32_t parity, volatile int* fail, int32_t* status) {
    if (mbar_try_wait(b, parity)) return;
    mbar_wait_slow(b, parity, fail, status);
}
// Eq.4 for one (row, column): a call, for the same reason.
__device__ __noinline__ float basis_value(int m, int j, int T) {
    float cs, sn;
    basis_cs(m >> 1, j, T, &cs, &sn);
    return (m & 1) ? sn : cs;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
// One box of a window tensor map: dims x0.., rows y0.., (batch, KV head) z.
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* tm, int x0, int y0, int z, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                     smem_addr(dst)),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(x0), "r"(y0), "r"(z), "r"(smem_addr(bar))
                 : "memory");
}
// 16-byte asynchronous copy that bypasses L1 (the source may have been written by another SM)
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst)), "l"(__cvta_generic_to_global(src)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory"); }
// Barrier ID among NT threads: the consumer warps (all of them: barrier 1; the transform group of the split kernel: barrier 2)
template <int NT = kConsumers, int ID = 1>
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(NT) : "memory"); }

// Barrier among the CTAs of one (b, KV head, pass) on a global counter (fused kernel only: a
// cooperative launch makes all of them resident).  Arrive: the consumer warps meet, then one thread
// fences (cumulative over what the others wrote before the meeting) and adds 1 with release
// semantics.  Wait: one thread polls with acquire loads, bounded like every other wait of this
// kernel, then the consumer warps meet.
template <int NT = kConsumers>
__device__ __forceinline__ void part_arrive(int32_t* cnt, int n, int tid) {
    consumer_sync<NT>();
    if (n > 1 && tid == 0) {                              // a part on its own meets nobody: no counter
        __threadfence();
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(cnt) : "memory");
    }
}
template <int NT = kConsumers>
__device__ __forceinline__ void part_wait(const int32_t* cnt, int n, int tid, volatile int* fail, int32_t* status) {
    if (n > 1 && tid == 0 && !*fail) {
        bool ok = false;
        for (uint32_t i = 0; i < (1u << 22); ++i) {
            int v;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(cnt) : "memory");
            if (v >= n) { ok = true; break; }
            if (i > 64) __nanosleep(64);
        }
        if (!ok) { *fail = 1; atomicExch(status, (int)FA_ERR_TIMEOUT); }
    }
    consumer_sync<NT>();
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
// shared-memory accesses by 32-bit address (no generic-pointer arithmetic in the inner loops)
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts64(uint32_t a, float x, float y) {
    asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(a), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(bf16 lo, bf16 hi) {
    return (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
}
// cos and sin of 2 pi * frac, frac in [0, 1): hardware approximations on an angle folded into
// [-pi, pi) (absolute error ~5e-7, far below what bf16 operands carry)
__device__ __forceinline__ float2 cis_frac(float frac) {
    const float a = 6.283185307179586f * (frac - (frac >= 0.5f ? 1.0f : 0.0f));
    return make_float2(__cosf(a), __sinf(a));
}
// Order-independent accumulation of fp32 values: 64-bit fixed point, 30 fractional bits.  The sums here are
// probabilities (<= 1 each, at most 2^20 of them) times bf16 values, far inside the 33 integer bits.
constexpr float kFix = 1073741824.0f, kFixInv = 1.0f / 1073741824.0f;     // (scaling by a power of two is exact in fp32)
__device__ __forceinline__ void fix_add(long long* p, float v) {
    atomicAdd(reinterpret_cast<unsigned long long*>(p), (unsigned long long)__float2ll_rn(v * kFix));
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
// a + (the same value of the neighbouring lane)
__device__ __forceinline__ PR<2> pair_sum(PR<2> a) { PR<2> o; o.v = __shfl_xor_sync(0xffffffffu, a.v, 1); return a + o; }
__device__ __forceinline__ PR<1> pair_sum(PR<1> a) { return PR<1>{a.v + __shfl_xor_sync(0xffffffffu, a.v, 1)}; }
template <int N> __device__ __forceinline__ PC<N> pair_sum(PC<N> a) { return PC<N>{pair_sum(a.re), pair_sum(a.im)}; }
__device__ __forceinline__ float2 cmulf(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
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
// of the passes and the digit-reversed accesses of token-ordered code (consecutive slots sit 64, 8
// or 1 points apart after a radix-8 decimation) all spread over the banks.
__host__ __device__ constexpr int pf(int f) { return f + ((f >> 5) << 2) + ((f >> 8) << 2) + ((f >> 11) << 2); }
__host__ __device__ constexpr int pf_size(int floats) { return pf(floats) + 8; }

// Radix of the pass that handles a sub-transform of length 2^l (8 where possible, two 4s for 16).
__host__ __device__ constexpr int radix_log2(int l) { return (l >= 3 && l != 4) ? 3 : (l >= 2 ? 2 : 1); }
// Number of twiddles (per complex lane) of all passes from length 2^LS down to, not including, 2^l.
__host__ __device__ constexpr int tw_offset(int LS, int l) {
    int off = 0;
    for (int cur = LS; cur > l;) {
        const int rl = radix_log2(cur);
        if (cur > rl) off += ((1 << rl) - 1) << (cur - rl);
        cur -= rl;
    }
    return off;
}
__host__ __device__ constexpr int tw_total(int LS) { return tw_offset(LS, 0); }

// One in-place pass of radix R = 2^RL over sub-transforms of length 2^LL, for nb transforms of
// length 2^LS held in consecutive buffers.  DIF: butterfly, then twiddle the outputs; DIT:
// twiddle the inputs, then butterfly.  Twiddles are stored [q - 1][j] as splat pairs (wr, wi).
template <int GH, int LS, int LL, bool DIT>
__device__ __forceinline__ void fft_pass(float* fbuf, int fb_floats, int nb, const float* twf, int tid) {
    constexpr int N = GH / 2;
    constexpr int RL = radix_log2(LL), R = 1 << RL;
    constexpr int STL = LL - RL, PERL = LS - RL;          // log2 butterflies per sub-transform / per transform
    constexpr bool kTw = LL > RL;
    constexpr int kTwOff = tw_offset(LS, LL);
    for (int item = tid; item < (nb << PERL); item += kConsumers) {
        const int ci = item >> PERL, rest = item & ((1 << PERL) - 1);
        const int blk = rest >> STL, j = rest & ((1 << STL) - 1);
        float* base = fbuf + ci * fb_floats;
        const int e0 = (blk << LL) + j;
        PC<N> v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = ld_pt<N>(base + pf((e0 + (r << STL)) * GH));
        PR<N> wr[R], wi[R];
        if constexpr (kTw) {
#pragma unroll
            for (int q = 1; q < R; ++q) {
                const float2 w = *reinterpret_cast<const float2*>(twf + 2 * (kTwOff + ((q - 1) << STL) + j));
                wr[q] = splat<N>(w.x);
                wi[q] = splat<N>(w.y);
            }
            if constexpr (DIT) {
#pragma unroll
                for (int q = 1; q < R; ++q) v[q] = cmulw(v[q], wr[q], wi[q]);
            }
        }
        dft<R, N>(v);
        if constexpr (kTw && !DIT) {
#pragma unroll
            for (int q = 1; q < R; ++q) v[q] = cmulw(v[q], wr[q], wi[q]);
        }
#pragma unroll
        for (int r = 0; r < R; ++r) st_pt(base + pf((e0 + (r << STL)) * GH), v[r]);
    }
}

// All passes of the transform, ending each with a barrier of the consumer warps.
// (kConsumers threads take part: all consumer warps, or the transform group of the split kernel with its barrier BID)
template <int GH, int LS, int LL, bool DIT, int BID = 1>
__device__ __forceinline__ void fft_run(float* fbuf, int fb_floats, int nb, const float* twf, int tid) {
    constexpr int RL = radix_log2(LL);
    if constexpr (!DIT) {
        fft_pass<GH, LS, LL, false>(fbuf, fb_floats, nb, twf, tid);
        consumer_sync<kConsumers, BID>();
        if constexpr (LL - RL > 0) fft_run<GH, LS, LL - RL, false, BID>(fbuf, fb_floats, nb, twf, tid);
    } else {
        if constexpr (LL - RL > 0) fft_run<GH, LS, LL - RL, true, BID>(fbuf, fb_floats, nb, twf, tid);
        fft_pass<GH, LS, LL, true>(fbuf, fb_floats, nb, twf, tid);
        consumer_sync<kConsumers, BID>();
    }
}

// Position of output index a after the decimation-in-frequency passes.
template <int LS>
__host__ __device__ constexpr int dif_pos(int a) {
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
    int tok[3];      // logical offset of the first row relative to t0
};
__device__ __forceinline__ WinSegs win_segments(int t0, int t1, int n_init, int n_local, int head, int l_local) {
    WinSegs w;
    w.n = 0;
    int a0 = t0, a1 = min(t1, n_init);
    if (a1 > a0) { w.buf[w.n] = 0; w.row[w.n] = a0; w.cnt[w.n] = a1 - a0; w.tok[w.n] = 0; ++w.n; }
    int u0 = max(t0 - n_init, 0), u1 = min(t1 - n_init, n_local);
    if (u1 > u0) {
        int ps = (head + u0) % l_local;
        int len1 = min(u1 - u0, l_local - ps);
        w.buf[w.n] = 1; w.row[w.n] = ps; w.cnt[w.n] = len1; w.tok[w.n] = n_init + u0 - t0; ++w.n;
        if (u1 - u0 > len1) {
            w.buf[w.n] = 1; w.row[w.n] = 0; w.cnt[w.n] = u1 - u0 - len1; w.tok[w.n] = n_init + u0 + len1 - t0; ++w.n;
        }
    }
    return w;
}

struct FftSmem {
    int stages_off, fbuf_off, kb_off, pbt_off, twf_off, rev_off, E_off, ut_off, z_off, o_off, red_off, pend_off, zero_off, total;
    int fb_floats, pbs;
};
// True if the kernel packs two residue classes of ONE query head into a complex transform (one query head per KV head:
// the second slot would otherwise be empty).  Then a batch of NB classes needs half the transform and score buffers.
__host__ __device__ inline bool class_pairs(int G, int GH, int split) { return G == 1 && GH == 2 && !split; }
__host__ __device__ inline FftSmem fft_smem_layout(int log2S, int k, int GH, int NB, int d, int occ, int split = 0, bool cp = false) {
    const int S = 1 << log2S;
    const int NT = cp ? (NB + 1) >> 1 : NB;               // transforms of a batch
    FftSmem L;
    L.fb_floats = pf_size(S * GH);
    L.pbs = S + 8;                                        // bf16 per (class, slot) row of rounded probabilities
    int off = 256;                                        // mbarriers + flags
    L.zero_off = off; off += 16;
    off = 1024;                                           // stages are 1024-byte aligned (swizzled window tiles)
    L.stages_off = off; off += ring_stages(occ, split) * kStageBytes;
    L.fbuf_off = off; off += 4 * NT * L.fb_floats;
    off = (off + 15) / 16 * 16;
    L.kb_off = off; off += 4 * NT * S * GH;               // kept-dim scores of the batch, natural token order
    off = (off + 15) / 16 * 16;
    L.pbt_off = off; off += cp ? 2 * (NB + 1) * L.pbs : 2 * NB * GH * L.pbs;   // class pairs: one row per class and one of zeros
    off = (off + 15) / 16 * 16;
    L.twf_off = off; off += 8 * (tw_total(log2S) + 1);
    L.rev_off = off; off += 2 * S;
    off = (off + 15) / 16 * 16;
    L.E_off = off; off += (8 * k + 15) / 16 * 16;
    L.ut_off = off; off += (8 * k * GH + 15) / 16 * 16;
    L.z_off = off; off += (8 * k * GH + 15) / 16 * 16;
    off = (off + 15) / 16 * 16;
    L.o_off = off; off += 8 * GH * d;
    L.red_off = off; off += 4 * ((split ? kSplitWarps : kWarps) * GH + GH + 8);
    off = (off + 15) / 16 * 16;
    L.pend_off = off; off += 8 * d + 4 * kPendRows + 4 * d + 2 * GH * d + 4 * d;   // fused step: compressed dims of the leaving row, basis column of this part's rows, the leaving row; the query rows
    L.total = (off + 127) / 128 * 128 + 1024;             // slack to align the base to 1024 bytes at run time
    return L;
}

// Fused step: the kept dims of the middle token that is not in the cache yet, written by one warp over its row of a
// tile in shared memory.  Out of line: taken once per kernel, and the tile loops keep their registers.
__device__ __noinline__ void patch_mid_k(uint32_t row_addr, const int32_t* idf, int nfk, const bf16* xrow, int lane) {
#pragma unroll 1
    for (int e = lane; e < nfk; e += 32)
        asm volatile("st.shared.b16 [%0], %1;" ::"r"(row_addr + (uint32_t)(2 * e)), "h"(__bfloat16_as_ushort(xrow[idf[e]])) : "memory");
    __syncwarp();
}
__device__ __noinline__ void patch_mid_v(uint32_t row_addr, const int32_t* idf, int nfv, const bf16* xrow, int slot, int lane) {
#pragma unroll 1
    for (int e = lane; e < nfv; e += 32)
        asm volatile("st.shared.b16 [%0], %1;" ::"r"(row_addr + (uint32_t)(2 * v_mid_col(slot, e, nfv, FA_BF16))), "h"(__bfloat16_as_ushort(xrow[idf[e]])) : "memory");
    __syncwarp();
}

template <int GH> __host__ __device__ constexpr int hperm(int s) { return GH == 4 ? (((s & 1) << 1) | (s >> 1)) : s; }

// GH query heads per CTA (2 or 4), transform length S = 2^LS, OCC CTAs per SM (2: shorter ring, register cap),
// STEP: the instance that also carries the push of a fused step (the plain decode call pays nothing for it).
template <int GH, int LS, int OCC, bool STEP, bool SPLIT>
__global__ void __launch_bounds__(threads_of(SPLIT), OCC) decode_fft_kernel(const __grid_constant__ CUtensorMap tm_ki,
                                                                  const __grid_constant__ CUtensorMap tm_vi,
                                                                  const __grid_constant__ CUtensorMap tm_kl,
                                                                  const __grid_constant__ CUtensorMap tm_vl, Dims s, CacheDev c,
                                                                  DecodePlan p, const bf16* __restrict__ q, bf16* __restrict__ out,
                                                                  char* wsp, const bf16* __restrict__ k_new,
                                                                  const bf16* __restrict__ v_new) {
    constexpr bool step = STEP;
    constexpr int N = GH / 2;
    constexpr int S = 1 << LS;
    constexpr int NS = ring_stages(OCC, SPLIT ? 1 : 0);
    // Consumer threads: kAll of them; the warps that consume ring tiles (kept-dim and window products) are all of them,
    // or, in the split kernel, the last six, while the first eight (the transform group) run the compressed-dim phases
    // of the class batches beside them.
    constexpr int kAll = SPLIT ? kSplitConsumers : kConsumers, kAllW = kAll / 32, kAllT = kAll + 32;
    constexpr int kMW = SPLIT ? kAllW - kWarps : kWarps, kM0 = SPLIT ? kWarps : 0;
    auto all_sync = [] { consumer_sync<kAll, 1>(); };
    extern __shared__ __align__(128) unsigned char smem_unaligned[];
    unsigned char* smem_raw = smem_unaligned + ((1024u - (smem_addr(smem_unaligned) & 1023u)) & 1023u);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the epilogue may be scheduled behind us at once
    Ws ws = ws_view(wsp, p);
    const int NB = p.nb;
    const FftSmem L = fft_smem_layout(LS, s.k, GH, NB, s.d, OCC, SPLIT ? 1 : 0, class_pairs(s.G, GH, SPLIT ? 1 : 0));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw);
    uint64_t* empty = full + NS;
    volatile int* fail = reinterpret_cast<volatile int*>(smem_raw + 128);
    unsigned char* zero16 = smem_raw + L.zero_off;
    unsigned char* stages = smem_raw + L.stages_off;
    float* fbuf = reinterpret_cast<float*>(smem_raw + L.fbuf_off);        // [NB][fb_floats] points of GH floats
    float* kb = reinterpret_cast<float*>(smem_raw + L.kb_off);            // [NB][S][GH]
    bf16* pbt = reinterpret_cast<bf16*>(smem_raw + L.pbt_off);           // [NB][GH slots][pbs]
    float* twf = reinterpret_cast<float*>(smem_raw + L.twf_off);          // pass twiddles (float2 each)
    uint16_t* rev = reinterpret_cast<uint16_t*>(smem_raw + L.rev_off);    // slot -> point after the DIF passes
    float2* E = reinterpret_cast<float2*>(smem_raw + L.E_off);            // e^{i theta n}
    float* ut = reinterpret_cast<float*>(smem_raw + L.ut_off);            // [k] (A.re, A.im, B.re, B.im) x N: (1/2) u~
    float* z_s = reinterpret_cast<float*>(smem_raw + L.z_off);            // [k] same packing
    // [GH heads][d]: the warps' output fragments are summed here as 64-bit fixed-point numbers (scale 2^30):
    // integer additions commute, so the shared-memory atomics give the same bits in whatever order they land
    long long* o_s = reinterpret_cast<long long*>(smem_raw + L.o_off);
    float* red_s = reinterpret_cast<float*>(smem_raw + L.red_off);        // [kAllW][GH] + l_s[GH]
    const int fb_floats = L.fb_floats, pbs = L.pbs;

    const int part = blockIdx.x;                          // partial-result index: class CTAs, then window CTAs
    const bool is_win = part >= p.n_split;
    const int h = blockIdx.y / p.n_pass, pass = blockIdx.y % p.n_pass;
    const int b = blockIdx.z;
    const int g_first = h * s.G + pass * GH;
    const int ng = min(GH, s.G - pass * GH);
    // One query head in two slots (MHA): the second slot would carry nothing.  Instead both slots belong to the head
    // and a packed transform carries two residue classes, class 2 t in the real parts (slot 0) and class 2 t + 1 in the
    // imaginary parts (slot 1): half as many spectra, transforms, softmax points and folds.  The slots keep their own
    // running maxima, sums, outputs and z (slot 1 sees no window token) and are folded into slot 0 before the
    // partial results are written.
    const bool cp = class_pairs(s.G, GH, SPLIT ? 1 : 0);
    const int tid = threadIdx.x;
    const int log2P = 31 - __clz(s.P);

    TL(0);
    SPAN(0);
    // ---- one-time set-up, independent of the cache: it may overlap the tail of the previous kernel ----
    if (tid < kAll) {
        #pragma unroll 1
        for (int i = tid; i < s.k; i += kAll) {
            E[i] = cis_frac((float)i / (float)s.T);
        }
        for (int l = LS; l > 0;) {
            const int rl = radix_log2(l), R = 1 << rl, st = 1 << (l - rl);
            if (l > rl) {
                const int off = tw_offset(LS, l);
                #pragma unroll 1
                for (int i = tid; i < (R - 1) * st; i += kAll) {
                    const int qm1 = i / st, j = i - qm1 * st;
                    reinterpret_cast<float2*>(twf)[off + i] = cis_frac((float)(((qm1 + 1) * j) & ((1 << l) - 1)) / (float)(1 << l));
                }
            }
            l -= rl;
        }
        #pragma unroll 1
        for (int a = tid; a < S; a += kAll) rev[a] = (uint16_t)dif_pos<LS>(a);
        if (tid < GH + 8) red_s[kAllW * GH + tid] = 0.f;

    }
    // This part's rows of C^K start towards the transform buffers, and its rows of C^V towards L2, as soon as
    // the kernels before this one are done (the previous step's kernel writes coefficient rows).
    const int m0 = part * (s.M >> 2) / p.n_part * 4, m1 = (part + 1) * (s.M >> 2) / p.n_part * 4;
    // rows of C^K staged at a time: the transform buffers and, behind them, the kept-dim score and probability
    // buffers (one contiguous area, all idle until the first batch)
    const int uch = s.dck > 0 ? (((L.twf_off - L.fbuf_off) >> 2) / s.dck) & ~3 : 0;
    auto start_coef_rows = [&]() {
        if (tid >= kAll) return;
        if (s.dck > 0) {
            const float* ck = coef_rows(c.coef_k, s, b, h, s.dck) + (size_t)m0 * s.dck;
#pragma unroll 1
            for (int i = tid; i < min(m1 - m0, uch) * (s.dck >> 2); i += kAll) cp_async16(fbuf + 4 * i, ck + 4 * i);
        }
        if (s.dcv > 0) {
            const char* cv = reinterpret_cast<const char*>(coef_rows(c.coef_v, s, b, h, s.dcv) + (size_t)m0 * s.dcv);
            const int bytes = (m1 - m0) * s.dcv * 4;
#pragma unroll 1
            for (int o = tid * 128; o < bytes; o += kAll * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(cv + o));
        }
    };
    // The inputs of the call, staged once: the query rows of this pass [GH heads][d] and, for a fused step, the
    // new token of this KV head [2 sides][d].
    bf16* xrow_s = reinterpret_cast<bf16*>(smem_raw + L.pend_off + 8 * s.d + 4 * kPendRows);     // [2][d] the row that leaves the window
    bf16* qs_s = xrow_s + 2 * s.d;                                                                 // [GH][d]
    bf16* nrow_s = qs_s + GH * s.d;                                                                // [2][d]
    const bf16* knew_bh = nrow_s;
    const bf16* vnew_bh = nrow_s + s.d;
    auto stage_inputs = [&]() {
        const int per_row = s.d >> 3;
        if (tid < GH * per_row) {
            const int g = tid / per_row, ch = tid - g * per_row;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (g < ng) v = *reinterpret_cast<const uint4*>(q + ((size_t)b * s.Hq + g_first + g) * s.d + 8 * ch);
            *reinterpret_cast<uint4*>(qs_s + g * s.d + 8 * ch) = v;
        } else if (STEP && tid < (GH + 2) * per_row) {
            const int side = (tid - GH * per_row) / per_row, ch = tid - (GH + side) * per_row;
            *reinterpret_cast<uint4*>(nrow_s + side * s.d + 8 * ch) =
                *reinterpret_cast<const uint4*>((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + h) * s.d + 8 * ch);
        }
    };
    // fused kernel: everything below reads what earlier kernels in the stream wrote (state, cache, coefficients, q)
    if (p.fused) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        SPAN(1);
        start_coef_rows();
    }
    stage_inputs();

    int n_init = c.state[kStateStride * b + 0], n_local = c.state[kStateStride * b + 1];
    int n_mid_raw = c.state[kStateStride * b + 2], head = c.state[kStateStride * b + 3];
    // Fused step (Eq.5 then Eq.6 in this one launch): every CTA applies the push to its own view of the counters
    // and works on the cache as it will be.  The rows that the push moves are not in place yet: the CTA that
    // meets one in a tile patches the tile in shared memory (the new token's window row from k_new / v_new, the
    // kept dims of the row that leaves the local window at middle token j_pend), the rank-1 update f_j x^T is
    // added to the coefficient rows as they stream by, and the rows and counters are written to the cache
    // when every CTA that reads the old ones is past them.
    int j_pend = -1;                                      // basis column of the coefficient update, or -1
    int new_buf = -1, new_row = 0, new_tok = -1;          // buffer (0 init, 1 local) and row of the new token, its logical window index
    bool cap_full = false;
    if (step) {
        const bool to_init = n_init < s.l_init;
        const bool evict = !to_init && n_local == s.l_local;
        cap_full = evict && (n_mid_raw >= s.max_mid || n_mid_raw >= s.T);
        if (cap_full) {
            if (tid == 0 && part == 0 && h == 0 && pass == 0) atomicExch(c.status, (int)FA_ERR_CAPACITY);
        } else if (to_init) {
            new_buf = 0; new_row = n_init; new_tok = n_init; ++n_init;
        } else if (!evict) {
            new_buf = 1; new_row = (head + n_local) % s.l_local; new_tok = n_init + n_local; ++n_local;
        } else {
            j_pend = n_mid_raw; ++n_mid_raw;
            if (s.l_local > 0) { new_buf = 1; new_row = head; head = (head + 1) % s.l_local; new_tok = n_init + n_local - 1; }
        }
    }
    const int n_mid = min(n_mid_raw, s.max_mid);
    const int cstar = j_pend >= 0 ? j_pend & (s.P - 1) : -1, astar = j_pend >= 0 ? j_pend >> log2P : 0;   // class and slot of token j_pend
    // the row that leaves the local window (or the new token itself without a local window), both sides, natural dim order
    if (j_pend >= 0 && tid >= kAll - 2 * (s.d >> 3) && tid < kAll) {
        const int t2 = tid - (kAll - 2 * (s.d >> 3));
        const int side = t2 / (s.d >> 3), ch = t2 - side * (s.d >> 3);
        if (s.l_local > 0)
            *reinterpret_cast<uint4*>(xrow_s + side * s.d + 8 * ch) =
                *reinterpret_cast<const uint4*>(win_row<bf16>(side == 0 ? c.k_local : c.v_local, s, b, h, s.l_local, new_row) + 8 * ch);
        else
            *reinterpret_cast<uint4*>(xrow_s + side * s.d + 8 * ch) =
                *reinterpret_cast<const uint4*>((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + h) * s.d + 8 * ch);
    }
    const int c0 = is_win ? 0 : part * s.P / p.n_split;
    const int c1 = is_win ? 0 : (part + 1) * s.P / p.n_split;
    const int n_win = n_init + n_local;
    // window tokens: spread over the class CTAs, or over CTAs of their own
    const int wi = p.n_wsplit ? part - p.n_split : part, wn = p.n_wsplit ? p.n_wsplit : p.n_split;
    const bool has_win = p.n_wsplit ? is_win : true;
    const int w0 = has_win ? wi * n_win / wn : 0, w1 = has_win ? (wi + 1) * n_win / wn : 0;
    auto n_of_class = [&](int cls) { return cls < n_mid ? (n_mid - cls + s.P - 1) >> log2P : 0; };

    const int rowb_k = s.nfk * 2, rowb_v = s.nfv * 2;
    const int nhalf = (s.d + 63) >> 6;                                     // 64-dim boxes per window row
    const int ts_k = rowb_k ? (kStageBytes / rowb_k) & ~15 : 0, ts_v = rowb_v ? (kStageBytes / rowb_v) & ~15 : 0;
    const int ts_w = kWinRowsPerTile;
    // window tokens per softmax chunk: the score and probability buffers of all NB classes when
    // they can be addressed as one, else those of one class
    const int NT = class_pairs(s.G, GH, SPLIT ? 1 : 0) ? (NB + 1) >> 1 : NB;       // transform buffers of a batch
    const int wchunk = pf_size(NT * S * GH) <= NT * L.fb_floats ? NT * S : S;
    // row stride of the window probabilities (class pairs: two rows in the NB + 1 rows of the classes)
    const int pbw = class_pairs(s.G, GH, SPLIT ? 1 : 0) ? (((NB + 1) * L.pbs) >> 1) & ~7 : NB * L.pbs;

    if (tid == 0) {
        for (int i = 0; i < NS; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, kMW); }
        if constexpr (SPLIT) {                            // the handshakes between the tile group and the transform group
            uint64_t* gb = reinterpret_cast<uint64_t*>(smem_raw + 160);
            mbar_init(gb, kMW); mbar_init(gb + 1, kWarps); mbar_init(gb + 2, kWarps); mbar_init(gb + 3, kMW);   // kb_full, kb_free, p_full, p_free
        }
        *fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // stale shared memory must hold finite numbers: rows past the end of a tile are multiplied by p = 0
    #pragma unroll 1
    for (int i = tid; i < (NS * kStageBytes) / 16; i += kAllT) reinterpret_cast<uint4*>(stages)[i] = make_uint4(0, 0, 0, 0);
    if (tid < 4) reinterpret_cast<uint32_t*>(zero16)[tid] = 0;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    TL(1);

    // ============================ producer warp =================================
    if (tid >= kAll) {
        // Same order as the consumers: the K tiles of the first batch of classes, the window rows,
        // then per batch the V tiles (and, from the second batch on, its K tiles first).
        const int plane = tid - kAll;
        if (plane == 0) {
            int it = 0;
            auto acquire = [&](uint32_t bytes) -> unsigned char* {
                const int st = it % NS;
                if (it >= NS) mbar_wait(empty + st, ((it / NS) - 1) & 1, fail, c.status);
                if (*fail) return nullptr;
                mbar_expect_tx(full + st, bytes);
                return stages + (size_t)st * kStageBytes;
            };
            auto class_tiles = [&](int cb, int nb, int side) {
                const int ts = side == 0 ? ts_k : ts_v, rowb = side == 0 ? rowb_k : rowb_v;
                if (!ts) return;
#pragma unroll 1
                for (int cls = cb; cls < cb + nb; ++cls) {
                    const int n_c = n_of_class(cls);
#pragma unroll 1
                    for (int a0 = 0; a0 < n_c; a0 += ts) {
                        const uint32_t bytes = (uint32_t)(min(ts, n_c - a0) * rowb);
                        const bf16* src = side == 0 ? mid_row<bf16>(c.k_mid, s, b, h, cls, a0, s.nfk)
                                                    : mid_row<bf16>(c.v_mid, s, b, h, cls, a0, s.nfv);
                        if (unsigned char* dst = acquire(bytes)) bulk_g2s(dst, src, bytes, full + it % NS);
                        ++it;
                    }
                }
            };
            if (c0 < c1) class_tiles(c0, min(NB, c1 - c0), 0);
            // window rows: tiles of 64 rows, one TMA box per 64 dims
#pragma unroll 1
            for (int t0 = w0; t0 < w1; t0 += wchunk) {
                const WinSegs sg = win_segments(t0, min(w1, t0 + wchunk), n_init, n_local, head, s.l_local);
#pragma unroll 1
                for (int side = 0; side < 2; ++side)
#pragma unroll 1
                    for (int i = 0; i < sg.n; ++i)
#pragma unroll 1
                        for (int r0 = 0; r0 < sg.cnt[i]; r0 += ts_w) {
                            const CUtensorMap* tm = sg.buf[i] == 0 ? (side == 0 ? &tm_ki : &tm_vi) : (side == 0 ? &tm_kl : &tm_vl);
                            if (unsigned char* dst = acquire((uint32_t)(nhalf * kWinHalfBytes))) {
#pragma unroll 1
                                for (int hf = 0; hf < nhalf; ++hf)
                                    tma_load_3d(dst + hf * kWinHalfBytes, tm, hf * 64, sg.row[i] + r0, b * s.Hkv + h, full + it % NS);
                            }
                            ++it;
                        }
            }
#pragma unroll 1
            for (int cb = c0; cb < c1; cb += NB) {
                const int nb = min(NB, c1 - cb);
                if (cb != c0) class_tiles(cb, nb, 0);
                class_tiles(cb, nb, 1);
            }
        }
        return;
    }

    // ============================ consumer warps =================================
    const int warp = tid >> 5, lane = tid & 31;
    const bool is_m = warp >= kM0;                        // this warp consumes ring tiles
    const int wm = warp - kM0;
    const int gq = lane >> 2, tq = lane & 3;              // mma fragment coordinates
    const int npk = s.nfk >> 3, nchv = s.nfv >> 3, npw = s.d >> 3;
    const float sl2 = s.scale * kLog2e;

    int32_t* bar = ws.bar + 4 * (((size_t)b * s.Hkv + h) * p.n_pass + pass);
    // gathered query of the compressed K dims (one element per thread and round), loaded early
    float qc_early = 0.f;
    if (p.fused && s.dck > 0 && tid < GH * s.dck) {
        const int g = tid / s.dck, e = tid - g * s.dck;
        if (g < ng) qc_early = __bfloat162float(qs_s[g * s.d + c.idx_comp_k[(size_t)h * s.dck + e]]);
    }
    // fused step: the coefficient update the light append kernel left pending (basis column j_pend, or -1);
    // the leaving row's compressed dims and the basis values of this part's rows are fetched / formed now
    float* xp_s = reinterpret_cast<float*>(smem_raw + L.pend_off);       // [dck + dcv]
    float* f_s = xp_s + 2 * s.d;                                          // [kPendRows]
    if (j_pend >= 0) {
        for (int i = tid; i < s.dck + s.dcv; i += kAll)
            xp_s[i] = i < s.dck ? __bfloat162float(xrow_s[c.idx_comp_k[(size_t)h * s.dck + i]])
                                : __bfloat162float(xrow_s[s.d + c.idx_comp_v[(size_t)h * s.dcv + i - s.dck]]);
#pragma unroll 1
        for (int r = tid; r < min(m1 - m0, kPendRows); r += kAll) f_s[r] = basis_value(m0 + r, j_pend, s.T);
    }
    // basis value of row r of this part (tabulated for the first kPendRows rows)
    auto f_row = [&](int r) -> float {
        return r < kPendRows ? f_s[r] : basis_value(m0 + r, j_pend, s.T);
    };

    // B fragments of q for the kept K dims: column gq is slot gq = head hperm(gq);
    // round rd covers pieces 4 rd + tq of a row, two k-steps each
    const int my_head = hperm<GH>(gq & (GH - 1));
    const bool col_on = gq < GH && my_head < ng;
    const bf16* qrow = qs_s + my_head * s.d;
    uint32_t qk[2][2][2];
    {
        const int32_t* idf_k = c.idx_full_k + (size_t)h * s.nfk;
#pragma unroll
        for (int rd = 0; rd < 2; ++rd)
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const int piece = 4 * rd + tq, e0 = 8 * piece + 4 * ks;
                const bool on = col_on && piece < npk;
                qk[rd][ks][0] = on ? pack_bf16(qrow[idf_k[e0]], qrow[idf_k[e0 + 1]]) : 0u;
                qk[rd][ks][1] = on ? pack_bf16(qrow[idf_k[e0 + 2]], qrow[idf_k[e0 + 3]]) : 0u;
            }
    }
    int it = 0;                                           // tile counter, mirrors the producer's

    auto wait_tile = [&]() -> const unsigned char* {
        const int st = it % NS;
        mbar_wait(full + st, (it / NS) & 1, fail, c.status);
        return stages + (size_t)st * kStageBytes;
    };
    const uint32_t stages_u = smem_addr(stages), zero_u = smem_addr(zero16);
    auto wait_tile_u = [&]() -> uint32_t {                // the same, as a shared-memory address
        const int st = it % NS;
        mbar_wait(full + st, (it / NS) & 1, fail, c.status);
        return stages_u + (uint32_t)st * kStageBytes;
    };
    auto release_tile = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + (it % NS));
        ++it;
    };
    // kept dims of one batch of classes: kb[class][token][slot] = sl2 * (q_u . K^mu), 16 tokens per mma.
    // It needs nothing but q, so the first batch runs before u is known.
    // per-lane constants of the K loop: byte offsets of the two 16-byte pieces inside a 16-row group
    uint32_t k_off[2];
    bool k_on[2];
#pragma unroll
    for (int rd = 0; rd < 2; ++rd) {
        k_off[rd] = (uint32_t)(gq * rowb_k + 16 * (4 * rd + tq));
        k_on[rd] = 4 * rd + tq < npk;
    }
    const uint32_t kb_lane_off = (uint32_t)(gq * GH + 2 * tq) * 4;
    auto k_phase = [&](int cb, int nb, float* kbuf) {
        if (!ts_k || !is_m) return;
#pragma unroll 1
        for (int ci = 0; ci < nb; ++ci) {
            const int n_c = n_of_class(cb + ci);
#pragma unroll 1
            for (int a0 = 0; a0 < n_c; a0 += ts_k) {
                const int nt = min(ts_k, n_c - a0);
                const uint32_t tile = wait_tile_u();
#pragma unroll 1
                for (int grp = wm; grp * 16 < nt; grp += kMW) {
                    const uint32_t gbase = tile + (uint32_t)(grp * 16) * rowb_k;
                    if (STEP && cb + ci == cstar && astar >= a0 + grp * 16 && astar < a0 + grp * 16 + 16) {
                        // fused step: middle token j_pend is not in the cache yet; its kept dims from the row that leaves the window
                        patch_mid_k(tile + (uint32_t)((astar - a0) * rowb_k), c.idx_full_k + (size_t)h * s.nfk, s.nfk, xrow_s, lane);
                    }
                    float d4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int rd = 0; rd < 2; ++rd) {
                        if (4 * rd < npk) {
                            uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
                            if (k_on[rd]) {
                                lo = lds128(gbase + k_off[rd]);
                                hi = lds128(gbase + k_off[rd] + 8 * rowb_k);
                            }
                            mma_bf16(d4, lo.x, hi.x, lo.y, hi.y, qk[rd][0][0], qk[rd][0][1]);
                            mma_bf16(d4, lo.z, hi.z, lo.w, hi.w, qk[rd][1][0], qk[rd][1][1]);
                        }
                    }
                    if (cp) {
                        if (tq == 0) {                      // the head's column, to the slot of this class in its pair
                            float* dst = kbuf + (((ci >> 1) * S + a0 + grp * 16 + gq) * GH + (ci & 1));
                            dst[0] = d4[0] * sl2;
                            dst[8 * GH] = d4[2] * sl2;
                        }
                    } else if (2 * tq < GH) {
                        const uint32_t dst = smem_addr(kbuf) + kb_lane_off + (uint32_t)((ci * S + a0 + grp * 16) * GH) * 4;
                        sts64(dst, d4[0] * sl2, d4[1] * sl2);
                        sts64(dst + 8 * GH * 4, d4[2] * sl2, d4[3] * sl2);
                    }
                }
                release_tile();
            }
        }
    };
    const bool has_classes = !is_win && c0 < c1 && n_of_class(c0) > 0;
    // Fused kernel: this part's rows of u first, then the kept-dim scores of the first batch (they need
    // only q) while the other parts finish theirs, then the wait for all of u.
    if (p.fused) {
        // u_g[m] = scale * log2(e) * w_m * sum_e C^K[m][e] q_g[D^kc[e]] for rows [m0, m1): eight lanes per row
        if (s.dck > 0) {
            float* qc = reinterpret_cast<float*>(o_s);     // [GH][dck] gathered query, fp32 (o_s is not in use yet)
            const int32_t* idc_k = c.idx_comp_k + (size_t)h * s.dck;
            for (int i = tid; i < GH * s.dck; i += kAll) {
                const int g = i / s.dck, e = i - g * s.dck;
                qc[i] = i < kAll ? qc_early : (g < ng ? __bfloat162float(qs_s[g * s.d + idc_k[e]]) : 0.f);
            }
            const int l8 = tid & 7, rgi = tid >> 3, nv = s.dck >> 2;
            float* ckg = coef_rows(c.coef_k, s, b, h, s.dck);
#pragma unroll 1
            for (int q0 = m0; q0 < m1; q0 += uch) {         // chunks of rows staged in the transform buffers
                const int q1 = min(m1, q0 + uch);
                if (q0 > m0) {
                    all_sync();
#pragma unroll 1
                    for (int i = tid; i < (q1 - q0) * nv; i += kAll) cp_async16(fbuf + 4 * i, ckg + (size_t)q0 * s.dck + 4 * i);
                }
                cp_async_wait_all();
                all_sync();
#pragma unroll 1
                for (int r0 = q0; r0 < q1; r0 += kAll / 8) {
                    const int r = r0 + rgi;
                    float a[GH];
#pragma unroll
                    for (int g = 0; g < GH; ++g) a[g] = 0.f;
                    if (r < q1) {
                        const float4* row = reinterpret_cast<const float4*>(fbuf + (r - q0) * s.dck);
                        // fused step: the rank-1 update of Eq.5 that the light append kernel left pending, applied to
                        // each piece of this part's rows as it passes here (exactly once), and written back
                        const float f = j_pend >= 0 ? f_row(r - m0) : 0.f;
#pragma unroll 1
                        for (int v = l8; v < nv; v += 8) {
                            float4 x = row[v];
                            if (j_pend >= 0) {
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
                    if (r < q1 && l8 < ng)
                        ws.u[((size_t)b * s.Hq + g_first + l8) * s.M + r] = recon_weight(s.norm, r, s.k, s.T) * sl2 * mine;
                }
            }
            TL(2);
            part_arrive<kAll>(bar + 0, p.n_part, tid);
        }
        TL(3);
        if (has_classes) k_phase(c0, min(NB, c1 - c0), kb);
        TL(4);
        if (s.dck > 0 && !is_win) part_wait<kAll>(bar + 0, p.n_part, tid, fail, c.status);
        TL(5);
    } else {
        if (has_classes) k_phase(c0, min(NB, c1 - c0), kb);
        // everything above is independent of the prologue kernel; its output u is first needed here
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    for (int i = tid; i < GH * s.d; i += kAll) o_s[i] = 0;
    // ut[n] = (A.re, A.im, B.re, B.im), A = heads of the real slots, B = heads of the imaginary slots;
    // all loads of an entry are issued together
    #pragma unroll 1
    for (int n = tid; n < s.k; n += kAll) {
        float2 uv[GH];
#pragma unroll
        for (int sl = 0; sl < GH; ++sl) {
            const int g = hperm<GH>(sl);
            uv[sl] = make_float2(0.f, 0.f);
            if (g < ng && s.dck > 0 && !is_win) uv[sl] = __ldcg(reinterpret_cast<const float2*>(ws.u + ((size_t)b * s.Hq + g_first + g) * s.M + 2 * n));
        }
        float* e = ut + n * 2 * GH;
        float* zz = z_s + n * 2 * GH;
#pragma unroll
        for (int sl = 0; sl < GH; ++sl) {
            const int ab = sl / N, ln = sl - ab * N;
            e[(2 * ab) * N + ln] = 0.5f * uv[sl].x;
            e[(2 * ab + 1) * N + ln] = -0.5f * uv[sl].y;
            zz[(2 * ab) * N + ln] = 0.f;
            zz[(2 * ab + 1) * N + ln] = 0.f;
        }
    }
    all_sync();

    float m_run[GH], l_acc[GH];                           // per slot
#pragma unroll
    for (int g = 0; g < GH; ++g) { m_run[g] = kNegBig; l_acc[g] = 0.f; }
    // per-slot maximum over per-thread partial maxima, broadcast to every consumer thread
    auto block_max = [&](float (&mx)[GH]) {
#pragma unroll
        for (int g = 0; g < GH; ++g) {
            float v = mx[g];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
            if (lane == 0) red_s[warp * GH + g] = v;
        }
        all_sync();
#pragma unroll
        for (int g = 0; g < GH; ++g) {
            float r = red_s[g];
#pragma unroll
            for (int w = 1; w < kAllW; ++w) r = fmaxf(r, red_s[w * GH + g]);
            mx[g] = r;
        }
    };
    auto load_vals = [&](const float* pt, float (&v)[GH]) {
        if constexpr (GH == 4) {
            const float4 x = *reinterpret_cast<const float4*>(pt);
            v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
        } else {
            const float2 x = *reinterpret_cast<const float2*>(pt);
            v[0] = x.x; v[1] = x.y;
        }
    };
    auto store_vals = [&](float* pt, const float (&v)[GH]) {
        if constexpr (GH == 4) *reinterpret_cast<float4*>(pt) = make_float4(v[0], v[1], v[2], v[3]);
        else *reinterpret_cast<float2*>(pt) = make_float2(v[0], v[1]);
    };
    // entry n of ut / z_s as two packed complex numbers
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
    const PC<N> czero = PC<N>{splat<N>(0.f), splat<N>(0.f)};
    auto seed_tw = [&](int n, int cls) -> float2 {
        return cis_frac((float)((n * cls) & (s.T - 1)) / (float)s.T);
    };

    // fused step: writes the new token's row (all d dims) over row `prow` of a window tile (128-byte swizzle), by one warp
    auto patch_win = [&](const unsigned char* tile, int prow, const bf16* src) {
#pragma unroll 1
        for (int cc = lane; cc < npw; cc += 32)
            *reinterpret_cast<uint4*>(const_cast<unsigned char*>(tile) + (cc >> 3) * kWinHalfBytes + prow * 128 + (((cc & 7) ^ (prow & 7)) << 4)) =
                *reinterpret_cast<const uint4*>(src + 8 * cc);
        __syncwarp();
    };

    TL(6);
    // ------------------------------ window tokens -------------------------------
    if (w1 > w0) {
        uint32_t qw[4][2][2];
#pragma unroll
        for (int rd = 0; rd < 4; ++rd)
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                // round rd covers the 16-byte pieces 2 tq + (rd & 1) of half rd >> 1: with the 128-byte
                // swizzle the eight lanes of a quarter warp (two rows) then hit eight different bank groups
                const int piece = ((rd >> 1) << 3) + 2 * tq + (rd & 1), e0 = 8 * piece + 4 * ks;
                const bool on = col_on && piece < npw;
                qw[rd][ks][0] = on ? pack_bf16(qrow[e0], qrow[e0 + 1]) : 0u;
                qw[rd][ks][1] = on ? pack_bf16(qrow[e0 + 2], qrow[e0 + 3]) : 0u;
            }
        float accw[8][4];
#pragma unroll
        for (int mt = 0; mt < 8; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) accw[mt][i] = 0.f;
        const int nmtw = (s.d + 15) >> 4;
        float* sb = fbuf;                                 // natural order, no transform
        bf16* pb = pbt;
        #pragma unroll 1
        for (int t0 = w0; t0 < w1; t0 += wchunk) {
            const int n_tok = min(w1, t0 + wchunk) - t0;
            const WinSegs sg = win_segments(t0, t0 + n_tok, n_init, n_local, head, s.l_local);
            #pragma unroll 1
            for (int si = 0; si < sg.n; ++si)
                #pragma unroll 1
                for (int r0 = 0; r0 < sg.cnt[si]; r0 += ts_w) {
                    const int nt = min(ts_w, sg.cnt[si] - r0);
                    if (!is_m) continue;
                    const unsigned char* tile = wait_tile();
                    const int nrow = new_buf == sg.buf[si] ? new_row - (sg.row[si] + r0) : -1;   // fused step: the new token's row in this tile
                    #pragma unroll 1
                    for (int grp = (wm + kMW - (it * (kWinRowsPerTile / 16)) % kMW) % kMW; grp * 16 < nt; grp += kMW) {   // tiles rotate over the warps
                        if (STEP && nrow >= grp * 16 && nrow < grp * 16 + 16) patch_win(tile, nrow, knew_bh);
                        const unsigned char* r_lo = tile + (size_t)(grp * 16 + gq) * 128;      // row & 7 == gq for both rows
                        float d4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int rd = 0; rd < 4; ++rd) {
                            const int cj = 2 * tq + (rd & 1), piece = ((rd >> 1) << 3) + cj;
                            if (((rd >> 1) << 3) < npw) {
                                uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
                                if (piece < npw) {
                                    const unsigned char* src = r_lo + (rd >> 1) * kWinHalfBytes + ((cj ^ gq) << 4);
                                    lo = *reinterpret_cast<const uint4*>(src);
                                    hi = *reinterpret_cast<const uint4*>(src + 8 * 128);
                                }
                                mma_bf16(d4, lo.x, hi.x, lo.y, hi.y, qw[rd][0][0], qw[rd][0][1]);
                                mma_bf16(d4, lo.z, hi.z, lo.w, hi.w, qw[rd][1][0], qw[rd][1][1]);
                            }
                        }
                        if (2 * tq < GH) {
                            const int i_lo = grp * 16 + gq, i_hi = i_lo + 8;
                            if (i_lo < nt)
                                *reinterpret_cast<float2*>(sb + pf((sg.tok[si] + r0 + i_lo) * GH + 2 * tq)) = make_float2(d4[0] * sl2, d4[1] * sl2);
                            if (i_hi < nt)
                                *reinterpret_cast<float2*>(sb + pf((sg.tok[si] + r0 + i_hi) * GH + 2 * tq)) = make_float2(d4[2] * sl2, d4[3] * sl2);
                        }
                    }
                    release_tile();
                }
            all_sync();
            float mx[GH], alpha[GH];
#pragma unroll
            for (int g = 0; g < GH; ++g) mx[g] = kNegBig;
            #pragma unroll 1
            for (int a = tid; a < n_tok; a += kAll) {
                float v[GH];
                load_vals(sb + pf(a * GH), v);
#pragma unroll
                for (int g = 0; g < GH; ++g) if (!(cp && g == 1)) mx[g] = fmaxf(mx[g], v[g]);
            }
            block_max(mx);
#pragma unroll
            for (int g = 0; g < GH; ++g) {
                const float m_new = fmaxf(m_run[g], mx[g]);
                alpha[g] = ex2(m_run[g] - m_new);
                m_run[g] = m_new;
                l_acc[g] *= alpha[g];
            }
            const int n_pad = (n_tok + 15) & ~15;
            #pragma unroll 1
            for (int a = tid; a < n_pad; a += kAll) {
                float v[GH];
#pragma unroll
                for (int g = 0; g < GH; ++g) v[g] = 0.f;
                if (a < n_tok) load_vals(sb + pf(a * GH), v);
#pragma unroll
                for (int g = 0; g < GH; ++g) {
                    v[g] = (a < n_tok && !(cp && g == 1)) ? ex2(v[g] - m_run[g]) : 0.f;
                    l_acc[g] += v[g];
                    pb[g * pbw + a] = __float2bfloat16_rn(v[g]);
                }
            }
            {
                const float al = alpha[(2 * tq) & (GH - 1)], ah = alpha[(2 * tq + 1) & (GH - 1)];
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) { accw[mt][0] *= al; accw[mt][1] *= ah; accw[mt][2] *= al; accw[mt][3] *= ah; }
            }
            all_sync();
            const bf16* prow = pb + (size_t)(gq & (GH - 1)) * pbw;
            #pragma unroll 1
            for (int si = 0; si < sg.n; ++si)
                #pragma unroll 1
                for (int r0 = 0; r0 < sg.cnt[si]; r0 += ts_w) {
                    const int nt = min(ts_w, sg.cnt[si] - r0);
                    if (!is_m) continue;
                    const unsigned char* tile = wait_tile();
                    const int nrow = new_buf == sg.buf[si] ? new_row - (sg.row[si] + r0) : -1;
                    #pragma unroll 1
                    for (int grp = (wm + kMW - (it * (kWinRowsPerTile / 16)) % kMW) % kMW; grp * 16 < nt; grp += kMW) {
                        if (STEP && nrow >= grp * 16 && nrow < grp * 16 + 16) patch_win(tile, nrow, vnew_bh);
                        const int a = sg.tok[si] + r0 + grp * 16;
                        // the tile's rows may start at any token of the chunk: gather the four p values one by one
                        uint32_t b0 = 0, b1 = 0;
                        if (gq < GH) {
                            const int rem = nt - grp * 16;
                            const bf16 zero = __float2bfloat16_rn(0.f);
                            b0 = pack_bf16(2 * tq < rem ? prow[a + 2 * tq] : zero, 2 * tq + 1 < rem ? prow[a + 2 * tq + 1] : zero);
                            b1 = pack_bf16(2 * tq + 8 < rem ? prow[a + 2 * tq + 8] : zero, 2 * tq + 9 < rem ? prow[a + 2 * tq + 9] : zero);
                        }
                        if (nt - grp * 16 < 16) {
                            // rows past the end of the segment hold whatever follows it in the cache: zero them,
                            // p = 0 does not stop a NaN
                            const int rem = nt - grp * 16, per_row = nhalf * 8;
                            #pragma unroll 1
                            for (int i = lane; i < (16 - rem) * per_row; i += 32) {
                                const int rr = grp * 16 + rem + i / per_row, cc = i % per_row;
                                *reinterpret_cast<uint4*>(const_cast<unsigned char*>(tile) + (cc >> 3) * kWinHalfBytes + rr * 128 + ((cc & 7) << 4)) =
                                    make_uint4(0, 0, 0, 0);
                            }
                            __syncwarp();
                        }
                        const int mi = lane >> 3, tok = ((mi >> 1) << 3) + (lane & 7);
                        const unsigned char* vrow = tile + (size_t)(grp * 16 + tok) * 128;
#pragma unroll
                        for (int mt = 0; mt < 8; ++mt) {
                            if (mt < nmtw) {
                                const int chunk = 2 * mt + (mi & 1);
                                const unsigned char* src = chunk < npw ? vrow + (chunk >> 3) * kWinHalfBytes + (((chunk & 7) ^ (tok & 7)) << 4) : zero16;
                                uint32_t af[4];
                                ldmatrix_x4_trans(af, smem_addr(src));
                                mma_bf16(accw[mt], af[0], af[1], af[2], af[3], b0, b1);
                            }
                        }
                    }
                    release_tile();
                }
            all_sync();
        }
        // the window fragments open o_s; the class batches rescale it as the running maximum moves
        if (2 * tq < GH) {
            long long* o_lo = o_s + hperm<GH>(2 * tq) * s.d;
            long long* o_hi = o_s + hperm<GH>(2 * tq + 1) * s.d;
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                const int e_lo = 16 * mt + gq, e_hi = e_lo + 8;
                if (e_lo < s.d) { fix_add(o_lo + e_lo, accw[mt][0]); fix_add(o_hi + e_lo, accw[mt][1]); }
                if (e_hi < s.d) { fix_add(o_lo + e_hi, accw[mt][2]); fix_add(o_hi + e_hi, accw[mt][3]); }
            }
        }
    }
    all_sync();

    TL(7);
    // ------------------------------ middle classes ------------------------------
    {
        float acc[4][4];                                  // [m-tile of 16 dims][mma D fragment]
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
        const int nmt = (s.nfv + 15) >> 4;
        // per-lane constants of the V loop.  A group of 16 tokens starts at a multiple of 16, so the
        // chunk swizzle of a lane's row depends on the lane alone: the byte offset of its 8x8 matrix
        // row inside the group is fixed.  A chunk past the end of the row reads the zero block.
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
        const uint32_t p_lane = smem_addr(pbt) + (uint32_t)((gq & (GH - 1)) * pbs + 2 * tq) * 2;
        // natural positions of this lane's output rows (D^vu), fetched long before they are needed
        int o_idx[4][2];
        {
            const int32_t* idf_v = c.idx_full_v + (size_t)h * s.nfv;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const int e_lo = 16 * mt + gq, e_hi = e_lo + 8;
                o_idx[mt][0] = e_lo < s.nfv ? idf_v[e_lo] : -1;
                o_idx[mt][1] = e_hi < s.nfv ? idf_v[e_hi] : -1;
            }
        }

        if constexpr (!SPLIT) {
        if (cp) {
            // a class has one row of probabilities, read by its own slot; the other slot reads the row of zeros behind them
            #pragma unroll 1
            for (int i = tid; i < pbs / 2; i += kAll) reinterpret_cast<uint32_t*>(pbt + NB * pbs)[i] = 0u;
            all_sync();
        }
        #pragma unroll 1
        for (int cb = c0; cb < c1; cb += NB) {
            const int nb = min(NB, c1 - cb);
            if (n_of_class(cb) == 0) break;               // classes are filled in order: nothing further on
            if (cb != c0) k_phase(cb, nb, kb);
            // transforms of the batch, and classes from one transform to the next
            const int nbt = cp ? (nb + 1) >> 1 : nb, cstep = cp ? 2 : 1;

            // packed Hermitian spectra of the nb classes: X_m = V^A_m + i V^B_m per complex lane,
            // V_m = v_m + conj(v_{S-m}), v_n = (1/2) u~_n e^{i theta n c}.  Pair 0 is bins (0, S/2).
            if (s.dck > 0) {
                // neighbouring lanes share a pair of bins and take half of the classes each (a batch of one
                // class: one lane per pair, half as many rounds)
                const bool split2 = nbt > 1;
                const int hcls = split2 ? (nbt + 1) >> 1 : nbt;
                #pragma unroll 1
                for (int item = tid; item < (split2 ? S : S / 2); item += kAll) {
                    const int pr = split2 ? item >> 1 : item, ci0 = split2 ? (item & 1) * hcls : 0, ci1 = min(nbt, ci0 + hcls);
                    const int m = pr, mc = pr == 0 ? S / 2 : S - pr;
                    PC<N> Am = czero, Bm = czero, Ac = czero, Bc = czero;
                    float2 em = make_float2(1.f, 0.f), ec = make_float2(1.f, 0.f);
                    if (m < s.k) { ld_entry(ut, m, Am, Bm); em = E[m]; }
                    if (mc < s.k) { ld_entry(ut, mc, Ac, Bc); ec = E[mc]; }
                    float2 twm = seed_tw(m, cb + cstep * ci0), twc = seed_tw(mc, cb + cstep * ci0);
                    // class pairs: both slots are the head; slot 1 is one class further on
                    const float2 em1 = em, ec1 = ec;
                    if (cp) { Bm = Am; Bc = Ac; em = cmulf(em, em); ec = cmulf(ec, ec); }
                    #pragma unroll 1
                    for (int ci = ci0; ci < ci1; ++ci) {
                        const PR<N> wmr = splat<N>(twm.x), wmi = splat<N>(twm.y), wcr = splat<N>(twc.x), wci = splat<N>(twc.y);
                        const float2 twmB = cp ? cmulf(twm, em1) : twm, twcB = cp ? cmulf(twc, ec1) : twc;
                        const PC<N> vAm = cmulw(Am, wmr, wmi), vBm = cmulw(Bm, splat<N>(twmB.x), splat<N>(twmB.y));
                        const PC<N> vAc = cmulw(Ac, wcr, wci), vBc = cmulw(Bc, splat<N>(twcB.x), splat<N>(twcB.y));
                        float* base = fbuf + ci * fb_floats;
                        if (pr != 0) {
                            const PC<N> VA = cconj_add(vAm, vAc), VB = cconj_add(vBm, vBc);
                            st_pt(base + pf(m * GH), PC<N>{VA.re - VB.im, VA.im + VB.re});        // V^A + i V^B
                            st_pt(base + pf(mc * GH), PC<N>{VA.re + VB.im, VB.re - VA.im});       // conj(V^A) + i conj(V^B)
                        } else {                                                                   // self-conjugate bins
                            const PC<N> VA0 = cconj_add(vAm, vAm), VB0 = cconj_add(vBm, vBm);
                            const PC<N> VA1 = cconj_add(vAc, vAc), VB1 = cconj_add(vBc, vBc);
                            st_pt(base + pf(0), PC<N>{VA0.re - VB0.im, VA0.im + VB0.re});
                            st_pt(base + pf((S / 2) * GH), PC<N>{VA1.re - VB1.im, VA1.im + VB1.re});
                        }
                        twm = cmulf(twm, em);
                        twc = cmulf(twc, ec);
                    }
                }
                all_sync();
                if (cb == c0) TL(8);
                fft_run<GH, LS, LS, false>(fbuf, fb_floats, nbt, twf, tid);       // score of slot a at point rev[a]
                if (cb == c0) TL(9);
            } else {
                #pragma unroll 1
                for (int i = tid; i < nbt * fb_floats; i += kAll) fbuf[i] = 0.f;
                all_sync();
            }

            all_sync();

            // online softmax over the batch
            float mx[GH], alpha[GH];
#pragma unroll
            for (int g = 0; g < GH; ++g) mx[g] = kNegBig;
            #pragma unroll 1
            for (int i = tid; i < (nbt << LS); i += kAll) {
                const int ci = i >> LS, a = i & (S - 1);
                // class pairs: slot g of the point is token a of class cstep ci + g
                const bool ok0 = a < n_of_class(cb + cstep * ci);
                const bool ok1 = cp ? (2 * ci + 1 < nb && a < n_of_class(cb + 2 * ci + 1)) : ok0;
                if (ok0 || ok1) {
                    // score = compressed part (transform output) + kept part
                    float* pt = fbuf + ci * fb_floats + pf(rev[a] * GH);
                    float v[GH], kv[GH];
                    load_vals(pt, v);
                    if (ts_k) {
                        load_vals(kb + (size_t)i * GH, kv);
#pragma unroll
                        for (int g = 0; g < GH; ++g) v[g] += kv[g];
                        store_vals(pt, v);
                    }
#pragma unroll
                    for (int g = 0; g < GH; ++g) if (g == 1 ? ok1 : ok0) mx[g] = fmaxf(mx[g], v[g]);
                }
            }
            block_max(mx);
#pragma unroll
            for (int g = 0; g < GH; ++g) {
                const float m_new = fmaxf(m_run[g], mx[g]);
                alpha[g] = ex2(m_run[g] - m_new);
                m_run[g] = m_new;
                l_acc[g] *= alpha[g];
            }
            #pragma unroll 1
            for (int i = tid; i < (nbt << LS); i += kAll) {
                const int ci = i >> LS, a = i & (S - 1);
                float* pt = fbuf + ci * fb_floats + pf(rev[a] * GH);
                float v[GH];
                load_vals(pt, v);
                const bool ok0 = a < n_of_class(cb + cstep * ci);
                const bool ok1 = cp ? (2 * ci + 1 < nb && a < n_of_class(cb + 2 * ci + 1)) : ok0;
#pragma unroll
                for (int g = 0; g < GH; ++g) {
                    v[g] = (g == 1 ? ok1 : ok0) ? ex2(v[g] - m_run[g]) : 0.f;
                    l_acc[g] += v[g];
                    if (!cp) pbt[(ci * GH + g) * pbs + a] = __float2bfloat16_rn(v[g]);
                    else if (2 * ci + g < nb) pbt[(2 * ci + g) * pbs + a] = __float2bfloat16_rn(v[g]);
                }
                store_vals(pt, v);
            }
            {
                const float al = alpha[(2 * tq) & (GH - 1)], ah = alpha[(2 * tq + 1) & (GH - 1)];
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) { acc[mt][0] *= al; acc[mt][1] *= ah; acc[mt][2] *= al; acc[mt][3] *= ah; }
            }
            for (int i = tid; i < GH * s.d; i += kAll) {          // what the windows left in o_s (rows are heads)
                const int g = i / s.d;
                float a = alpha[0];
#pragma unroll
                for (int sl = 1; sl < GH; ++sl) if (hperm<GH>(sl) == g) a = alpha[sl];
                o_s[i] = __float2ll_rn(__ll2float_rn(o_s[i]) * a);
            }
            all_sync();

            if (cb == c0) TL(10);
            // o^u[dim][slot] += V^mu^T p, 16 tokens per mma
            if (ts_v) {
                #pragma unroll 1
                for (int ci = 0; ci < nb; ++ci) {
                    const int n_c = n_of_class(cb + ci);
                    const uint32_t prow = cp ? smem_addr(pbt) + (uint32_t)((((gq & 1) == (ci & 1) ? ci : NB) * pbs) + 2 * tq) * 2
                                             : p_lane + (uint32_t)(ci * GH * pbs) * 2;
                    #pragma unroll 1
                    for (int a0 = 0; a0 < n_c; a0 += ts_v) {
                        const int nt = min(ts_v, n_c - a0);
                        const uint32_t tile = wait_tile_u();
                        #pragma unroll 1
                        for (int grp = wm; grp * 16 < nt; grp += kMW) {
                            const uint32_t gbase = tile + (uint32_t)(grp * 16) * rowb_v;
                            if (STEP && cb + ci == cstar && astar >= a0 + grp * 16 && astar < a0 + grp * 16 + 16) {
                                patch_mid_v(tile + (uint32_t)((astar - a0) * rowb_v), c.idx_full_v + (size_t)h * s.nfv, s.nfv, xrow_s + s.d, astar, lane);
                            }
                            uint32_t b0 = 0, b1 = 0;
                            if (gq < GH) {
                                b0 = lds32(prow + (uint32_t)(a0 + grp * 16) * 2);
                                b1 = lds32(prow + (uint32_t)(a0 + grp * 16 + 8) * 2);
                            }
#pragma unroll
                            for (int mt = 0; mt < 4; ++mt) {
                                if (mt < nmt) {
                                    uint32_t af[4];
                                    ldmatrix_x4_trans(af, v_off[mt] + gbase * v_mul[mt]);
                                    mma_bf16(acc[mt], af[0], af[1], af[2], af[3], b0, b1);
                                }
                            }
                        }
                        release_tile();
                    }
                }
            }

            if (cb == c0) TL(11);
            // z_n = alpha z_n + sum_c e^{i theta n c} Y^c_n, Y^c = transform of the packed probabilities
            if (s.dcv > 0) {
                fft_run<GH, LS, LS, true>(fbuf, fb_floats, nbt, twf, tid);
                if (cb == c0) TL(12);
                PR<N> alA, alB;
                if constexpr (N == 2) { alA = pk(alpha[0], alpha[1]); alB = pk(alpha[2], alpha[3]); }
                else { alA = PR<1>{alpha[0]}; alB = PR<1>{alpha[1]}; }
                const PR<N> half = splat<N>(0.5f);
                const bool split2 = nbt > 1;               // as for the spectra: one lane per pair when the batch is one transform
                const int hcls = split2 ? (nbt + 1) >> 1 : nbt;
                #pragma unroll 1
                for (int item = tid; item < (split2 ? S : S / 2); item += kAll) {       // split: whole warps (S is a multiple of 32)
                    const int pr = split2 ? item >> 1 : item, ci0 = split2 ? (item & 1) * hcls : 0;
                    const int m = pr, mc = pr == 0 ? S / 2 : S - pr;
                    const int ci1 = (m >= s.k && mc >= s.k) ? ci0 : min(nbt, ci0 + hcls);
                    float2 em = make_float2(1.f, 0.f), ec = make_float2(1.f, 0.f);
                    if (m < s.k) em = E[m];
                    if (mc < s.k) ec = E[mc];
                    float2 twm = seed_tw(m, cb + cstep * ci0), twc = seed_tw(mc, cb + cstep * ci0);
                    const float2 em1 = em, ec1 = ec;        // class pairs: slot 1 is one class further on than slot 0
                    if (cp) { em = cmulf(em, em); ec = cmulf(ec, ec); }
                    PC<N> zAm = czero, zBm = czero, zAc = czero, zBc = czero;
                    #pragma unroll 1
                    for (int ci = ci0; ci < ci1; ++ci) {
                        const float* base = fbuf + ci * fb_floats;
                        const PC<N> ya = ld_pt<N>(base + pf(m * GH)), yb = ld_pt<N>(base + pf(mc * GH));
                        const PR<N> wmr = splat<N>(twm.x), wmi = splat<N>(twm.y), wcr = splat<N>(twc.x), wci = splat<N>(twc.y);
                        const float2 twmB = cp ? cmulf(twm, em1) : twm, twcB = cp ? cmulf(twc, ec1) : twc;
                        const PR<N> wmrB = splat<N>(twmB.x), wmiB = splat<N>(twmB.y), wcrB = splat<N>(twcB.x), wciB = splat<N>(twcB.y);
                        if (pr != 0) {
                            // real slots: y0 = (ya + conj(yb)) / 2, imaginary slots: y1 = (ya - conj(yb)) / (2 i); bin mc holds the conjugates
                            const PC<N> y0 = PC<N>{(ya.re + yb.re) * half, (ya.im - yb.im) * half};
                            const PC<N> y1 = PC<N>{(ya.im + yb.im) * half, (yb.re - ya.re) * half};
                            zAm = zAm + cmulw(y0, wmr, wmi);
                            zBm = zBm + cmulw(y1, wmrB, wmiB);
                            zAc = zAc + cmulw(PC<N>{y0.re, splat<N>(0.f) - y0.im}, wcr, wci);
                            zBc = zBc + cmulw(PC<N>{y1.re, splat<N>(0.f) - y1.im}, wcrB, wciB);
                        } else {
                            // bins 0 and S/2 are real for each real sequence: (re, im) of the packed value are the two heads
                            const PC<N> y0m = PC<N>{ya.re, splat<N>(0.f)}, y1m = PC<N>{ya.im, splat<N>(0.f)};
                            const PC<N> y0c = PC<N>{yb.re, splat<N>(0.f)}, y1c = PC<N>{yb.im, splat<N>(0.f)};
                            zAm = zAm + cmulw(y0m, wmr, wmi);
                            zBm = zBm + cmulw(y1m, wmrB, wmiB);
                            zAc = zAc + cmulw(y0c, wcr, wci);
                            zBc = zBc + cmulw(y1c, wcrB, wciB);
                        }
                        twm = cmulf(twm, em);
                        twc = cmulf(twc, ec);
                    }
                    if (split2) {
                        zAm = pair_sum(zAm); zBm = pair_sum(zBm); zAc = pair_sum(zAc); zBc = pair_sum(zBc);
                        if (item & 1) continue;
                    }
                    if (m < s.k) {
                        PC<N> A, B;
                        ld_entry(z_s, m, A, B);
                        st_entry(z_s, m, PC<N>{pfma(A.re, alA, zAm.re), pfma(A.im, alA, zAm.im)},
                                 PC<N>{pfma(B.re, alB, zBm.re), pfma(B.im, alB, zBm.im)});
                    }
                    if (mc < s.k) {
                        PC<N> A, B;
                        ld_entry(z_s, mc, A, B);
                        st_entry(z_s, mc, PC<N>{pfma(A.re, alA, zAc.re), pfma(A.im, alA, zAc.im)},
                                 PC<N>{pfma(B.re, alB, zBc.re), pfma(B.im, alB, zBc.im)});
                    }
                }
            }
            all_sync();
        }
        } else {
            // ---- split kernel: the tile group (kept-dim products) beside the transform group, batch by batch ----
            // kb_full (tile group -> transform group: the kept-dim scores of the batch are in), kb_free (back: softmax has
            // read them), p_full (transform group -> tile group: probabilities and the rescale factors of the batch are
            // in), p_free (back: the V products have read them).  The scores of a batch are formed under its spectra and
            // score transform, its V products run under its probability transform and fold (and the next batch's
            // scores under that batch's spectra).  Batch 0's scores were formed before the window tokens.
            uint64_t* kb_full = reinterpret_cast<uint64_t*>(smem_raw + 160);
            uint64_t* kb_free = kb_full + 1;
            uint64_t* p_full = kb_full + 2;
            uint64_t* p_free = kb_full + 3;
            float* alpha_s = reinterpret_cast<float*>(smem_raw + 224);     // [GH] rescale factors of a batch, per slot
            auto xf_sync = [] { consumer_sync<kConsumers, 2>(); };
            int n_bat = 0;
            for (int cb = c0; cb < c1 && n_of_class(cb) > 0; cb += NB) ++n_bat;
            if (is_m) {
                // ================= tile group =================
                #pragma unroll 1
                for (int bi = 0; bi < n_bat; ++bi) {
                    const int cb = c0 + bi * NB, nb = min(NB, c1 - cb);
                    if (bi >= 1) {
                        if (lane == 0) mbar_wait(kb_free, (bi - 1) & 1, fail, c.status);   // softmax of the previous batch has read the scores
                        __syncwarp();
                        k_phase(cb, nb, kb);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(kb_full);
                    }
                    if (lane == 0) mbar_wait(p_full, bi & 1, fail, c.status);   // one lane polls, the warp follows
                    __syncwarp();
                    {
                        const float al = alpha_s[(2 * tq) & (GH - 1)], ah = alpha_s[(2 * tq + 1) & (GH - 1)];
#pragma unroll
                        for (int mt = 0; mt < 4; ++mt) { acc[mt][0] *= al; acc[mt][1] *= ah; acc[mt][2] *= al; acc[mt][3] *= ah; }
#pragma unroll
                        for (int g = 0; g < GH; ++g) l_acc[g] *= alpha_s[g];
                    }
            // o^u[dim][slot] += V^mu^T p, 16 tokens per mma
            if (ts_v) {
                #pragma unroll 1
                for (int ci = 0; ci < nb; ++ci) {
                    const int n_c = n_of_class(cb + ci);
                    const uint32_t prow = p_lane + (uint32_t)(ci * GH * pbs) * 2;
                    #pragma unroll 1
                    for (int a0 = 0; a0 < n_c; a0 += ts_v) {
                        const int nt = min(ts_v, n_c - a0);
                        const uint32_t tile = wait_tile_u();
                        #pragma unroll 1
                        for (int grp = wm; grp * 16 < nt; grp += kMW) {
                            const uint32_t gbase = tile + (uint32_t)(grp * 16) * rowb_v;
                            if (STEP && cb + ci == cstar && astar >= a0 + grp * 16 && astar < a0 + grp * 16 + 16) {
                                patch_mid_v(tile + (uint32_t)((astar - a0) * rowb_v), c.idx_full_v + (size_t)h * s.nfv, s.nfv, xrow_s + s.d, astar, lane);
                            }
                            uint32_t b0 = 0, b1 = 0;
                            if (gq < GH) {
                                b0 = lds32(prow + (uint32_t)(a0 + grp * 16) * 2);
                                b1 = lds32(prow + (uint32_t)(a0 + grp * 16 + 8) * 2);
                            }
#pragma unroll
                            for (int mt = 0; mt < 4; ++mt) {
                                if (mt < nmt) {
                                    uint32_t af[4];
                                    ldmatrix_x4_trans(af, v_off[mt] + gbase * v_mul[mt]);
                                    mma_bf16(acc[mt], af[0], af[1], af[2], af[3], b0, b1);
                                }
                            }
                        }
                        release_tile();
                    }
                }
            }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(p_free);
                }
            } else {
                // ================= transform group =================
                // per-slot maximum over the group's threads (as block_max, on the group's barrier)
                auto block_max_t = [&](float (&mx)[GH]) {
#pragma unroll
                    for (int g = 0; g < GH; ++g) {
                        float v = mx[g];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
                        if (lane == 0) red_s[warp * GH + g] = v;
                    }
                    xf_sync();
#pragma unroll
                    for (int g = 0; g < GH; ++g) {
                        float r = red_s[g];
#pragma unroll
                        for (int w = 1; w < kWarps; ++w) r = fmaxf(r, red_s[w * GH + g]);
                        mx[g] = r;
                    }
                };
                #pragma unroll 1
                for (int bi = 0; bi < n_bat; ++bi) {
                    const int cb = c0 + bi * NB, nb = min(NB, c1 - cb);
                    const float* kbuf = kb;
                    bf16* pbuf = pbt;
            // packed Hermitian spectra of the nb classes: X_m = V^A_m + i V^B_m per complex lane,
            // V_m = v_m + conj(v_{S-m}), v_n = (1/2) u~_n e^{i theta n c}.  Pair 0 is bins (0, S/2).
            if (s.dck > 0) {
                // neighbouring lanes share a pair of bins and take half of the classes each (a batch of one
                // class: one lane per pair, half as many rounds)
                const bool split2 = nb > 1;
                const int hcls = split2 ? (nb + 1) >> 1 : nb;
                #pragma unroll 1
                for (int item = tid; item < (split2 ? S : S / 2); item += kConsumers) {
                    const int pr = split2 ? item >> 1 : item, ci0 = split2 ? (item & 1) * hcls : 0, ci1 = min(nb, ci0 + hcls);
                    const int m = pr, mc = pr == 0 ? S / 2 : S - pr;
                    PC<N> Am = czero, Bm = czero, Ac = czero, Bc = czero;
                    float2 em = make_float2(1.f, 0.f), ec = make_float2(1.f, 0.f);
                    if (m < s.k) { ld_entry(ut, m, Am, Bm); em = E[m]; }
                    if (mc < s.k) { ld_entry(ut, mc, Ac, Bc); ec = E[mc]; }
                    float2 twm = seed_tw(m, cb + ci0), twc = seed_tw(mc, cb + ci0);
                    #pragma unroll 1
                    for (int ci = ci0; ci < ci1; ++ci) {
                        const PR<N> wmr = splat<N>(twm.x), wmi = splat<N>(twm.y), wcr = splat<N>(twc.x), wci = splat<N>(twc.y);
                        const PC<N> vAm = cmulw(Am, wmr, wmi), vBm = cmulw(Bm, wmr, wmi);
                        const PC<N> vAc = cmulw(Ac, wcr, wci), vBc = cmulw(Bc, wcr, wci);
                        float* base = fbuf + ci * fb_floats;
                        if (pr != 0) {
                            const PC<N> VA = cconj_add(vAm, vAc), VB = cconj_add(vBm, vBc);
                            st_pt(base + pf(m * GH), PC<N>{VA.re - VB.im, VA.im + VB.re});        // V^A + i V^B
                            st_pt(base + pf(mc * GH), PC<N>{VA.re + VB.im, VB.re - VA.im});       // conj(V^A) + i conj(V^B)
                        } else {                                                                   // self-conjugate bins
                            const PC<N> VA0 = cconj_add(vAm, vAm), VB0 = cconj_add(vBm, vBm);
                            const PC<N> VA1 = cconj_add(vAc, vAc), VB1 = cconj_add(vBc, vBc);
                            st_pt(base + pf(0), PC<N>{VA0.re - VB0.im, VA0.im + VB0.re});
                            st_pt(base + pf((S / 2) * GH), PC<N>{VA1.re - VB1.im, VA1.im + VB1.re});
                        }
                        twm = cmulf(twm, em);
                        twc = cmulf(twc, ec);
                    }
                }
                xf_sync();
                fft_run<GH, LS, LS, false, 2>(fbuf, fb_floats, nb, twf, tid);        // score of slot a at point rev[a]
            } else {
                #pragma unroll 1
                for (int i = tid; i < nb * fb_floats; i += kConsumers) fbuf[i] = 0.f;
                xf_sync();
            }

                    xf_sync();
                    // the kept-dim scores of this batch (batch 0: formed by everybody's earlier barriers)
                    if (bi >= 1) {
                        if (tid == 0) mbar_wait(kb_full, (bi - 1) & 1, fail, c.status);   // one thread polls
                        xf_sync();
                    }
            // online softmax over the batch
            float mx[GH], alpha[GH];
#pragma unroll
            for (int g = 0; g < GH; ++g) mx[g] = kNegBig;
            #pragma unroll 1
            for (int i = tid; i < (nb << LS); i += kConsumers) {
                const int ci = i >> LS, a = i & (S - 1);
                if (a < n_of_class(cb + ci)) {
                    // score = compressed part (transform output) + kept part
                    float* pt = fbuf + ci * fb_floats + pf(rev[a] * GH);
                    float v[GH], kv[GH];
                    load_vals(pt, v);
                    if (ts_k) {
                        load_vals(kbuf + (size_t)i * GH, kv);
#pragma unroll
                        for (int g = 0; g < GH; ++g) v[g] += kv[g];
                        store_vals(pt, v);
                    }
#pragma unroll
                    for (int g = 0; g < GH; ++g) mx[g] = fmaxf(mx[g], v[g]);
                }
            }
            block_max_t(mx);
#pragma unroll
            for (int g = 0; g < GH; ++g) {
                const float m_new = fmaxf(m_run[g], mx[g]);
                alpha[g] = ex2(m_run[g] - m_new);
                m_run[g] = m_new;
                l_acc[g] *= alpha[g];
            }
            if (bi >= 1) {                                // the tile group is done with the previous batch's probabilities
                if (tid == 0) mbar_wait(p_free, (bi - 1) & 1, fail, c.status);
                xf_sync();
            }
            #pragma unroll 1
            for (int i = tid; i < (nb << LS); i += kConsumers) {
                const int ci = i >> LS, a = i & (S - 1);
                float* pt = fbuf + ci * fb_floats + pf(rev[a] * GH);
                float v[GH];
                load_vals(pt, v);
                const bool ok = a < n_of_class(cb + ci);
#pragma unroll
                for (int g = 0; g < GH; ++g) {
                    v[g] = ok ? ex2(v[g] - m_run[g]) : 0.f;
                    l_acc[g] += v[g];
                    pbuf[(ci * GH + g) * pbs + a] = __float2bfloat16_rn(v[g]);
                }
                store_vals(pt, v);
            }
            for (int i = tid; i < GH * s.d; i += kConsumers) {          // what the windows left in o_s (rows are heads)
                const int g = i / s.d;
                float a = alpha[0];
#pragma unroll
                for (int sl = 1; sl < GH; ++sl) if (hperm<GH>(sl) == g) a = alpha[sl];
                o_s[i] = __float2ll_rn(__ll2float_rn(o_s[i]) * a);
            }
                    if (tid < GH) alpha_s[tid] = alpha[0];
#pragma unroll
                    for (int g = 1; g < GH; ++g) if (tid == g) alpha_s[g] = alpha[g];
                    xf_sync();
                    if (lane == 0) { mbar_arrive(kb_free); mbar_arrive(p_full); }
            // z_n = alpha z_n + sum_c e^{i theta n c} Y^c_n, Y^c = transform of the packed probabilities
            if (s.dcv > 0) {
                fft_run<GH, LS, LS, true, 2>(fbuf, fb_floats, nb, twf, tid);
                PR<N> alA, alB;
                if constexpr (N == 2) { alA = pk(alpha[0], alpha[1]); alB = pk(alpha[2], alpha[3]); }
                else { alA = PR<1>{alpha[0]}; alB = PR<1>{alpha[1]}; }
                const PR<N> half = splat<N>(0.5f);
                const bool split2 = nb > 1;                // as for the spectra: one lane per pair when the batch is one class
                const int hcls = split2 ? (nb + 1) >> 1 : nb;
                #pragma unroll 1
                for (int item = tid; item < (split2 ? S : S / 2); item += kConsumers) {       // split: whole warps (S is a multiple of 32)
                    const int pr = split2 ? item >> 1 : item, ci0 = split2 ? (item & 1) * hcls : 0;
                    const int m = pr, mc = pr == 0 ? S / 2 : S - pr;
                    const int ci1 = (m >= s.k && mc >= s.k) ? ci0 : min(nb, ci0 + hcls);
                    float2 em = make_float2(1.f, 0.f), ec = make_float2(1.f, 0.f);
                    if (m < s.k) em = E[m];
                    if (mc < s.k) ec = E[mc];
                    float2 twm = seed_tw(m, cb + ci0), twc = seed_tw(mc, cb + ci0);
                    PC<N> zAm = czero, zBm = czero, zAc = czero, zBc = czero;
                    #pragma unroll 1
                    for (int ci = ci0; ci < ci1; ++ci) {
                        const float* base = fbuf + ci * fb_floats;
                        const PC<N> ya = ld_pt<N>(base + pf(m * GH)), yb = ld_pt<N>(base + pf(mc * GH));
                        const PR<N> wmr = splat<N>(twm.x), wmi = splat<N>(twm.y), wcr = splat<N>(twc.x), wci = splat<N>(twc.y);
                        if (pr != 0) {
                            // real slots: y0 = (ya + conj(yb)) / 2, imaginary slots: y1 = (ya - conj(yb)) / (2 i); bin mc holds the conjugates
                            const PC<N> y0 = PC<N>{(ya.re + yb.re) * half, (ya.im - yb.im) * half};
                            const PC<N> y1 = PC<N>{(ya.im + yb.im) * half, (yb.re - ya.re) * half};
                            zAm = zAm + cmulw(y0, wmr, wmi);
                            zBm = zBm + cmulw(y1, wmr, wmi);
                            zAc = zAc + cmulw(PC<N>{y0.re, splat<N>(0.f) - y0.im}, wcr, wci);
                            zBc = zBc + cmulw(PC<N>{y1.re, splat<N>(0.f) - y1.im}, wcr, wci);
                        } else {
                            // bins 0 and S/2 are real for each real sequence: (re, im) of the packed value are the two heads
                            const PC<N> y0m = PC<N>{ya.re, splat<N>(0.f)}, y1m = PC<N>{ya.im, splat<N>(0.f)};
                            const PC<N> y0c = PC<N>{yb.re, splat<N>(0.f)}, y1c = PC<N>{yb.im, splat<N>(0.f)};
                            zAm = zAm + cmulw(y0m, wmr, wmi);
                            zBm = zBm + cmulw(y1m, wmr, wmi);
                            zAc = zAc + cmulw(y0c, wcr, wci);
                            zBc = zBc + cmulw(y1c, wcr, wci);
                        }
                        twm = cmulf(twm, em);
                        twc = cmulf(twc, ec);
                    }
                    if (split2) {
                        zAm = pair_sum(zAm); zBm = pair_sum(zBm); zAc = pair_sum(zAc); zBc = pair_sum(zBc);
                        if (item & 1) continue;
                    }
                    if (m < s.k) {
                        PC<N> A, B;
                        ld_entry(z_s, m, A, B);
                        st_entry(z_s, m, PC<N>{pfma(A.re, alA, zAm.re), pfma(A.im, alA, zAm.im)},
                                 PC<N>{pfma(B.re, alB, zBm.re), pfma(B.im, alB, zBm.im)});
                    }
                    if (mc < s.k) {
                        PC<N> A, B;
                        ld_entry(z_s, mc, A, B);
                        st_entry(z_s, mc, PC<N>{pfma(A.re, alA, zAc.re), pfma(A.im, alA, zAc.im)},
                                 PC<N>{pfma(B.re, alB, zBc.re), pfma(B.im, alB, zBc.im)});
                    }
                }
            }
                    xf_sync();
                }
            }
            all_sync();
        }
        TL(13);
        // fold the per-warp output fragments into o_s at the natural positions of D^vu
        if (2 * tq < GH && is_m) {
            long long* o_lo = o_s + hperm<GH>(2 * tq) * s.d;
            long long* o_hi = o_s + hperm<GH>(2 * tq + 1) * s.d;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                if (o_idx[mt][0] >= 0) { fix_add(o_lo + o_idx[mt][0], acc[mt][0]); fix_add(o_hi + o_idx[mt][0], acc[mt][1]); }
                if (o_idx[mt][1] >= 0) { fix_add(o_lo + o_idx[mt][1], acc[mt][2]); fix_add(o_hi + o_idx[mt][1], acc[mt][3]); }
            }
        }
    }
    // sum of p per slot: the warps' sums in a fixed order
#pragma unroll
    for (int g = 0; g < GH; ++g) {
        float v = l_acc[g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) red_s[warp * GH + g] = v;
    }
    all_sync();
    if (tid < GH) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < kAllW; ++w) v += red_s[w * GH + tid];
        red_s[kAllW * GH + tid] = v;
    }
    all_sync();

    if (cp) {
        // class pairs: slot 1 (the odd classes of the batches) into slot 0, as two partial softmax results of one head
        const float mm = fmaxf(m_run[0], m_run[1]);
        const float e0 = ex2(m_run[0] - mm), e1 = ex2(m_run[1] - mm);
        #pragma unroll 1
        for (int e = tid; e < s.d; e += kAll)
            o_s[e] = __float2ll_rn(__ll2float_rn(o_s[e]) * e0 + __ll2float_rn(o_s[s.d + e]) * e1);
        #pragma unroll 1
        for (int n = tid; n < s.k; n += kAll) {
            float* e = z_s + n * 2 * GH;                  // (re, im) of slot 0, then of slot 1
            e[0] = e0 * e[0] + e1 * e[2];
            e[1] = e0 * e[1] + e1 * e[3];
        }
        all_sync();
        if (tid == 0) red_s[kAllW * GH] = e0 * red_s[kAllW * GH] + e1 * red_s[kAllW * GH + 1];
        m_run[0] = mm;
        all_sync();
    }

    TL(14);
    // ------------------------------ partial results ------------------------------
    for (int i = tid; i < GH * s.d; i += kAll) {
        const int g = i / s.d, e = i - g * s.d;
        if (g < ng) ws.o[(((size_t)b * s.Hq + g_first + g) * p.n_part + part) * s.d + e] = __ll2float_rn(o_s[i]) * kFixInv;
    }
    #pragma unroll 1
    for (int n = tid; n < s.k; n += kAll) {
        const float* e = z_s + n * 2 * GH;
#pragma unroll
        for (int sl = 0; sl < GH; ++sl) {
            const int g = hperm<GH>(sl), ab = sl / N, ln = sl - ab * N;
            if (g < ng)
                *reinterpret_cast<float2*>(ws.z + (((size_t)b * s.Hq + g_first + g) * p.n_part + part) * s.M + 2 * n) =
                    make_float2(e[(2 * ab) * N + ln], e[(2 * ab + 1) * N + ln]);
        }
    }
    if (tid < GH) {
        const int g = hperm<GH>(tid);                     // slot tid holds head g
        if (g < ng) {
            float* ml = ws.ml + (((size_t)b * s.Hq + g_first + g) * p.n_part + part) * 2;
            float mv = m_run[0];
#pragma unroll
            for (int sl = 1; sl < GH; ++sl) if (tid == sl) mv = m_run[sl];
            ml[0] = mv;
            ml[1] = red_s[kAllW * GH + tid];
        }
    }
    TL(15);
    if (!p.fused) return;

    // ------------------------------ merge (fused kernel) ------------------------------
    // All parts of this (b, KV head, pass) have written their partial results.  Each part then
    // merges a slice of the coefficient rows: its rows of every part's z against its rows of C^V.
    // The last part to finish adds the slices and the parts' o in a fixed order, normalises and
    // writes the output rows.  Everything a step needs from global memory is fetched with one batch
    // of 16-byte asynchronous copies into the stage ring (every tile has been consumed), so each
    // step costs one memory round trip.
    const int np = p.n_part;
    const int rows = m1 - m0;
    const size_t qh0 = (size_t)b * s.Hq + g_first;
    const int nv = s.dcv >> 2, nrg = nv ? kAll / nv : 0;
    // rows of the slice handled at a time: what the stage ring holds of C^V rows, z slices and weighted z
    constexpr int kRing = NS * kStageBytes / 4;
    const int head_f = (2 * GH * np + GH + 3) & ~3;
    const int mch = max(4, min((rows + 3) & ~3, ((kRing - head_f - nrg * GH * s.dcv) / (GH + s.dcv + GH * np)) & ~3));
    float* al_s = reinterpret_cast<float*>(stages);        // [GH][np] maxima, then exp2(m - max)
    float* l_s = al_s + GH * np;                           // [GH][np]
    float* linv_s = l_s + GH * np;                         // [GH]
    float* zw_s = al_s + head_f;                           // [GH][mch]
    float* big_s = zw_s + GH * mch;                        // step 1: C^V rows, z slices, partial sums; step 2: o and o^c parts
    float* cv_s = big_s;                                   // [mch][dcv]
    float* zs_s = cv_s + mch * s.dcv;                      // [GH][np][mch]
    float* ps_s = zs_s + GH * np * mch;                    // [row groups][GH][dcv]
    volatile int* last_s = fail + 1;
    float* cvg = s.dcv > 0 ? coef_rows(c.coef_v, s, b, h, s.dcv) + (size_t)m0 * s.dcv : nullptr;
    auto stage_cv = [&](int r0, int cr) {
#pragma unroll 1
        for (int i = tid; i < cr * nv; i += kAll) cp_async16(cv_s + 4 * i, cvg + (size_t)r0 * s.dcv + 4 * i);
    };

    if (s.dcv > 0) stage_cv(0, min(rows, mch));            // under the barrier
    part_arrive<kAll>(bar + 1, np, tid);
    TL(16);
    part_wait<kAll>(bar + 1, np, tid, fail, c.status);
    TL(17);
    // Fused step: every part of this (b, KV head) has read the row that leaves the window and is past its token
    // loop, so the rows the push moves can be written to the cache now, each by the part that owns it.
    if (step && !cap_full) {
        if (j_pend >= 0 && !is_win && cstar >= c0 && cstar < c1) {
            bf16* dk = mid_row<bf16>(c.k_mid, s, b, h, cstar, astar, s.nfk);
            bf16* dv = mid_row<bf16>(c.v_mid, s, b, h, cstar, astar, s.nfv);
#pragma unroll 1
            for (int e = tid; e < s.nfk; e += kAll) dk[e] = xrow_s[c.idx_full_k[(size_t)h * s.nfk + e]];
#pragma unroll 1
            for (int e = tid; e < s.nfv; e += kAll) dv[v_mid_col(astar, e, s.nfv, FA_BF16)] = xrow_s[s.d + c.idx_full_v[(size_t)h * s.nfv + e]];
        }
        if (new_buf >= 0 && new_tok >= w0 && new_tok < w1 && tid < 2 * (s.d >> 3)) {
            const int side = tid / (s.d >> 3), ch = tid - side * (s.d >> 3);
            bf16* dst = new_buf == 0 ? win_row<bf16>(side == 0 ? c.k_init : c.v_init, s, b, h, s.l_init, new_row)
                                     : win_row<bf16>(side == 0 ? c.k_local : c.v_local, s, b, h, s.l_local, new_row);
            *reinterpret_cast<uint4*>(dst + 8 * ch) = *reinterpret_cast<const uint4*>((side == 0 ? knew_bh : vnew_bh) + 8 * ch);
        }
    }
#pragma unroll 1
    for (int i = tid; i < GH * np; i += kAll) {
        float2 ml = make_float2(kNegBig, 0.f);
        if (i / np < ng) ml = __ldcg(reinterpret_cast<const float2*>(ws.ml + (qh0 * np + i) * 2));
        al_s[i] = ml.x;
        l_s[i] = ml.y;
    }
    float4 acc4[GH];
#pragma unroll
    for (int g = 0; g < GH; ++g) acc4[g] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
    for (int r0 = 0; r0 < rows || r0 == 0; r0 += mch) {
        const int cr = max(0, min(rows - r0, mch));
        if (s.dcv > 0) {
            if (r0 > 0) {
                all_sync();                           // the previous chunk has been consumed
                stage_cv(r0, cr);
            }
            const int r4 = cr >> 2;
#pragma unroll 1
            for (int i = tid; i < GH * np * r4; i += kAll) {
                const int gs = i / r4, j = i - gs * r4, g = gs / np;
                if (g < ng) cp_async16(zs_s + gs * mch + 4 * j, ws.z + (qh0 * np + gs) * s.M + m0 + r0 + 4 * j);
            }
        }
        cp_async_wait_all();
        all_sync();
        if (r0 == 0) {
            if (warp < GH) {                               // one warp per head, lanes over the parts
                float mx = kNegBig;
#pragma unroll 1
                for (int sp = lane; sp < np; sp += 32) mx = fmaxf(mx, al_s[warp * np + sp]);
                mx = warp_max(mx);
                float Lsum = 0.f;
#pragma unroll 1
                for (int sp = lane; sp < np; sp += 32) {
                    const float a = ex2(al_s[warp * np + sp] - mx);
                    al_s[warp * np + sp] = a;
                    Lsum = fmaf(a, l_s[warp * np + sp], Lsum);
                }
                Lsum = warp_sum(Lsum);
                if (lane == 0) linv_s[warp] = Lsum > 0.f ? __fdividef(1.0f, Lsum) : 0.f;
            }
        }
        all_sync();
        if (s.dcv > 0) {
#pragma unroll 1
            for (int t = tid; t < GH * cr; t += kAll) {
                const int g = t / cr, r = t - g * cr;
                float v = 0.f;
                if (g < ng) {
                    const float* z = zs_s + g * np * mch + r;
#pragma unroll 2
                    for (int sp = 0; sp < np; ++sp) v = fmaf(al_s[g * np + sp], z[sp * mch], v);
                    v *= recon_weight(s.norm, m0 + r0 + r, s.k, s.T);
                }
                zw_s[g * mch + r] = v;
            }
            all_sync();
            if (tid < nrg * nv) {
                const int v = tid % nv, rgi = tid / nv;
#pragma unroll 1
                for (int r = rgi; r < cr; r += nrg) {
                    float4 x = *reinterpret_cast<const float4*>(cv_s + r * s.dcv + 4 * v);
                    if (j_pend >= 0) {
                        // fused step: the pending rank-1 update of this piece of a C^V row (every piece passes here
                        // exactly once), used below and written back
                        const float f = f_row(r0 + r);
                        const float4 y = *reinterpret_cast<const float4*>(xp_s + s.dck + 4 * v);
                        x.x = fmaf(f, y.x, x.x); x.y = fmaf(f, y.y, x.y); x.z = fmaf(f, y.z, x.z); x.w = fmaf(f, y.w, x.w);
                        *reinterpret_cast<float4*>(cvg + (size_t)(r0 + r) * s.dcv + 4 * v) = x;
                    }
#pragma unroll
                    for (int g = 0; g < GH; ++g) {
                        const float w = zw_s[g * mch + r];
                        acc4[g].x = fmaf(w, x.x, acc4[g].x);
                        acc4[g].y = fmaf(w, x.y, acc4[g].y);
                        acc4[g].z = fmaf(w, x.z, acc4[g].z);
                        acc4[g].w = fmaf(w, x.w, acc4[g].w);
                    }
                }
            }
        }
    }
    if (s.dcv > 0) {
        if (tid < nrg * nv) {
            const int v = tid % nv, rgi = tid / nv;
#pragma unroll
            for (int g = 0; g < GH; ++g) *reinterpret_cast<float4*>(ps_s + (rgi * GH + g) * s.dcv + 4 * v) = acc4[g];
        }
        all_sync();
#pragma unroll 1
        for (int t = tid; t < GH * s.dcv; t += kAll) {
            const int g = t / s.dcv, e = t - g * s.dcv;
            float v = 0.f;
#pragma unroll 1
            for (int rgi = 0; rgi < nrg; ++rgi) v += ps_s[(rgi * GH + g) * s.dcv + e];
            if (g < ng) ws.oc[((qh0 + g) * np + part) * s.dcv + e] = v;
        }
    }
    TL(18);
    // ticket: the last part to get here finishes the rows
    all_sync();
    if (tid == 0) {
        int old = 0;
        if (np > 1) {
            __threadfence();
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(bar + 2) : "memory");
        }
        *last_s = old == np - 1;
    }
    all_sync();
    TL(19);
    if (!*last_s) { SPAN(2); return; }
    float* op_s = zw_s;                                    // [GH][np][d] (the slice buffers are free again)
    float* ocp_s = op_s + GH * np * s.d;                   // [GH][np][dcv]
    int* inv_s = reinterpret_cast<int*>(ocp_s + GH * np * s.dcv);   // [d] dim -> slot in D^vc, or -1
    {
        const int nd4 = s.d >> 2;
#pragma unroll 1
        for (int i = tid; i < ng * np * nd4; i += kAll) cp_async16(op_s + 4 * i, ws.o + qh0 * np * s.d + 4 * i);
#pragma unroll 1
        for (int i = tid; i < ng * np * nv; i += kAll) cp_async16(ocp_s + 4 * i, ws.oc + qh0 * np * s.dcv + 4 * i);
    }
#pragma unroll 1
    for (int e = tid; e < s.d; e += kAll) inv_s[e] = -1;
    all_sync();
    if (s.dcv > 0) {
        const int32_t* idc_v = c.idx_comp_v + (size_t)h * s.dcv;
#pragma unroll 1
        for (int e = tid; e < s.dcv; e += kAll) inv_s[idc_v[e]] = e;
    }
    cp_async_wait_all();
    all_sync();
#pragma unroll 1
    for (int t = tid; t < ng * s.d; t += kAll) {
        const int g = t / s.d, e = t - g * s.d;
        const float* o = op_s + g * np * s.d + e;
        float v = 0.f;
#pragma unroll 2
        for (int sp = 0; sp < np; ++sp) v = fmaf(al_s[g * np + sp], o[sp * s.d], v);
        const int slot = inv_s[e];
        if (slot >= 0) {
            const float* oc = ocp_s + g * np * s.dcv + slot;
            float w = 0.f;
#pragma unroll 2
            for (int x = 0; x < np; ++x) w += oc[x * s.dcv];
            v += w;
        }
        out[(qh0 + g) * s.d + e] = __float2bfloat16_rn(v * linv_s[g]);
    }
    TL(20);
    SPAN(3);
    if (tid == 0 && np > 1) { bar[0] = 0; bar[1] = 0; bar[2] = 0; }   // the counters are zero again for the next call
    // Fused step: the last (KV head, pass) of this batch row to finish publishes the counters after the push
    // (the others read the old ones when they started; the next kernel in the stream sees the new ones).
    if (step && !cap_full && tid == 0) {
        int32_t* st = c.state + kStateStride * b;
        const int old = atomicAdd(st + 4, 1);
        if (old == s.Hkv * p.n_pass - 1) {
            st[0] = n_init; st[1] = n_local; st[2] = n_mid_raw; st[3] = head;
            st[4] = 0;
        }
    }
}

// Whether the driver takes the cooperative and the programmatic-serialization launch attributes
// together, per device: -1 not probed, 0 no, 1 yes.  set = -2 reads, anything else records.
static int coop_pdl_state(int set) {
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

template <int GH, int LS, int OCC, bool STEP, bool SPLIT = false>
cudaError_t launch_fft_t(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* q, void* out, char* ws, int step,
                         const void* k_new, const void* v_new, cudaStream_t st) {
    const FftSmem L = fft_smem_layout(LS, s.k, GH, p.nb, s.d, OCC, SPLIT ? 1 : 0, class_pairs(s.G, GH, SPLIT ? 1 : 0));
    cudaError_t err = ensure_dynamic_smem(decode_fft_kernel<GH, LS, OCC, STEP, SPLIT>, (size_t)L.total);
    if (err != cudaSuccess) return err;
    // window buffers as tensor maps (cached per buffer)
    CUtensorMap tki, tvi, tkl, tvl;
    const int n_bh = s.B * s.Hkv;
    const bool ok_i = window_map(&tki, c.k_init, s.l_init, s.d, n_bh) & window_map(&tvi, c.v_init, s.l_init, s.d, n_bh);
    const bool ok_l = window_map(&tkl, c.k_local, s.l_local, s.d, n_bh) & window_map(&tvl, c.v_local, s.l_local, s.d, n_bh);
    if ((s.l_init > 0 && !ok_i) || (s.l_local > 0 && !ok_l)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_part, s.Hkv * p.n_pass, s.B);
    cfg.blockDim = dim3(threads_of(SPLIT));
    cfg.dynamicSmemBytes = (size_t)L.total;
    cfg.stream = st;
    // Programmatic dependent launch: the kernel may be scheduled while its predecessor in the stream
    // still runs and waits (griddepcontrol.wait) where it first reads what the predecessor wrote.  The
    // fused kernel is also a cooperative launch (its CTAs wait for one another); whether the driver
    // takes both attributes together is found out on the first launch outside a stream capture.
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
            cudaError_t err2 = cudaLaunchKernelEx(&cfg, decode_fft_kernel<GH, LS, OCC, STEP, SPLIT>, tki, tvi, tkl, tvl, s, c, p,
                                                  static_cast<const bf16*>(q), static_cast<bf16*>(out), ws,
                                                  static_cast<const bf16*>(k_new), static_cast<const bf16*>(v_new));
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
    return cudaLaunchKernelEx(&cfg, decode_fft_kernel<GH, LS, OCC, STEP, SPLIT>, tki, tvi, tkl, tvl, s, c, p, static_cast<const bf16*>(q),
                              static_cast<bf16*>(out), ws, static_cast<const bf16*>(k_new), static_cast<const bf16*>(v_new));
}

template <int GH>
cudaError_t launch_fft_ls(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* q, void* out, char* ws, int step,
                          const void* k_new, const void* v_new, cudaStream_t st) {
    switch (p.fft_log2) {
        case 5: return p.occ == 2 ? (step ? launch_fft_t<GH, 5, 2, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 5, 2, false>(s, c, p, q, out, ws, step, k_new, v_new, st)) : (step ? launch_fft_t<GH, 5, 1, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 5, 1, false>(s, c, p, q, out, ws, step, k_new, v_new, st));
        case 6: return p.occ == 2 ? (step ? launch_fft_t<GH, 6, 2, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 6, 2, false>(s, c, p, q, out, ws, step, k_new, v_new, st)) : (step ? launch_fft_t<GH, 6, 1, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 6, 1, false>(s, c, p, q, out, ws, step, k_new, v_new, st));
        case 7: return p.occ == 2 ? (step ? launch_fft_t<GH, 7, 2, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 7, 2, false>(s, c, p, q, out, ws, step, k_new, v_new, st)) : (step ? launch_fft_t<GH, 7, 1, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 7, 1, false>(s, c, p, q, out, ws, step, k_new, v_new, st));
        case 8: return p.occ == 2 ? (step ? launch_fft_t<GH, 8, 2, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 8, 2, false>(s, c, p, q, out, ws, step, k_new, v_new, st)) : (step ? launch_fft_t<GH, 8, 1, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 8, 1, false>(s, c, p, q, out, ws, step, k_new, v_new, st));
        case 9:
            return (step ? launch_fft_t<GH, 9, 1, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 9, 1, false>(s, c, p, q, out, ws, step, k_new, v_new, st));
        case 10:
            if (p.split) return (step ? launch_fft_t<GH, 10, 1, true, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 10, 1, false, true>(s, c, p, q, out, ws, step, k_new, v_new, st));
            return (step ? launch_fft_t<GH, 10, 1, true>(s, c, p, q, out, ws, step, k_new, v_new, st) : launch_fft_t<GH, 10, 1, false>(s, c, p, q, out, ws, step, k_new, v_new, st));
        default: return cudaErrorInvalidValue;
    }
}

// Resident CTAs of this kernel instance on the whole device for the plan's shared memory (cached per instance).
template <int GH, int LS, int OCC, bool SPLIT = false, bool STEP = true>
int resident_ctas_t(const Dims& s, const DecodePlan& p) {
    // answers cached per (device, shared memory size) of this instance
    struct Entry { int dev; size_t smem; int ctas; };
    static Entry table[16];
    static int used = 0;
    static std::mutex mu;
    const size_t smem = (size_t)fft_smem_layout(LS, s.k, GH, p.nb, s.d, OCC, SPLIT ? 1 : 0, class_pairs(s.G, GH, SPLIT ? 1 : 0)).total;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i)
        if (table[i].dev == dev && table[i].smem == smem) return table[i].ctas;
    if (ensure_dynamic_smem(decode_fft_kernel<GH, LS, OCC, STEP, SPLIT>, smem) != cudaSuccess) { cudaGetLastError(); return 0; }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_fft_kernel<GH, LS, OCC, STEP, SPLIT>, threads_of(SPLIT), smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    const int ctas = per_sm * sm_count();
    if (used < 16) table[used++] = Entry{dev, smem, ctas};
    return ctas;
}
template <int GH>
int resident_ctas_ls(const Dims& s, const DecodePlan& p) {
    switch (p.fft_log2) {
        case 5: return p.occ == 2 ? resident_ctas_t<GH, 5, 2>(s, p) : resident_ctas_t<GH, 5, 1>(s, p);
        case 6: return p.occ == 2 ? resident_ctas_t<GH, 6, 2>(s, p) : resident_ctas_t<GH, 6, 1>(s, p);
        case 7: return p.occ == 2 ? resident_ctas_t<GH, 7, 2>(s, p) : resident_ctas_t<GH, 7, 1>(s, p);
        case 8: return p.occ == 2 ? resident_ctas_t<GH, 8, 2>(s, p) : resident_ctas_t<GH, 8, 1>(s, p);
        case 9: return resident_ctas_t<GH, 9, 1>(s, p);
        case 10: return p.split ? resident_ctas_t<GH, 10, 1, true, false>(s, p) : resident_ctas_t<GH, 10, 1>(s, p);
        default: return 0;
    }
}

}  // namespace

// True if the fused kernel of this plan can be launched as planned: a part that waits for nobody runs in
// waves; parts that wait for one another must all be resident at once (what a cooperative launch checks),
// which depends on the registers and shared memory of the compiled instance, so the runtime is asked.
bool decode_fft_launchable(const Dims& s, const DecodePlan& p) {
    if (!p.fused) return true;
    if (p.n_part <= 1) return true;
    const long long grid = (long long)p.n_part * s.Hkv * p.n_pass * s.B;
    const int resident = p.gh == 4 ? resident_ctas_ls<4>(s, p) : resident_ctas_ls<2>(s, p);
    return grid <= resident;
}

size_t decode_fft_smem_bytes(const Dims& s, int log2S, int gh, int nb, int occ, int split) {
    return (size_t)fft_smem_layout(log2S, s.k, gh, nb, s.d, occ, split, class_pairs(s.G, gh, split)).total;
}

// True if the fused kernel's staging areas hold a part's share of the coefficient rows: the rows
// of C^K in the transform buffers at the start, the merge scratch in the stage ring at the end.
bool decode_fft_fused_fits(const Dims& s, int log2S, int gh, int nb, int n_part, int occ, int split) {
    if (s.M % 4 != 0) return false;
    if (occ == 2 && log2S > 8) return false;                                           // no two-per-SM build of the long transforms
    const FftSmem L = fft_smem_layout(log2S, s.k, gh, nb, s.d, occ, split, class_pairs(s.G, gh, split));
    // at least eight rows of C^K per staged chunk (class pairs: the chunk may use the score and probability buffers too, as the kernel does)
    if (s.dck > 0 && (class_pairs(s.G, gh, split) ? (long long)((L.twf_off - L.fbuf_off) >> 2) : (long long)nb * L.fb_floats) < 8LL * s.dck) return false;
    const long long ring = (long long)ring_stages(occ, split) * kStageBytes / 4;
    const long long nrg = s.dcv ? (split ? kSplitConsumers : kConsumers) / (s.dcv >> 2) : 0;
    const long long head = ((2LL * gh * n_part + gh + 3) & ~3LL);
    if (s.dcv > 0 && (ring - head - nrg * gh * s.dcv) / (gh + s.dcv + (long long)gh * n_part) < 8) return false;   // and of C^V
    const long long step2 = (long long)gh * n_part * (s.d + s.dcv) + s.d;               // the last part's merge of all parts
    return head + 8LL * gh + step2 <= ring;
}

cudaError_t launch_decode_fft(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, const void* q, void* out,
                              char* ws, const void* k_new, const void* v_new, cudaStream_t st) {
    if (dtype != FA_BF16) return cudaErrorInvalidValue;
    const int step = k_new != nullptr && v_new != nullptr ? 1 : 0;      // a fused step: the push of (k_new, v_new) rides on this launch
    if (p.gh == 4) return launch_fft_ls<4>(s, c, p, q, out, ws, step, k_new, v_new, st);
    return launch_fft_ls<2>(s, c, p, q, out, ws, step, k_new, v_new, st);
}

}  // namespace fa
