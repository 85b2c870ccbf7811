// fa_decode_attention, main kernel for bf16 caches: residue-class (FFT) evaluation of the
// compressed dims and tensor-core dot products for the kept dims (Eq.6 re-associated).
//
// With theta = 2 pi / T, u~_n = u[2n] - i u[2n+1] and the middle tokens of class c,
// j = c + P a (a = 0..S-1, S = T / P >= k):
//   scores   sum_m F[m][j] u[m]  = Re sum_n (u~_n e^{i theta n c}) e^{2 pi i n a / S}
//   outputs  z_n = sum_j p_j e^{i theta n j} = sum_c e^{i theta n c} sum_a p_{c+Pa} e^{2 pi i n a / S}
// so a class costs one length-S transform per side instead of S * k basis terms.  Two query
// heads share one complex transform (real-pair packing); with GH = 4 heads a point is a float4.
// The score transform runs decimation-in-frequency (natural in, digit-reversed out), the
// probability transform decimation-in-time (digit-reversed in, natural out), both in place:
// softmax is pointwise, so nothing is ever reordered.  NB classes are transformed together.
//
// K^mu / V^mu are class-major, so the tokens of a class are one contiguous stream; a producer
// warp brings it in with bulk (TMA) copies through a ring of shared-memory stages.  The eight
// consumer warps feed the tiles to mma.sync (bf16 x bf16 -> fp32; exact for q . K, p rounded to
// bf16 for p . V): K fragments are read with 128-bit loads using the freedom to permute the
// contraction index, V^T fragments with transposing 8x8 matrix loads, conflict-free because
// V^mu rows are stored chunk-swizzled.  Window rows (init + local ring) are copied row by row
// into padded shared-memory rows and take the same route.  Every wait is bounded.
#include "fa_common.cuh"
#include "fa_decode_ws.cuh"

namespace fa {
namespace {

constexpr int kConsumers = 256;
constexpr int kThreads = kConsumers + 32;
constexpr int kStageBytes = 16384;
constexpr int kStages = 3;
constexpr int kWinRowsPerTile = 48;
constexpr uint32_t kSpinLimit = 1u << 24;
using bf16 = __nv_bfloat16;

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
// Bounded wait: gives up after kSpinLimit polls, records the failure, never hangs.
__device__ __forceinline__ void mbar_wait(uint64_t* b, uint32_t parity, volatile int* fail, int32_t* status) {
    if (*fail) return;
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(b, parity)) return;
    *fail = 1;
    atomicExch(status, (int)FA_ERR_TIMEOUT);
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

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
__device__ __forceinline__ uint32_t pack_bf16(bf16 lo, bf16 hi) {
    return (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
}

// ---- complex helpers --------------------------------------------------------
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 mul_i(float2 a) { return make_float2(-a.y, a.x); }
__device__ __forceinline__ float2 conj(float2 a) { return make_float2(a.x, -a.y); }

// In-place DFTs with exponent +2 pi i / R, natural order in and out.
__device__ __forceinline__ void dft4(float2& a0, float2& a1, float2& a2, float2& a3) {
    float2 t0 = cadd(a0, a2), t1 = csub(a0, a2), t2 = cadd(a1, a3), t3 = mul_i(csub(a1, a3));
    a0 = cadd(t0, t2);
    a1 = cadd(t1, t3);
    a2 = csub(t0, t2);
    a3 = csub(t1, t3);
}
template <int R>
__device__ __forceinline__ void dft(float2 (&v)[R]) {
    if constexpr (R == 2) {
        float2 t = v[0];
        v[0] = cadd(t, v[1]);
        v[1] = csub(t, v[1]);
    } else if constexpr (R == 4) {
        dft4(v[0], v[1], v[2], v[3]);
    } else {
        constexpr float h = 0.70710678118654752440f;
        dft4(v[0], v[2], v[4], v[6]);     // even part -> E0..E3
        dft4(v[1], v[3], v[5], v[7]);     // odd part  -> O0..O3
        float2 o1 = make_float2(h * (v[3].x - v[3].y), h * (v[3].x + v[3].y));        // w   O1
        float2 o2 = mul_i(v[5]);                                                        // w^2 O2
        float2 o3 = make_float2(-h * (v[7].x + v[7].y), h * (v[7].x - v[7].y));       // w^3 O3
        float2 e0 = v[0], e1 = v[2], e2 = v[4], e3 = v[6], o0 = v[1];
        v[0] = cadd(e0, o0); v[4] = csub(e0, o0);
        v[1] = cadd(e1, o1); v[5] = csub(e1, o1);
        v[2] = cadd(e2, o2); v[6] = csub(e2, o2);
        v[3] = cadd(e3, o3); v[7] = csub(e3, o3);
    }
}

// Shared-memory float index of float f of a transform buffer: 16 bytes of padding after every
// 128, which spreads strided point accesses over the banks and keeps points 16-byte aligned.
__host__ __device__ inline int pf(int f) { return f + ((f >> 5) << 2); }
__host__ __device__ inline int pf_size(int floats) { return floats + ((floats >> 5) << 2) + 4; }

// Radix plan of the length-2^log2S transform; identical on host and device.
struct FftPlan {
    int n;            // stages
    int radix[4];
    int len[4];       // sub-transform length entering stage s (DIF order)
    int twoff[4];     // offset (in float2) of the stage's twiddles [q-1][j], -1 if none (len == radix)
    int twtotal;
};
__host__ __device__ inline FftPlan make_fft_plan(int log2S) {
    FftPlan p;
    p.n = 0;
    p.twtotal = 0;
    int rem = log2S, L = 1 << log2S;
    while (rem > 0) {
        int r = (rem >= 3 && rem != 4) ? 8 : (rem >= 2 ? 4 : 2);
        p.radix[p.n] = r;
        p.len[p.n] = L;
        if (L > r) { p.twoff[p.n] = p.twtotal; p.twtotal += (r - 1) * (L / r); } else p.twoff[p.n] = -1;
        L /= r;
        rem -= (r == 8 ? 3 : (r == 4 ? 2 : 1));
        ++p.n;
    }
    return p;
}

// One in-place pass over nb transforms held in consecutive buffers.  DIF: butterfly, then
// twiddle the outputs; DIT: twiddle the inputs, then butterfly.  A point holds GH / 2 complex
// numbers (independent transforms sharing the twiddles).
template <int R, int GH, bool DIT>
__device__ __forceinline__ void fft_pass(float* fbuf, int fb_floats, int nb, int S, int L, const float2* tw, int tid) {
    constexpr int NC = GH / 2;
    const int st = L / R, per = S / R;
    for (int item = tid; item < nb * per; item += kConsumers) {
        const int ci = item / per, rest = item - ci * per;
        const int blk = rest / st, j = rest - blk * st;
        float* base = fbuf + ci * fb_floats;
        const int e0 = blk * L + j;
        float2 v[NC][R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float* p = base + pf((e0 + r * st) * GH);
            if constexpr (GH == 4) {
                const float4 x = *reinterpret_cast<const float4*>(p);
                v[0][r] = make_float2(x.x, x.y);
                v[1][r] = make_float2(x.z, x.w);
            } else {
                v[0][r] = *reinterpret_cast<const float2*>(p);
            }
        }
        float2 w[R];
        if (tw) {
#pragma unroll
            for (int q = 1; q < R; ++q) w[q] = tw[(q - 1) * st + j];
        }
        if (DIT && tw) {
#pragma unroll
            for (int c = 0; c < NC; ++c)
#pragma unroll
                for (int q = 1; q < R; ++q) v[c][q] = cmul(v[c][q], w[q]);
        }
#pragma unroll
        for (int c = 0; c < NC; ++c) dft<R>(v[c]);
        if (!DIT && tw) {
#pragma unroll
            for (int c = 0; c < NC; ++c)
#pragma unroll
                for (int q = 1; q < R; ++q) v[c][q] = cmul(v[c][q], w[q]);
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float* p = base + pf((e0 + r * st) * GH);
            if constexpr (GH == 4) *reinterpret_cast<float4*>(p) = make_float4(v[0][r].x, v[0][r].y, v[1][r].x, v[1][r].y);
            else *reinterpret_cast<float2*>(p) = v[0][r];
        }
    }
}

template <int GH, bool DIT>
__device__ __forceinline__ void fft_run(float* fbuf, int fb_floats, int nb, int S, const FftPlan& pl, const float2* twf, int tid) {
    for (int i = 0; i < pl.n; ++i) {
        const int sidx = DIT ? pl.n - 1 - i : i;
        const int R = pl.radix[sidx], L = pl.len[sidx];
        const float2* tw = pl.twoff[sidx] >= 0 ? twf + pl.twoff[sidx] : nullptr;
        if (R == 8) fft_pass<8, GH, DIT>(fbuf, fb_floats, nb, S, L, tw, tid);
        else if (R == 4) fft_pass<4, GH, DIT>(fbuf, fb_floats, nb, S, L, tw, tid);
        else fft_pass<2, GH, DIT>(fbuf, fb_floats, nb, S, L, tw, tid);
        consumer_sync();
    }
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
    int stages_off, fbuf_off, pbt_off, twf_off, rev_off, E_off, ut_off, z_off, o_off, red_off, zero_off, total;
    int fb_floats, pbs;
};
__host__ __device__ inline FftSmem fft_smem_layout(int S, int log2S, int k, int GH, int NB, int d) {
    FftSmem L;
    L.fb_floats = pf_size(S * GH);
    L.pbs = S + 8;                                        // bf16 per (class, head) row of rounded probabilities
    int off = 256;                                        // mbarriers + flags
    L.zero_off = off; off += 16;
    off = (off + 127) / 128 * 128;
    L.stages_off = off; off += kStages * kStageBytes;
    L.fbuf_off = off; off += 4 * NB * L.fb_floats;
    off = (off + 15) / 16 * 16;
    L.pbt_off = off; off += 2 * NB * GH * L.pbs;
    off = (off + 15) / 16 * 16;
    L.twf_off = off; off += 8 * (make_fft_plan(log2S).twtotal + 1);
    L.rev_off = off; off += 2 * S;
    off = (off + 15) / 16 * 16;
    L.E_off = off; off += 8 * k;
    L.ut_off = off; off += 8 * k * GH;
    L.z_off = off; off += 8 * k * GH;
    L.o_off = off; off += 4 * GH * d;
    L.red_off = off; off += 4 * (8 * GH + GH + 8);
    L.total = (off + 127) / 128 * 128;
    return L;
}

// GH query heads per CTA (2 or 4).
template <int GH>
__global__ void __launch_bounds__(kThreads, 1) decode_fft_kernel(Dims s, CacheDev c, DecodePlan p, const bf16* __restrict__ q,
                                                                  char* wsp) {
    constexpr int NC = GH / 2;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Ws ws = ws_view(wsp, p);
    const int S = s.T / s.P, log2S = p.fft_log2, NB = p.nb;
    const FftSmem L = fft_smem_layout(S, log2S, s.k, GH, NB, s.d);
    const FftPlan pl = make_fft_plan(log2S);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw);
    uint64_t* empty = full + kStages;
    volatile int* fail = reinterpret_cast<volatile int*>(smem_raw + 128);
    unsigned char* zero16 = smem_raw + L.zero_off;
    unsigned char* stages = smem_raw + L.stages_off;
    float* fbuf = reinterpret_cast<float*>(smem_raw + L.fbuf_off);        // [NB][fb_floats] points of GH floats
    bf16* pbt = reinterpret_cast<bf16*>(smem_raw + L.pbt_off);           // [NB][GH][pbs]
    float2* twf = reinterpret_cast<float2*>(smem_raw + L.twf_off);        // stage twiddles
    uint16_t* rev = reinterpret_cast<uint16_t*>(smem_raw + L.rev_off);    // slot -> position after the DIF
    float2* E = reinterpret_cast<float2*>(smem_raw + L.E_off);            // e^{i theta n}
    float2* ut = reinterpret_cast<float2*>(smem_raw + L.ut_off);          // [k][GH] (1/2) u~
    float2* z_s = reinterpret_cast<float2*>(smem_raw + L.z_off);          // [k][GH]
    float* o_s = reinterpret_cast<float*>(smem_raw + L.o_off);            // [GH][d]
    float* red_s = reinterpret_cast<float*>(smem_raw + L.red_off);        // [8][GH] + l_s[GH]
    const int fb_floats = L.fb_floats, pbs = L.pbs;

    const int split = blockIdx.x;
    const int h = blockIdx.y / p.n_pass, pass = blockIdx.y % p.n_pass;
    const int b = blockIdx.z;
    const int g_first = h * s.G + pass * GH;
    const int ng = min(GH, s.G - pass * GH);
    const int tid = threadIdx.x;

    const int n_init = c.state[kStateStride * b + 0], n_local = c.state[kStateStride * b + 1];
    const int n_mid = min(c.state[kStateStride * b + 2], s.max_mid), head = c.state[kStateStride * b + 3];
    const int c0 = (int)((long long)split * s.P / p.n_split), c1 = (int)((long long)(split + 1) * s.P / p.n_split);
    const int n_win = n_init + n_local;
    const int w0 = (int)((long long)split * n_win / p.n_split), w1 = (int)((long long)(split + 1) * n_win / p.n_split);

    const int rowb_k = s.nfk * 2, rowb_v = s.nfv * 2, rowb_w = s.d * 2;
    const int rbw_pad = rowb_w + 16;                                       // padded window row in shared memory
    const int ts_k = rowb_k ? (kStageBytes / rowb_k) & ~15 : 0, ts_v = rowb_v ? (kStageBytes / rowb_v) & ~15 : 0;
    const int ts_w = kWinRowsPerTile;
    const int wchunk = S;

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 8); }
        *fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // stale shared memory must hold finite numbers: rows past the end of a tile are multiplied by p = 0
    for (int i = tid; i < (kStages * kStageBytes) / 16; i += kThreads) reinterpret_cast<uint4*>(stages)[i] = make_uint4(0, 0, 0, 0);
    if (tid < 4) reinterpret_cast<uint32_t*>(zero16)[tid] = 0;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();

    // ============================ producer warp =================================
    if (tid >= kConsumers) {
        if (tid == kConsumers) {
            int it = 0;
            auto acquire = [&](uint32_t bytes) -> unsigned char* {
                const int st = it % kStages;
                if (it >= kStages) mbar_wait(empty + st, ((it / kStages) - 1) & 1, fail, c.status);
                if (*fail) return nullptr;
                mbar_expect_tx(full + st, bytes);
                return stages + (size_t)st * kStageBytes;
            };
            // same order as the consumers: per batch of NB classes all K tiles, then all V tiles
            for (int cb = c0; cb < c1; cb += NB) {
                const int nb = min(NB, c1 - cb);
                for (int side = 0; side < 2; ++side) {
                    const int ts = side == 0 ? ts_k : ts_v, rowb = side == 0 ? rowb_k : rowb_v;
                    if (!ts) continue;
                    for (int cls = cb; cls < cb + nb; ++cls) {
                        const int n_c = cls < n_mid ? (n_mid - cls + s.P - 1) / s.P : 0;
                        for (int a0 = 0; a0 < n_c; a0 += ts) {
                            const uint32_t bytes = (uint32_t)(min(ts, n_c - a0) * rowb);
                            const bf16* src = side == 0 ? mid_row<bf16>(c.k_mid, s, b, h, cls, a0, s.nfk)
                                                        : mid_row<bf16>(c.v_mid, s, b, h, cls, a0, s.nfv);
                            if (unsigned char* dst = acquire(bytes)) bulk_g2s(dst, src, bytes, full + it % kStages);
                            ++it;
                        }
                    }
                }
            }
            for (int t0 = w0; t0 < w1; t0 += wchunk) {
                const WinSegs sg = win_segments(t0, min(w1, t0 + wchunk), n_init, n_local, head, s.l_local);
                for (int side = 0; side < 2; ++side)
                    for (int i = 0; i < sg.n; ++i)
                        for (int r0 = 0; r0 < sg.cnt[i]; r0 += ts_w) {
                            const int nt = min(ts_w, sg.cnt[i] - r0);
                            void* base = sg.buf[i] == 0 ? (side == 0 ? c.k_init : c.v_init) : (side == 0 ? c.k_local : c.v_local);
                            const int rows = sg.buf[i] == 0 ? s.l_init : s.l_local;
                            const bf16* src = win_row<bf16>(base, s, b, h, rows, sg.row[i] + r0);
                            if (unsigned char* dst = acquire((uint32_t)(nt * rowb_w)))
                                for (int r = 0; r < nt; ++r)
                                    bulk_g2s(dst + (size_t)r * rbw_pad, src + (size_t)r * s.d, (uint32_t)rowb_w, full + it % kStages);
                            ++it;
                        }
            }
        }
        return;
    }

    // ============================ consumer warps =================================
    const int warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;              // mma fragment coordinates
    const int npk = s.nfk >> 3, nchv = s.nfv >> 3, npw = s.d >> 3;
    const float sl2 = s.scale * kLog2e;

    // ---- one-time set-up ----
    for (int i = tid; i < GH * s.d; i += kConsumers) o_s[i] = 0.f;
    for (int i = tid; i < s.k; i += kConsumers) {
        float sn, cs;
        sincospif(2.0f * (float)i / (float)s.T, &sn, &cs);
        E[i] = make_float2(cs, sn);
    }
    for (int i = tid; i < s.k * GH; i += kConsumers) {
        const int n = i / GH, g = i - n * GH;
        float2 v = make_float2(0.f, 0.f);
        if (g < ng && s.dck > 0) {
            const float* u = ws.u + ((size_t)b * s.Hq + g_first + g) * s.M;
            v = make_float2(0.5f * u[2 * n], -0.5f * u[2 * n + 1]);
        }
        ut[i] = v;
        z_s[i] = make_float2(0.f, 0.f);
    }
    for (int sidx = 0; sidx < pl.n; ++sidx) {
        if (pl.twoff[sidx] < 0) continue;
        const int R = pl.radix[sidx], Ls = pl.len[sidx], st = Ls / R;
        for (int i = tid; i < (R - 1) * st; i += kConsumers) {
            const int qm1 = i / st, j = i - qm1 * st;
            float sn, cs;
            sincospif(2.0f * (float)(((qm1 + 1) * j) & (Ls - 1)) / (float)Ls, &sn, &cs);
            twf[pl.twoff[sidx] + i] = make_float2(cs, sn);
        }
    }
    for (int a = tid; a < S; a += kConsumers) {
        int kk = a, pos = 0, Lc = S;
        for (int sidx = 0; sidx < pl.n; ++sidx) {
            const int R = pl.radix[sidx];
            Lc /= R;
            pos += (kk % R) * Lc;
            kk /= R;
        }
        rev[a] = (uint16_t)pos;
    }
    if (tid < GH + 8) red_s[8 * GH + tid] = 0.f;

    // B fragments of q for the kept K dims: round rd covers pieces 4 rd + tq of a row, two k-steps each
    uint32_t qk[2][2][2];
    {
        const int32_t* idf_k = c.idx_full_k + (size_t)h * s.nfk;
        const bf16* qrow = q + ((size_t)b * s.Hq + g_first + gq) * s.d;
#pragma unroll
        for (int rd = 0; rd < 2; ++rd)
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const int piece = 4 * rd + tq, e0 = 8 * piece + 4 * ks;
                const bool on = gq < ng && piece < npk;
                qk[rd][ks][0] = on ? pack_bf16(qrow[idf_k[e0]], qrow[idf_k[e0 + 1]]) : 0u;
                qk[rd][ks][1] = on ? pack_bf16(qrow[idf_k[e0 + 2]], qrow[idf_k[e0 + 3]]) : 0u;
            }
    }
    consumer_sync();

    float m_run[GH], l_acc[GH];
#pragma unroll
    for (int g = 0; g < GH; ++g) { m_run[g] = kNegBig; l_acc[g] = 0.f; }
    int it = 0;                                           // tile counter, mirrors the producer's

    auto wait_tile = [&]() -> const unsigned char* {
        const int st = it % kStages;
        mbar_wait(full + st, (it / kStages) & 1, fail, c.status);
        return stages + (size_t)st * kStageBytes;
    };
    auto release_tile = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + (it % kStages));
        ++it;
    };
    // per-head maximum over per-thread partial maxima, broadcast to every consumer thread
    auto block_max = [&](float (&mx)[GH]) {
#pragma unroll
        for (int g = 0; g < GH; ++g) {
            float v = mx[g];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
            if (lane == 0) red_s[warp * GH + g] = v;
        }
        consumer_sync();
#pragma unroll
        for (int g = 0; g < GH; ++g) {
            float r = red_s[g];
#pragma unroll
            for (int w = 1; w < 8; ++w) r = fmaxf(r, red_s[w * GH + g]);
            mx[g] = r;
        }
    };
    auto load_point = [&](const float* pt, float (&v)[GH]) {
        if constexpr (GH == 4) {
            const float4 x = *reinterpret_cast<const float4*>(pt);
            v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
        } else {
            const float2 x = *reinterpret_cast<const float2*>(pt);
            v[0] = x.x; v[1] = x.y;
        }
    };
    auto store_point = [&](float* pt, const float (&v)[GH]) {
        if constexpr (GH == 4) *reinterpret_cast<float4*>(pt) = make_float4(v[0], v[1], v[2], v[3]);
        else *reinterpret_cast<float2*>(pt) = make_float2(v[0], v[1]);
    };

    // ------------------------------ middle classes ------------------------------
    {
        float acc[4][4];                                  // [m-tile of 16 dims][mma D fragment]
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
        const int nmt = (s.nfv + 15) >> 4;

        for (int cb = c0; cb < c1; cb += NB) {
            const int nb = min(NB, c1 - cb);
            auto n_of = [&](int ci) { const int cls = cb + ci; return cls < n_mid ? (n_mid - cls + s.P - 1) / s.P : 0; };
            if (n_of(0) == 0) break;                      // classes are filled in order: nothing further on

            // packed Hermitian spectra of the nb classes: X_m = V^{g0}_m + i V^{g1}_m (and g2, g3)
            if (s.dck > 0) {
                for (int m = tid; m <= S / 2; m += kConsumers) {
                    const int mc = (S - m) & (S - 1);
                    float2 um[GH], uc[GH];
#pragma unroll
                    for (int g = 0; g < GH; ++g) {
                        um[g] = m < s.k ? ut[m * GH + g] : make_float2(0.f, 0.f);
                        uc[g] = mc < s.k ? ut[mc * GH + g] : make_float2(0.f, 0.f);
                    }
                    float2 twm, twc, em = make_float2(1.f, 0.f), ec = make_float2(1.f, 0.f);
                    {
                        float sn, cs;
                        sincospif(2.0f * (float)((m * cb) & (s.T - 1)) / (float)s.T, &sn, &cs);
                        twm = make_float2(cs, sn);
                        sincospif(2.0f * (float)((mc * cb) & (s.T - 1)) / (float)s.T, &sn, &cs);
                        twc = make_float2(cs, sn);
                        if (m < s.k) em = E[m];
                        if (mc < s.k) ec = E[mc];
                    }
                    for (int ci = 0; ci < nb; ++ci) {
                        float2 vm[GH];
#pragma unroll
                        for (int g = 0; g < GH; ++g) vm[g] = cadd(cmul(um[g], twm), conj(cmul(uc[g], twc)));
                        float xm[GH], xc[GH];
#pragma unroll
                        for (int cl = 0; cl < NC; ++cl) {
                            xm[2 * cl] = vm[2 * cl].x - vm[2 * cl + 1].y;
                            xm[2 * cl + 1] = vm[2 * cl].y + vm[2 * cl + 1].x;
                            xc[2 * cl] = vm[2 * cl].x + vm[2 * cl + 1].y;
                            xc[2 * cl + 1] = vm[2 * cl + 1].x - vm[2 * cl].y;
                        }
                        float* base = fbuf + ci * fb_floats;
                        store_point(base + pf(m * GH), xm);
                        if (mc != m) store_point(base + pf(mc * GH), xc);
                        twm = cmul(twm, em);
                        twc = cmul(twc, ec);
                    }
                }
                consumer_sync();
                fft_run<GH, false>(fbuf, fb_floats, nb, S, pl, twf, tid);     // scores of slot a at point rev[a]
            } else {
                for (int i = tid; i < nb * fb_floats; i += kConsumers) fbuf[i] = 0.f;
                consumer_sync();
            }

            // kept dims: s = sl2 * (q_u . K^mu) + compressed part, 16 tokens per mma
            if (ts_k) {
                for (int ci = 0; ci < nb; ++ci) {
                    const int n_c = n_of(ci);
                    float* base = fbuf + ci * fb_floats;
                    for (int a0 = 0; a0 < n_c; a0 += ts_k) {
                        const int nt = min(ts_k, n_c - a0);
                        const unsigned char* tile = wait_tile();
                        for (int grp = warp; grp * 16 < nt; grp += 8) {
                            const unsigned char* r_lo = tile + (size_t)(grp * 16 + gq) * rowb_k;
                            const unsigned char* r_hi = r_lo + 8 * rowb_k;
                            float d4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                            for (int rd = 0; rd < 2; ++rd) {
                                const int piece = 4 * rd + tq;
                                if (4 * rd < npk) {
                                    uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
                                    if (piece < npk) {
                                        lo = *reinterpret_cast<const uint4*>(r_lo + 16 * piece);
                                        hi = *reinterpret_cast<const uint4*>(r_hi + 16 * piece);
                                    }
                                    mma_bf16(d4, lo.x, hi.x, lo.y, hi.y, qk[rd][0][0], qk[rd][0][1]);
                                    mma_bf16(d4, lo.z, hi.z, lo.w, hi.w, qk[rd][1][0], qk[rd][1][1]);
                                }
                            }
                            if (2 * tq < GH) {
                                const int a_lo = a0 + grp * 16 + gq, a_hi = a_lo + 8;
                                if (a_lo < n_c) {
                                    float2* dst = reinterpret_cast<float2*>(base + pf(rev[a_lo] * GH + 2 * tq));
                                    float2 v = *dst;
                                    *dst = make_float2(fmaf(d4[0], sl2, v.x), fmaf(d4[1], sl2, v.y));
                                }
                                if (a_hi < n_c) {
                                    float2* dst = reinterpret_cast<float2*>(base + pf(rev[a_hi] * GH + 2 * tq));
                                    float2 v = *dst;
                                    *dst = make_float2(fmaf(d4[2], sl2, v.x), fmaf(d4[3], sl2, v.y));
                                }
                            }
                        }
                        release_tile();
                    }
                }
            }
            consumer_sync();

            // online softmax over the batch
            float mx[GH], alpha[GH];
#pragma unroll
            for (int g = 0; g < GH; ++g) mx[g] = kNegBig;
            for (int i = tid; i < nb * S; i += kConsumers) {
                const int ci = i / S, a = i - ci * S;
                if (a < n_of(ci)) {
                    float v[GH];
                    load_point(fbuf + ci * fb_floats + pf(rev[a] * GH), v);
#pragma unroll
                    for (int g = 0; g < GH; ++g) mx[g] = fmaxf(mx[g], v[g]);
                }
            }
            block_max(mx);
#pragma unroll
            for (int g = 0; g < GH; ++g) {
                const float m_new = fmaxf(m_run[g], mx[g]);
                alpha[g] = exp2f(m_run[g] - m_new);
                m_run[g] = m_new;
                l_acc[g] *= alpha[g];
            }
            for (int i = tid; i < nb * S; i += kConsumers) {
                const int ci = i / S, a = i - ci * S;
                float* pt = fbuf + ci * fb_floats + pf(rev[a] * GH);
                float v[GH];
                load_point(pt, v);
                const bool ok = a < n_of(ci);
#pragma unroll
                for (int g = 0; g < GH; ++g) {
                    v[g] = ok ? exp2f(v[g] - m_run[g]) : 0.f;
                    l_acc[g] += v[g];
                    pbt[(ci * GH + g) * pbs + a] = __float2bfloat16_rn(v[g]);
                }
                store_point(pt, v);
            }
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                acc[mt][0] *= alpha[(2 * tq) & (GH - 1)];
                acc[mt][1] *= alpha[(2 * tq + 1) & (GH - 1)];
                acc[mt][2] *= alpha[(2 * tq) & (GH - 1)];
                acc[mt][3] *= alpha[(2 * tq + 1) & (GH - 1)];
            }
            consumer_sync();

            // o^u[dim][head] += V^mu^T p, 16 tokens per mma
            if (ts_v) {
                for (int ci = 0; ci < nb; ++ci) {
                    const int n_c = n_of(ci);
                    const bf16* prow = pbt + (size_t)(ci * GH + gq) * pbs;
                    for (int a0 = 0; a0 < n_c; a0 += ts_v) {
                        const int nt = min(ts_v, n_c - a0);
                        const unsigned char* tile = wait_tile();
                        for (int grp = warp; grp * 16 < nt; grp += 8) {
                            const int a = a0 + grp * 16;
                            uint32_t b0 = 0, b1 = 0;
                            if (gq < GH) {
                                b0 = *reinterpret_cast<const uint32_t*>(prow + a + 2 * tq);
                                b1 = *reinterpret_cast<const uint32_t*>(prow + a + 2 * tq + 8);
                            }
                            const int mi = lane >> 3, tok = ((mi >> 1) << 3) + (lane & 7);
                            const unsigned char* vrow = tile + (size_t)(grp * 16 + tok) * rowb_v;
                            const int sw = v_swz(a + tok, nchv);
#pragma unroll
                            for (int mt = 0; mt < 4; ++mt) {
                                if (mt < nmt) {
                                    const int chunk = 2 * mt + (mi & 1);
                                    const unsigned char* src = chunk < nchv ? vrow + 16 * (chunk ^ sw) : zero16;
                                    uint32_t af[4];
                                    ldmatrix_x4_trans(af, smem_addr(src));
                                    mma_bf16(acc[mt], af[0], af[1], af[2], af[3], b0, b1);
                                }
                            }
                        }
                        release_tile();
                    }
                }
            }

            // z_n = alpha z_n + sum_c e^{i theta n c} Y^c_n, Y^c = transform of the packed probabilities
            if (s.dcv > 0) {
                fft_run<GH, true>(fbuf, fb_floats, nb, S, pl, twf, tid);
                for (int m = tid; m <= S / 2; m += kConsumers) {
                    const int mc = (S - m) & (S - 1);
                    if (m >= s.k && mc >= s.k) continue;
                    float2 twm, twc, em = make_float2(1.f, 0.f), ec = make_float2(1.f, 0.f);
                    {
                        float sn, cs;
                        sincospif(2.0f * (float)((m * cb) & (s.T - 1)) / (float)s.T, &sn, &cs);
                        twm = make_float2(cs, sn);
                        sincospif(2.0f * (float)((mc * cb) & (s.T - 1)) / (float)s.T, &sn, &cs);
                        twc = make_float2(cs, sn);
                        if (m < s.k) em = E[m];
                        if (mc < s.k) ec = E[mc];
                    }
                    float2 zm[GH], zc[GH];
#pragma unroll
                    for (int g = 0; g < GH; ++g) { zm[g] = make_float2(0.f, 0.f); zc[g] = make_float2(0.f, 0.f); }
                    for (int ci = 0; ci < nb; ++ci) {
                        const float* base = fbuf + ci * fb_floats;
                        float ya[GH], yb[GH];
                        load_point(base + pf(m * GH), ya);
                        load_point(base + pf(mc * GH), yb);
#pragma unroll
                        for (int cl = 0; cl < NC; ++cl) {
                            // heads 2cl, 2cl+1 of bin m; bin mc holds the conjugates
                            const float2 y0 = make_float2(0.5f * (ya[2 * cl] + yb[2 * cl]), 0.5f * (ya[2 * cl + 1] - yb[2 * cl + 1]));
                            const float2 y1 = make_float2(0.5f * (ya[2 * cl + 1] + yb[2 * cl + 1]), -0.5f * (ya[2 * cl] - yb[2 * cl]));
                            zm[2 * cl] = cadd(zm[2 * cl], cmul(twm, y0));
                            zm[2 * cl + 1] = cadd(zm[2 * cl + 1], cmul(twm, y1));
                            zc[2 * cl] = cadd(zc[2 * cl], cmul(twc, conj(y0)));
                            zc[2 * cl + 1] = cadd(zc[2 * cl + 1], cmul(twc, conj(y1)));
                        }
                        twm = cmul(twm, em);
                        twc = cmul(twc, ec);
                    }
#pragma unroll
                    for (int g = 0; g < GH; ++g) {
                        if (m < s.k) {
                            const float2 z0 = z_s[m * GH + g];
                            z_s[m * GH + g] = make_float2(fmaf(z0.x, alpha[g], zm[g].x), fmaf(z0.y, alpha[g], zm[g].y));
                        }
                        if (mc < s.k && mc != m) {
                            const float2 z0 = z_s[mc * GH + g];
                            z_s[mc * GH + g] = make_float2(fmaf(z0.x, alpha[g], zc[g].x), fmaf(z0.y, alpha[g], zc[g].y));
                        }
                    }
                }
            }
            consumer_sync();
        }
        // fold the per-warp output fragments into o_s at the natural positions of D^vu
        const int32_t* idf_v = c.idx_full_v + (size_t)h * s.nfv;
        if (2 * tq < GH) {
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const int e_lo = 16 * mt + gq, e_hi = e_lo + 8;
                if (e_lo < s.nfv) {
                    atomicAdd(o_s + (2 * tq) * s.d + idf_v[e_lo], acc[mt][0]);
                    atomicAdd(o_s + (2 * tq + 1) * s.d + idf_v[e_lo], acc[mt][1]);
                }
                if (e_hi < s.nfv) {
                    atomicAdd(o_s + (2 * tq) * s.d + idf_v[e_hi], acc[mt][2]);
                    atomicAdd(o_s + (2 * tq + 1) * s.d + idf_v[e_hi], acc[mt][3]);
                }
            }
        }
    }
    consumer_sync();

    // ------------------------------ window tokens -------------------------------
    if (w1 > w0) {
        float a_win[GH];                                  // rescale of what the classes left in o_s / z_s
#pragma unroll
        for (int g = 0; g < GH; ++g) a_win[g] = 1.f;
        uint32_t qw[4][2][2];
        {
            const bf16* qrow = q + ((size_t)b * s.Hq + g_first + gq) * s.d;
#pragma unroll
            for (int rd = 0; rd < 4; ++rd)
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
                    const int piece = 4 * rd + tq, e0 = 8 * piece + 4 * ks;
                    const bool on = gq < ng && piece < npw;
                    qw[rd][ks][0] = on ? pack_bf16(qrow[e0], qrow[e0 + 1]) : 0u;
                    qw[rd][ks][1] = on ? pack_bf16(qrow[e0 + 2], qrow[e0 + 3]) : 0u;
                }
        }
        float accw[8][4];
#pragma unroll
        for (int mt = 0; mt < 8; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) accw[mt][i] = 0.f;
        const int nmtw = (s.d + 15) >> 4;
        float* sb = fbuf;                                 // natural order, no transform
        bf16* pb = pbt;
        for (int t0 = w0; t0 < w1; t0 += wchunk) {
            const int n_tok = min(w1, t0 + wchunk) - t0;
            const WinSegs sg = win_segments(t0, t0 + n_tok, n_init, n_local, head, s.l_local);
            for (int si = 0; si < sg.n; ++si)
                for (int r0 = 0; r0 < sg.cnt[si]; r0 += ts_w) {
                    const int nt = min(ts_w, sg.cnt[si] - r0);
                    const unsigned char* tile = wait_tile();
                    for (int grp = warp; grp * 16 < nt; grp += 8) {
                        const unsigned char* r_lo = tile + (size_t)(grp * 16 + gq) * rbw_pad;
                        const unsigned char* r_hi = r_lo + 8 * rbw_pad;
                        float d4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int rd = 0; rd < 4; ++rd) {
                            const int piece = 4 * rd + tq;
                            if (4 * rd < npw) {
                                uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
                                if (piece < npw) {
                                    lo = *reinterpret_cast<const uint4*>(r_lo + 16 * piece);
                                    hi = *reinterpret_cast<const uint4*>(r_hi + 16 * piece);
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
            consumer_sync();
            float mx[GH], alpha[GH];
#pragma unroll
            for (int g = 0; g < GH; ++g) mx[g] = kNegBig;
            for (int a = tid; a < n_tok; a += kConsumers) {
                float v[GH];
                load_point(sb + pf(a * GH), v);
#pragma unroll
                for (int g = 0; g < GH; ++g) mx[g] = fmaxf(mx[g], v[g]);
            }
            block_max(mx);
#pragma unroll
            for (int g = 0; g < GH; ++g) {
                const float m_new = fmaxf(m_run[g], mx[g]);
                alpha[g] = exp2f(m_run[g] - m_new);
                m_run[g] = m_new;
                l_acc[g] *= alpha[g];
                a_win[g] *= alpha[g];
            }
            const int n_pad = (n_tok + 15) & ~15;
            for (int a = tid; a < n_pad; a += kConsumers) {
                float v[GH];
                if (a < n_tok) load_point(sb + pf(a * GH), v);
#pragma unroll
                for (int g = 0; g < GH; ++g) {
                    v[g] = a < n_tok ? exp2f(v[g] - m_run[g]) : 0.f;
                    l_acc[g] += v[g];
                    pb[g * pbs + a] = __float2bfloat16_rn(v[g]);
                }
            }
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                accw[mt][0] *= alpha[(2 * tq) & (GH - 1)];
                accw[mt][1] *= alpha[(2 * tq + 1) & (GH - 1)];
                accw[mt][2] *= alpha[(2 * tq) & (GH - 1)];
                accw[mt][3] *= alpha[(2 * tq + 1) & (GH - 1)];
            }
            consumer_sync();
            const bf16* prow = pb + (size_t)gq * pbs;
            for (int si = 0; si < sg.n; ++si)
                for (int r0 = 0; r0 < sg.cnt[si]; r0 += ts_w) {
                    const int nt = min(ts_w, sg.cnt[si] - r0);
                    const unsigned char* tile = wait_tile();
                    for (int grp = warp; grp * 16 < nt; grp += 8) {
                        const int a = sg.tok[si] + r0 + grp * 16;
                        // the tile's rows may start at any token of the chunk: gather the four p values one by one
                        uint32_t b0 = 0, b1 = 0;
                        if (gq < GH) {
                            const int rem = nt - grp * 16;
                            const bf16 zero = __float2bfloat16_rn(0.f);
                            b0 = pack_bf16(2 * tq < rem ? prow[a + 2 * tq] : zero, 2 * tq + 1 < rem ? prow[a + 2 * tq + 1] : zero);
                            b1 = pack_bf16(2 * tq + 8 < rem ? prow[a + 2 * tq + 8] : zero, 2 * tq + 9 < rem ? prow[a + 2 * tq + 9] : zero);
                        }
                        const int mi = lane >> 3, tok = ((mi >> 1) << 3) + (lane & 7);
                        const unsigned char* vrow = tile + (size_t)(grp * 16 + tok) * rbw_pad;
#pragma unroll
                        for (int mt = 0; mt < 8; ++mt) {
                            if (mt < nmtw) {
                                const int chunk = 2 * mt + (mi & 1);
                                const unsigned char* src = chunk < npw ? vrow + 16 * chunk : zero16;
                                uint32_t af[4];
                                ldmatrix_x4_trans(af, smem_addr(src));
                                mma_bf16(accw[mt], af[0], af[1], af[2], af[3], b0, b1);
                            }
                        }
                    }
                    release_tile();
                }
            consumer_sync();
        }
        // rescale what the classes left, then add the window fragments
        for (int i = tid; i < GH * s.d; i += kConsumers) {
            float a = a_win[0];
#pragma unroll
            for (int g = 1; g < GH; ++g) if (i / s.d == g) a = a_win[g];
            o_s[i] *= a;
        }
        for (int i = tid; i < s.k * GH; i += kConsumers) {
            float a = a_win[0];
#pragma unroll
            for (int g = 1; g < GH; ++g) if (i % GH == g) a = a_win[g];
            z_s[i] = make_float2(z_s[i].x * a, z_s[i].y * a);
        }
        consumer_sync();
        if (2 * tq < GH) {
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                const int e_lo = 16 * mt + gq, e_hi = e_lo + 8;
                if (e_lo < s.d) {
                    atomicAdd(o_s + (2 * tq) * s.d + e_lo, accw[mt][0]);
                    atomicAdd(o_s + (2 * tq + 1) * s.d + e_lo, accw[mt][1]);
                }
                if (e_hi < s.d) {
                    atomicAdd(o_s + (2 * tq) * s.d + e_hi, accw[mt][2]);
                    atomicAdd(o_s + (2 * tq + 1) * s.d + e_hi, accw[mt][3]);
                }
            }
        }
    }
    // sum of p per head
#pragma unroll
    for (int g = 0; g < GH; ++g) {
        float v = l_acc[g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) atomicAdd(red_s + 8 * GH + g, v);
    }
    consumer_sync();

    // ------------------------------ partial results ------------------------------
    for (int i = tid; i < GH * s.d; i += kConsumers) {
        const int g = i / s.d, e = i - g * s.d;
        if (g < ng) ws.o[(((size_t)b * s.Hq + g_first + g) * p.n_split + split) * s.d + e] = o_s[i];
    }
    for (int i = tid; i < s.k * GH; i += kConsumers) {
        const int n = i / GH, g = i - n * GH;
        if (g < ng) {
            float2* dst = reinterpret_cast<float2*>(ws.z + (((size_t)b * s.Hq + g_first + g) * p.n_split + split) * s.M) + n;
            *dst = z_s[i];
        }
    }
    if (tid < ng) {
        float* ml = ws.ml + (((size_t)b * s.Hq + g_first + tid) * p.n_split + split) * 2;
        float mv = m_run[0];
#pragma unroll
        for (int g = 1; g < GH; ++g) if (tid == g) mv = m_run[g];
        ml[0] = mv;
        ml[1] = red_s[8 * GH + tid];
    }
}

template <int GH>
cudaError_t launch_fft_t(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* q, char* ws, cudaStream_t st) {
    const FftSmem L = fft_smem_layout(s.T / s.P, p.fft_log2, s.k, GH, p.nb, s.d);
    cudaError_t err = ensure_dynamic_smem(decode_fft_kernel<GH>, (size_t)L.total);
    if (err != cudaSuccess) return err;
    decode_fft_kernel<GH><<<dim3(p.n_split, s.Hkv * p.n_pass, s.B), kThreads, L.total, st>>>(
        s, c, p, static_cast<const bf16*>(q), ws);
    return cudaGetLastError();
}

}  // namespace

size_t decode_fft_smem_bytes(const Dims& s, int log2S, int gh, int nb) {
    return (size_t)fft_smem_layout(s.T / s.P, log2S, s.k, gh, nb, s.d).total;
}

cudaError_t launch_decode_fft(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, const void* q, char* ws,
                              cudaStream_t st) {
    if (dtype != FA_BF16) return cudaErrorInvalidValue;
    if (p.gh == 4) return launch_fft_t<4>(s, c, p, q, ws, st);
    return launch_fft_t<2>(s, c, p, q, ws, st);
}

}  // namespace fa
