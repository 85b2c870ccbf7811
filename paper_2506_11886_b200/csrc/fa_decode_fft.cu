// fa_decode_attention, main kernel, residue-class (FFT) evaluation of the
// compressed dims (Eq.6 re-associated).
//
// With theta = 2 pi / T, u~_n = u[2n] - i u[2n+1] and the middle tokens of class
// c, j = c + P a (a = 0..S-1, S = T / P):
//   scores   sum_m F[m][j] u[m]  = Re sum_n (u~_n e^{i theta n c}) e^{2 pi i n a / S}
//   outputs  z_n = sum_j p_j e^{i theta n j} = sum_c e^{i theta n c} sum_a p_{c+Pa} e^{2 pi i n a / S}
// so each class costs one length-S transform per side instead of S * k terms.
// Two query heads share one complex transform (real pair packing); with GH = 4
// heads every point is a float4 = two complex numbers.  K^mu / V^mu are stored
// class-major, so the tokens of a class are one contiguous stream that a
// producer warp brings in with bulk (TMA) copies through a ring of shared
// memory stages, while eight consumer warps do dot products, softmax and the
// transforms.  Window tokens (init + local ring) go through the same ring as
// ordinary 128-dim attention.  Every wait is bounded.
#include "fa_common.cuh"
#include "fa_decode_ws.cuh"

namespace fa {
namespace {

constexpr int kConsumers = 256;
constexpr int kThreads = kConsumers + 32;
constexpr int kStageBytes = 16384;
constexpr int kStages = 4;
constexpr uint32_t kSpinLimit = 1u << 24;

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

// ---- complex helpers --------------------------------------------------------
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 mul_i(float2 a) { return make_float2(-a.y, a.x); }
__device__ __forceinline__ float2 conj(float2 a) { return make_float2(a.x, -a.y); }

// In-place DFTs with exponent +2 pi i / R, natural order in and out.
__device__ __forceinline__ void dft2(float2& a, float2& b) {
    float2 t = a;
    a = cadd(t, b);
    b = csub(t, b);
}
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
        dft2(v[0], v[1]);
    } else if constexpr (R == 4) {
        dft4(v[0], v[1], v[2], v[3]);
    } else {
        constexpr float h = 0.70710678118654752440f;
        dft4(v[0], v[2], v[4], v[6]);     // even part -> v0, v2, v4, v6 hold E0..E3
        dft4(v[1], v[3], v[5], v[7]);     // odd part  -> v1, v3, v5, v7 hold O0..O3
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

// Shared-memory index of float f of a transform buffer: 16 bytes of padding after every 128,
// which spreads the strided accesses of the first stages over the banks and keeps float4 aligned.
__device__ __forceinline__ int phys(int f) { return f + ((f >> 5) << 2); }
__host__ __device__ constexpr int phys_size(int floats) { return floats + ((floats >> 5) << 2) + 4; }

// One Stockham stage of radix R over NC interleaved complex lanes per point (exponent +).
template <int R, int NC>
__device__ __forceinline__ void fft_stage(const float* in, float* out, const float2* W, int S, int Ns, int tid) {
    const int nb = S / R;
    const int wstride = S / (Ns * R);
    for (int item = tid; item < nb * NC; item += kConsumers) {
        const int j = item / NC, cl = item % NC;
        const int kk = j & (Ns - 1);
        float2 v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = *reinterpret_cast<const float2*>(in + phys(2 * ((j + r * nb) * NC + cl)));
        if (Ns > 1) {
            float2 w[R];
            w[1] = W[kk * wstride];
            if constexpr (R >= 4) { w[2] = cmul(w[1], w[1]); w[3] = cmul(w[2], w[1]); }
            if constexpr (R >= 8) { w[4] = cmul(w[2], w[2]); w[5] = cmul(w[3], w[2]); w[6] = cmul(w[3], w[3]); w[7] = cmul(w[4], w[3]); }
#pragma unroll
            for (int r = 1; r < R; ++r) v[r] = cmul(v[r], w[r]);
        }
        dft<R>(v);
        const int jb = (j - kk) * R + kk;
#pragma unroll
        for (int r = 0; r < R; ++r) *reinterpret_cast<float2*>(out + phys(2 * ((jb + r * Ns) * NC + cl))) = v[r];
    }
}

// Full transform a -> (a or b); the caller has synchronised the consumers on the input.
template <int NC>
__device__ __forceinline__ float* fft_run(float* a, float* b, const float2* W, int S, int log2S, int tid) {
    int Ns = 1, rem = log2S;
    float *in = a, *out = b;
    while (rem > 0) {
        if (rem >= 3 && rem != 4) { fft_stage<8, NC>(in, out, W, S, Ns, tid); Ns *= 8; rem -= 3; }
        else if (rem >= 2) { fft_stage<4, NC>(in, out, W, S, Ns, tid); Ns *= 4; rem -= 2; }
        else { fft_stage<2, NC>(in, out, W, S, Ns, tid); Ns *= 2; rem -= 1; }
        consumer_sync();
        float* t = in; in = out; out = t;
    }
    return in;
}

// 8 consecutive elements (one "piece") of a staged row as floats.
__device__ __forceinline__ void ld_piece(const __nv_bfloat16* row, int piece, float (&x)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(row + 8 * piece);
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
    x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
    x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
}
__device__ __forceinline__ void ld_piece(const float* row, int piece, float (&x)[8]) {
    float4 a = *reinterpret_cast<const float4*>(row + 8 * piece);
    float4 b = *reinterpret_cast<const float4*>(row + 8 * piece + 4);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}

// Sum GH per-lane partials over a group of 4 lanes so that lane r of the group ends with the
// total of head head_of(r).  GH = 4: 3 shuffles; GH = 2: 2 shuffles.
template <int GH>
__device__ __forceinline__ int head_of(int r) {
    if constexpr (GH == 4) return ((r & 1) << 1) | ((r >> 1) & 1);
    return r & 1;
}
template <int GH>
__device__ __forceinline__ float quad_reduce(float (&part)[GH], int r) {
    if constexpr (GH == 4) {
        const bool odd = r & 1;
        float keep0 = odd ? part[2] : part[0], keep1 = odd ? part[3] : part[1];
        float send0 = odd ? part[0] : part[2], send1 = odd ? part[1] : part[3];
        keep0 += __shfl_xor_sync(0xffffffffu, send0, 1);
        keep1 += __shfl_xor_sync(0xffffffffu, send1, 1);
        const bool hi = r & 2;
        float keep = hi ? keep1 : keep0, send = hi ? keep0 : keep1;
        return keep + __shfl_xor_sync(0xffffffffu, send, 2);
    } else {
        const bool odd = r & 1;
        float keep = odd ? part[1] : part[0], send = odd ? part[0] : part[1];
        keep += __shfl_xor_sync(0xffffffffu, send, 1);
        return keep + __shfl_xor_sync(0xffffffffu, keep, 2);
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
    int stages_off, fa_off, fb_off, W_off, ut_off, tw_off, z_off, q_off, qk_off, o_off, red_off, total;
};
__host__ __device__ inline FftSmem fft_smem_layout(int S, int k, int GH, int d, int nfk) {
    FftSmem L;
    int off = 256;                                        // mbarriers + flags
    L.stages_off = off; off += kStages * kStageBytes;
    L.fa_off = off; off += 4 * phys_size(S * GH);
    L.fb_off = off; off += 4 * phys_size(S * GH);
    L.W_off = off; off += 8 * S;
    L.ut_off = off; off += 8 * k * GH;
    L.tw_off = off; off += 8 * k;
    L.z_off = off; off += 8 * k * GH;
    L.q_off = off; off += 4 * GH * d;
    L.qk_off = off; off += 4 * GH * (nfk > 0 ? nfk : 8);
    L.o_off = off; off += 4 * GH * d;
    L.red_off = off; off += 4 * (8 * GH + 2 * GH + 8);
    L.total = (off + 127) / 128 * 128;
    return L;
}

// GH query heads per CTA (2 or 4), SL = ceil(max(nfk, nfv) / 32) pieces of 8 dims per lane (1 or 2).
template <typename KV, int GH, int SL>
__global__ void __launch_bounds__(kThreads, 1) decode_fft_kernel(Dims s, CacheDev c, DecodePlan p, const KV* __restrict__ q,
                                                                  char* wsp) {
    constexpr int NC = GH / 2;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Ws ws = ws_view(wsp, p);
    const int S = s.T / s.P, log2S = p.fft_log2;
    const FftSmem L = fft_smem_layout(S, s.k, GH, s.d, s.nfk);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw);
    uint64_t* empty = full + kStages;
    volatile int* fail = reinterpret_cast<volatile int*>(smem_raw + 128);
    unsigned char* stages = smem_raw + L.stages_off;
    float* fA = reinterpret_cast<float*>(smem_raw + L.fa_off);
    float* fB = reinterpret_cast<float*>(smem_raw + L.fb_off);
    float2* W = reinterpret_cast<float2*>(smem_raw + L.W_off);
    float2* ut = reinterpret_cast<float2*>(smem_raw + L.ut_off);      // [k][GH] (1/2) u~
    float2* tw = reinterpret_cast<float2*>(smem_raw + L.tw_off);      // [k]
    float2* z_s = reinterpret_cast<float2*>(smem_raw + L.z_off);      // [k][GH]
    float* q_s = reinterpret_cast<float*>(smem_raw + L.q_off);        // [GH][d]
    float* qk_s = reinterpret_cast<float*>(smem_raw + L.qk_off);      // [nfk/8][GH][8]
    float* o_s = reinterpret_cast<float*>(smem_raw + L.o_off);        // [GH][d]
    float* red_s = reinterpret_cast<float*>(smem_raw + L.red_off);    // [8][GH] + l_s[GH] + spare

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

    const int eb = (int)sizeof(KV);
    const int rowb_k = s.nfk * eb, rowb_v = s.nfv * eb, rowb_w = s.d * eb;
    const int ts_k = rowb_k ? kStageBytes / rowb_k : 0, ts_v = rowb_v ? kStageBytes / rowb_v : 0;
    const int ts_w = kStageBytes / rowb_w;
    const int wchunk = S;                                  // window tokens scored per pass through the buffer

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 8); }
        *fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // ============================ producer warp =================================
    if (tid >= kConsumers) {
        if (tid == kConsumers) {
            int it = 0;
            auto produce = [&](const void* src, int bytes) {
                const int st = it % kStages;
                if (it >= kStages) mbar_wait(empty + st, ((it / kStages) - 1) & 1, fail, c.status);
                if (!*fail) {
                    mbar_expect_tx(full + st, (uint32_t)bytes);
                    bulk_g2s(stages + (size_t)st * kStageBytes, src, (uint32_t)bytes, full + st);
                }
                ++it;
            };
            for (int cls = c0; cls < c1; ++cls) {
                const int n_c = cls < n_mid ? (n_mid - cls + s.P - 1) / s.P : 0;
                if (ts_k)
                    for (int a0 = 0; a0 < n_c; a0 += ts_k)
                        produce(mid_row<KV>(c.k_mid, s, b, h, cls, a0, s.nfk), min(ts_k, n_c - a0) * rowb_k);
                if (ts_v)
                    for (int a0 = 0; a0 < n_c; a0 += ts_v)
                        produce(mid_row<KV>(c.v_mid, s, b, h, cls, a0, s.nfv), min(ts_v, n_c - a0) * rowb_v);
            }
            for (int t0 = w0; t0 < w1; t0 += wchunk) {
                const WinSegs sg = win_segments(t0, min(w1, t0 + wchunk), n_init, n_local, head, s.l_local);
                for (int side = 0; side < 2; ++side)
                    for (int i = 0; i < sg.n; ++i)
                        for (int r0 = 0; r0 < sg.cnt[i]; r0 += ts_w) {
                            void* base = sg.buf[i] == 0 ? (side == 0 ? c.k_init : c.v_init) : (side == 0 ? c.k_local : c.v_local);
                            int rows = sg.buf[i] == 0 ? s.l_init : s.l_local;
                            produce(win_row<KV>(base, s, b, h, rows, sg.row[i] + r0), min(ts_w, sg.cnt[i] - r0) * rowb_w);
                        }
            }
        }
        return;
    }

    // ============================ consumer warps =================================
    const int warp = tid >> 5, lane = tid & 31;
    const int r4 = tid & 3, tq4 = tid >> 2;               // middle tiles: 4 lanes per token, 64 tokens per pass
    const int r16 = tid & 15, tq16 = tid >> 4;            // window tiles: 16 lanes per token, 16 tokens per pass
    const int my_head = tid % GH;                         // head of the elements this thread owns in the score buffer
    const int npk = s.nfk >> 3, npv = s.nfv >> 3, npw = s.d >> 3;
    const int fold = (s.k + S - 1) / S;

    // ---- one-time set-up: q, gathered q, transform roots, u~, zeroed accumulators ----
    for (int i = tid; i < GH * s.d; i += kConsumers) {
        int g = i / s.d, e = i - g * s.d;
        q_s[i] = g < ng ? ld_f(q + ((size_t)b * s.Hq + g_first + g) * s.d + e) * s.scale * kLog2e : 0.f;
        o_s[i] = 0.f;
    }
    for (int i = tid; i < S; i += kConsumers) {
        float sn, cs;
        sincospif(2.0f * (float)i / (float)S, &sn, &cs);
        W[i] = make_float2(cs, sn);
    }
    for (int i = tid; i < s.k * GH; i += kConsumers) {
        int n = i / GH, g = i - n * GH;
        float2 v = make_float2(0.f, 0.f);
        if (g < ng && s.dck > 0) {
            const float* u = ws.u + ((size_t)b * s.Hq + g_first + g) * s.M;
            v = make_float2(0.5f * u[2 * n], -0.5f * u[2 * n + 1]);
        }
        ut[i] = v;
        z_s[i] = make_float2(0.f, 0.f);
    }
    if (tid < 2 * GH + 8) red_s[8 * GH + tid] = 0.f;
    consumer_sync();
    {
        const int32_t* idf_k = c.idx_full_k + (size_t)h * s.nfk;
        for (int i = tid; i < GH * s.nfk; i += kConsumers) {
            int piece = i / (GH * 8), rem = i - piece * GH * 8;
            int g = rem >> 3, e = rem & 7;
            qk_s[i] = q_s[g * s.d + idf_k[piece * 8 + e]];
        }
    }
    consumer_sync();

    float m_run[GH], l_part = 0.f;
#pragma unroll
    for (int g = 0; g < GH; ++g) m_run[g] = kNegBig;
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
    // max over the first n_tok tokens of the score buffer, per head, broadcast to all threads
    auto block_max = [&](const float* sb, int n_tok, float (&mx)[GH]) {
        float v = kNegBig;
        for (int i = tid; i < n_tok * GH; i += kConsumers) v = fmaxf(v, sb[phys(i)]);
#pragma unroll
        for (int o = 16; o >= GH; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
        if (lane < GH) red_s[warp * GH + lane] = v;
        consumer_sync();
#pragma unroll
        for (int g = 0; g < GH; ++g) {
            float r = red_s[g];
#pragma unroll
            for (int w = 1; w < 8; ++w) r = fmaxf(r, red_s[w * GH + g]);
            mx[g] = r;
        }
    };
    // scores -> probabilities in place (zero beyond n_tok), running sum
    auto to_prob = [&](float* sb, int n_tok, int n_buf, float m_mine) {
        for (int i = tid; i < n_buf * GH; i += kConsumers) {
            float pv = i < n_tok * GH ? exp2f(sb[phys(i)] - m_mine) : 0.f;
            sb[phys(i)] = pv;
            l_part += pv;
        }
    };

    // ------------------------------ middle classes ------------------------------
    {
        float qk[SL][GH][8], acc[SL][GH][8];
#pragma unroll
        for (int sl = 0; sl < SL; ++sl) {
            const int piece = r4 + 4 * sl;
#pragma unroll
            for (int g = 0; g < GH; ++g)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    qk[sl][g][e] = piece < npk ? qk_s[(piece * GH + g) * 8 + e] : 0.f;
                    acc[sl][g][e] = 0.f;
                }
        }
        for (int cls = c0; cls < c1; ++cls) {
            const int n_c = cls < n_mid ? (n_mid - cls + s.P - 1) / s.P : 0;
            if (n_c == 0) continue;
            // twiddles e^{i theta n cls}
            for (int n = tid; n < s.k; n += kConsumers) {
                float cs, sn;
                basis_cs(n, cls, s.T, &cs, &sn);
                tw[n] = make_float2(cs, sn);
            }
            consumer_sync();
            // packed, Hermitian-symmetrised spectrum of the class: X_m = V^{g0}_m + i V^{g1}_m (and g2, g3)
            float* sb = fA;
            if (s.dck > 0) {
                for (int m = tid; m < S; m += kConsumers) {
                    const int mc = (S - m) & (S - 1);
                    float2 va[GH], vb[GH];
#pragma unroll
                    for (int g = 0; g < GH; ++g) { va[g] = make_float2(0.f, 0.f); vb[g] = make_float2(0.f, 0.f); }
                    for (int f = 0; f < fold; ++f) {
                        const int na = m + f * S, nb = mc + f * S;
                        if (na < s.k) {
                            const float2 t = tw[na];
#pragma unroll
                            for (int g = 0; g < GH; ++g) va[g] = cadd(va[g], cmul(ut[na * GH + g], t));
                        }
                        if (nb < s.k) {
                            const float2 t = tw[nb];
#pragma unroll
                            for (int g = 0; g < GH; ++g) vb[g] = cadd(vb[g], cmul(ut[nb * GH + g], t));
                        }
                    }
#pragma unroll
                    for (int cl = 0; cl < NC; ++cl) {
                        const float2 v0 = cadd(va[2 * cl], conj(vb[2 * cl])), v1 = cadd(va[2 * cl + 1], conj(vb[2 * cl + 1]));
                        *reinterpret_cast<float2*>(fA + phys(2 * (m * NC + cl))) = make_float2(v0.x - v1.y, v0.y + v1.x);
                    }
                }
                consumer_sync();
                sb = fft_run<NC>(fA, fB, W, S, log2S, tid);           // sb[a][g] = compressed-dim score of slot a
            } else {
                for (int i = tid; i < S * GH; i += kConsumers) fA[phys(i)] = 0.f;
                consumer_sync();
            }
            float* other = sb == fA ? fB : fA;
            // kept dims: s += q_u . K^mu
            if (ts_k) {
                for (int a0 = 0; a0 < n_c; a0 += ts_k) {
                    const int nt = min(ts_k, n_c - a0);
                    const KV* tile = reinterpret_cast<const KV*>(wait_tile());
                    for (int i0 = 0; i0 < nt; i0 += 64) {
                        const int i = i0 + tq4;
                        const bool ok = i < nt;
                        const KV* row = tile + (size_t)(ok ? i : 0) * s.nfk;
                        float part[GH];
#pragma unroll
                        for (int g = 0; g < GH; ++g) part[g] = 0.f;
#pragma unroll
                        for (int sl = 0; sl < SL; ++sl) {
                            const int piece = r4 + 4 * sl;
                            if (piece < npk) {
                                float x[8];
                                ld_piece(row, piece, x);
#pragma unroll
                                for (int g = 0; g < GH; ++g)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) part[g] = fmaf(qk[sl][g][e], x[e], part[g]);
                            }
                        }
                        const float tot = quad_reduce<GH>(part, r4);
                        if (ok && r4 < GH) {
                            float* dst = sb + phys((a0 + i) * GH + head_of<GH>(r4));
                            *dst += tot;
                        }
                    }
                    release_tile();
                }
            }
            consumer_sync();
            // online softmax over the class
            float mx[GH], alpha[GH];
            block_max(sb, n_c, mx);
#pragma unroll
            for (int g = 0; g < GH; ++g) {
                const float m_new = fmaxf(m_run[g], mx[g]);
                alpha[g] = exp2f(m_run[g] - m_new);
                m_run[g] = m_new;
            }
            float m_mine = m_run[0], a_mine = alpha[0];
#pragma unroll
            for (int g = 1; g < GH; ++g) if (my_head == g) { m_mine = m_run[g]; a_mine = alpha[g]; }
            l_part *= a_mine;
            to_prob(sb, n_c, S, m_mine);
#pragma unroll
            for (int sl = 0; sl < SL; ++sl)
#pragma unroll
                for (int g = 0; g < GH; ++g)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[sl][g][e] *= alpha[g];
            consumer_sync();
            // o^u += p V^mu
            if (ts_v) {
                for (int a0 = 0; a0 < n_c; a0 += ts_v) {
                    const int nt = min(ts_v, n_c - a0);
                    const KV* tile = reinterpret_cast<const KV*>(wait_tile());
                    for (int i = tq4; i < nt; i += 64) {
                        float pg[GH];
                        if constexpr (GH == 4) {
                            const float4 t = *reinterpret_cast<const float4*>(sb + phys((a0 + i) * 4));
                            pg[0] = t.x; pg[1] = t.y; pg[2] = t.z; pg[3] = t.w;
                        } else {
                            const float2 t = *reinterpret_cast<const float2*>(sb + phys((a0 + i) * 2));
                            pg[0] = t.x; pg[1] = t.y;
                        }
                        const KV* row = tile + (size_t)i * s.nfv;
#pragma unroll
                        for (int sl = 0; sl < SL; ++sl) {
                            const int piece = r4 + 4 * sl;
                            if (piece < npv) {
                                float x[8];
                                ld_piece(row, piece, x);
#pragma unroll
                                for (int g = 0; g < GH; ++g)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) acc[sl][g][e] = fmaf(pg[g], x[e], acc[sl][g][e]);
                            }
                        }
                    }
                    release_tile();
                }
            }
            // z_n = alpha z_n + e^{i theta n cls} Y_n, Y = transform of the packed probabilities
            if (s.dcv > 0) {
                consumer_sync();
                const float* Y = fft_run<NC>(sb, other, W, S, log2S, tid);
                for (int n = tid; n < s.k; n += kConsumers) {
                    const int m = n & (S - 1), mc = (S - m) & (S - 1);
                    const float2 t = tw[n];
#pragma unroll
                    for (int cl = 0; cl < NC; ++cl) {
                        const float2 ya = *reinterpret_cast<const float2*>(Y + phys(2 * (m * NC + cl)));
                        const float2 yb = conj(*reinterpret_cast<const float2*>(Y + phys(2 * (mc * NC + cl))));
                        const float2 y0 = make_float2(0.5f * (ya.x + yb.x), 0.5f * (ya.y + yb.y));
                        const float2 dd = csub(ya, yb);
                        const float2 y1 = make_float2(0.5f * dd.y, -0.5f * dd.x);
                        float2 z0 = z_s[n * GH + 2 * cl], z1 = z_s[n * GH + 2 * cl + 1];
                        const float2 t0 = cmul(t, y0), t1 = cmul(t, y1);
                        z_s[n * GH + 2 * cl] = make_float2(fmaf(z0.x, alpha[2 * cl], t0.x), fmaf(z0.y, alpha[2 * cl], t0.y));
                        z_s[n * GH + 2 * cl + 1] = make_float2(fmaf(z1.x, alpha[2 * cl + 1], t1.x), fmaf(z1.y, alpha[2 * cl + 1], t1.y));
                    }
                }
            }
            consumer_sync();
        }
        // fold the per-lane output accumulators into o_s at the natural positions of D^vu
        const int32_t* idf_v = c.idx_full_v + (size_t)h * s.nfv;
#pragma unroll
        for (int sl = 0; sl < SL; ++sl) {
            const int piece = r4 + 4 * sl;
#pragma unroll
            for (int g = 0; g < GH; ++g)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float v = acc[sl][g][e];
                    v += __shfl_xor_sync(0xffffffffu, v, 4);
                    v += __shfl_xor_sync(0xffffffffu, v, 8);
                    v += __shfl_xor_sync(0xffffffffu, v, 16);
                    if (lane < 4 && piece < npv) atomicAdd(o_s + g * s.d + idf_v[piece * 8 + e], v);
                }
        }
    }
    consumer_sync();

    // ------------------------------ window tokens -------------------------------
    float a_win[GH];                                      // rescale of what the classes left in o_s / z_s
#pragma unroll
    for (int g = 0; g < GH; ++g) a_win[g] = 1.f;
    if (w1 > w0) {
        constexpr int SW = 1;                             // head_dim <= 128: at most 16 pieces over 16 lanes
        float qw[SW][GH][8], accw[SW][GH][8];
#pragma unroll
        for (int sl = 0; sl < SW; ++sl) {
            const int piece = r16 + 16 * sl;
#pragma unroll
            for (int g = 0; g < GH; ++g)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    qw[sl][g][e] = piece < npw ? q_s[g * s.d + piece * 8 + e] : 0.f;
                    accw[sl][g][e] = 0.f;
                }
        }
        float* sb = fA;
        for (int t0 = w0; t0 < w1; t0 += wchunk) {
            const int n_tok = min(w1, t0 + wchunk) - t0;
            const WinSegs sg = win_segments(t0, t0 + n_tok, n_init, n_local, head, s.l_local);
            for (int si = 0; si < sg.n; ++si)
                for (int r0 = 0; r0 < sg.cnt[si]; r0 += ts_w) {
                    const int nt = min(ts_w, sg.cnt[si] - r0);
                    const KV* tile = reinterpret_cast<const KV*>(wait_tile());
                    for (int i0 = 0; i0 < nt; i0 += 16) {
                        const int i = i0 + tq16;
                        const bool ok = i < nt;
                        const KV* row = tile + (size_t)(ok ? i : 0) * s.d;
                        float part[GH];
#pragma unroll
                        for (int g = 0; g < GH; ++g) part[g] = 0.f;
#pragma unroll
                        for (int sl = 0; sl < SW; ++sl) {
                            const int piece = r16 + 16 * sl;
                            if (piece < npw) {
                                float x[8];
                                ld_piece(row, piece, x);
#pragma unroll
                                for (int g = 0; g < GH; ++g)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) part[g] = fmaf(qw[sl][g][e], x[e], part[g]);
                            }
                        }
                        float tot = quad_reduce<GH>(part, r16 & 3);
                        tot += __shfl_xor_sync(0xffffffffu, tot, 4);
                        tot += __shfl_xor_sync(0xffffffffu, tot, 8);
                        if (ok && r16 < GH) sb[phys((sg.tok[si] + r0 + i) * GH + head_of<GH>(r16))] = tot;
                    }
                    release_tile();
                }
            consumer_sync();
            float mx[GH], alpha[GH];
            block_max(sb, n_tok, mx);
#pragma unroll
            for (int g = 0; g < GH; ++g) {
                const float m_new = fmaxf(m_run[g], mx[g]);
                alpha[g] = exp2f(m_run[g] - m_new);
                m_run[g] = m_new;
                a_win[g] *= alpha[g];
            }
            float m_mine = m_run[0], a_mine = alpha[0];
#pragma unroll
            for (int g = 1; g < GH; ++g) if (my_head == g) { m_mine = m_run[g]; a_mine = alpha[g]; }
            l_part *= a_mine;
            to_prob(sb, n_tok, n_tok, m_mine);
#pragma unroll
            for (int sl = 0; sl < SW; ++sl)
#pragma unroll
                for (int g = 0; g < GH; ++g)
#pragma unroll
                    for (int e = 0; e < 8; ++e) accw[sl][g][e] *= alpha[g];
            consumer_sync();
            for (int si = 0; si < sg.n; ++si)
                for (int r0 = 0; r0 < sg.cnt[si]; r0 += ts_w) {
                    const int nt = min(ts_w, sg.cnt[si] - r0);
                    const KV* tile = reinterpret_cast<const KV*>(wait_tile());
                    for (int i = tq16; i < nt; i += 16) {
                        float pg[GH];
                        const int a = sg.tok[si] + r0 + i;
                        if constexpr (GH == 4) {
                            const float4 t = *reinterpret_cast<const float4*>(sb + phys(a * 4));
                            pg[0] = t.x; pg[1] = t.y; pg[2] = t.z; pg[3] = t.w;
                        } else {
                            const float2 t = *reinterpret_cast<const float2*>(sb + phys(a * 2));
                            pg[0] = t.x; pg[1] = t.y;
                        }
                        const KV* row = tile + (size_t)i * s.d;
#pragma unroll
                        for (int sl = 0; sl < SW; ++sl) {
                            const int piece = r16 + 16 * sl;
                            if (piece < npw) {
                                float x[8];
                                ld_piece(row, piece, x);
#pragma unroll
                                for (int g = 0; g < GH; ++g)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) accw[sl][g][e] = fmaf(pg[g], x[e], accw[sl][g][e]);
                            }
                        }
                    }
                    release_tile();
                }
            consumer_sync();
        }
        // rescale what the classes left, then add the window accumulators
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
#pragma unroll
        for (int sl = 0; sl < SW; ++sl) {
            const int piece = r16 + 16 * sl;
#pragma unroll
            for (int g = 0; g < GH; ++g)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float v = accw[sl][g][e];
                    v += __shfl_xor_sync(0xffffffffu, v, 16);
                    if (lane < 16 && piece < npw) atomicAdd(o_s + g * s.d + piece * 8 + e, v);
                }
        }
    }
    // sum of p per head
    {
        float v = l_part;
#pragma unroll
        for (int o = 16; o >= GH; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane < GH) atomicAdd(red_s + 8 * GH + lane, v);
    }
    consumer_sync();

    // ------------------------------ partial results ------------------------------
    for (int i = tid; i < GH * s.d; i += kConsumers) {
        int g = i / s.d, e = i - g * s.d;
        if (g < ng) ws.o[(((size_t)b * s.Hq + g_first + g) * p.n_split + split) * s.d + e] = o_s[i];
    }
    for (int i = tid; i < s.k * GH; i += kConsumers) {
        int n = i / GH, g = i - n * GH;
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

template <typename KV, int GH, int SL>
cudaError_t launch_fft_t(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* q, char* ws, cudaStream_t st) {
    const int S = s.T / s.P;
    const FftSmem L = fft_smem_layout(S, s.k, GH, s.d, s.nfk);
    cudaError_t err = ensure_dynamic_smem(decode_fft_kernel<KV, GH, SL>, (size_t)L.total);
    if (err != cudaSuccess) return err;
    decode_fft_kernel<KV, GH, SL><<<dim3(p.n_split, s.Hkv * p.n_pass, s.B), kThreads, L.total, st>>>(
        s, c, p, static_cast<const KV*>(q), ws);
    return cudaGetLastError();
}

}  // namespace

size_t decode_fft_smem_bytes(const Dims& s, int gh) {
    return (size_t)fft_smem_layout(s.T / s.P, s.k, gh, s.d, s.nfk).total;
}

cudaError_t launch_decode_fft(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, const void* q, char* ws,
                              cudaStream_t st) {
    const int sl = ((s.nfk > s.nfv ? s.nfk : s.nfv) + 31) / 32;
    const bool two = sl > 1;
    if (dtype == FA_BF16) {
        if (p.gh == 4) return two ? launch_fft_t<__nv_bfloat16, 4, 2>(s, c, p, q, ws, st) : launch_fft_t<__nv_bfloat16, 4, 1>(s, c, p, q, ws, st);
        return two ? launch_fft_t<__nv_bfloat16, 2, 2>(s, c, p, q, ws, st) : launch_fft_t<__nv_bfloat16, 2, 1>(s, c, p, q, ws, st);
    }
    if (p.gh == 4) return two ? launch_fft_t<float, 4, 2>(s, c, p, q, ws, st) : launch_fft_t<float, 4, 1>(s, c, p, q, ws, st);
    return two ? launch_fft_t<float, 2, 2>(s, c, p, q, ws, st) : launch_fft_t<float, 2, 1>(s, c, p, q, ws, st);
}

}  // namespace fa
