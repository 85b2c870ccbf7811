// fa_compress, transform path (Eq.3-4 evaluated without forming F): the coefficients of a compressed
// dimension are the k lowest bins of the discrete Fourier transform of its zero-extended token column,
//   C[2n][e] + i C[2n+1][e] = Z_n = sum_j x_j e^{i theta n j},   theta = 2 pi / T,
// and with the middle tokens split into residue classes j = c + P a (a = 0..S-1, S = T / P >= k)
//   Z_n = sum_c e^{i theta n c} Y^c_n,   Y^c_m = sum_a x_{c + P a} e^{2 pi i m a / S},
// i.e. P transforms of length S and one twist-and-add per class instead of L_mid * k basis terms.
// All arithmetic is fp32 (no rounded basis), and the sums run in a fixed order: the result is the same
// bits on every run.
//
// One CTA owns four compressed dims of one (batch row, KV head, side): two real token columns ride in
// one complex transform (real-pair packing), two such complex lanes side by side in packed fp32 pairs
// (a point is (re0, re1, im0, im1)).  Per class: gather the class's tokens of the four dims from the
// prefilled K / V into the transform buffer at their digit-reversed places, run the decimation-in-time
// passes in place (natural order out), split each bin pair (m, S - m) into the spectra of the real
// columns, rotate by e^{i theta n c} and add into the CTA's accumulator.  At the end the accumulator is
// written to the coefficient rows (cos sums in even rows, sin sums in odd rows).
//
// The gather reads 2-byte elements from token rows that lie a whole K / V row apart: the 32-byte sectors
// it touches are shared by the CTAs of neighbouring dims through L2, but the load instructions are not
// coalesced; this path is the exact, order-fixed alternative to the tensor-core contraction, not the
// fast one.
#include "fa_common.cuh"

namespace fa {
namespace {

using bf16 = __nv_bfloat16;
typedef unsigned long long u64;
constexpr int kFftThreads = 256;

__device__ __forceinline__ uint32_t smem_a(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ float2 cis_frac(float frac) {
    const float a = 6.283185307179586f * (frac - (frac >= 0.5f ? 1.0f : 0.0f));
    return make_float2(__cosf(a), __sinf(a));
}
// Two complex numbers side by side: real parts and imaginary parts as packed fp32 pairs.
struct P2 { u64 v; };
__device__ __forceinline__ P2 pk(float a, float b) { P2 r; asm("mov.b64 %0, {%1,%2};" : "=l"(r.v) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ void unpk(P2 x, float& a, float& b) { asm("mov.b64 {%0,%1}, %2;" : "=f"(a), "=f"(b) : "l"(x.v)); }
__device__ __forceinline__ P2 operator+(P2 a, P2 b) { P2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ P2 operator-(P2 a, P2 b) { P2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ P2 operator*(P2 a, P2 b) { P2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ P2 pfma(P2 a, P2 b, P2 c) { P2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v)); return r; }
struct C2 { P2 re, im; };
__device__ __forceinline__ C2 operator+(C2 a, C2 b) { return C2{a.re + b.re, a.im + b.im}; }
__device__ __forceinline__ C2 operator-(C2 a, C2 b) { return C2{a.re - b.re, a.im - b.im}; }
__device__ __forceinline__ C2 cmulw(C2 a, float wr, float wi) {          // times the scalar wr + i wi
    const P2 r = pk(wr, wr), i = pk(wi, wi);
    return C2{(a.re * r) - (a.im * i), pfma(a.re, i, a.im * r)};
}
__device__ __forceinline__ C2 ld_pt(const float* p) {
    C2 r;
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(r.re.v), "=l"(r.im.v) : "r"(smem_a(p)) : "memory");
    return r;
}
__device__ __forceinline__ void st_pt(float* p, C2 v) {
    asm volatile("st.shared.v2.b64 [%0], {%1,%2};" ::"r"(smem_a(p)), "l"(v.re.v), "l"(v.im.v) : "memory");
}
// 16 bytes of padding after every 128 bytes, 1 KB and 8 KB of a transform buffer (bank spreading)
__host__ __device__ constexpr int pf(int f) { return f + ((f >> 5) << 2) + ((f >> 8) << 2) + ((f >> 11) << 2); }

// One in-place decimation-in-time pass of radix 2 or 4 (exponent +2 pi i) over the sub-transforms of
// length 2^LL of a length-2^LS transform: twiddle the inputs, then the butterfly.
template <int RL>
__device__ __forceinline__ void dit_pass(float* base, const float2* __restrict__ tws, int LS, int LL, int tid) {
    constexpr int R = 1 << RL;
    const int STL = LL - RL, PERL = LS - RL, sh = LS - LL, smask = (1 << LS) - 1;
#pragma unroll 1
    for (int item = tid; item < (1 << PERL); item += kFftThreads) {
        const int blk = item >> STL, j = item & ((1 << STL) - 1);
        const int e0 = (blk << LL) + j;
        C2 v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = ld_pt(base + pf((e0 + (r << STL)) * 4));
        if (STL > 0) {
#pragma unroll
            for (int q = 1; q < R; ++q) {
                const float2 w = tws[((q * j) << sh) & smask];
                v[q] = cmulw(v[q], w.x, w.y);
            }
        }
        if constexpr (R == 2) {
            const C2 t = v[0];
            v[0] = t + v[1];
            v[1] = t - v[1];
        } else {
            const C2 t0 = v[0] + v[2], t1 = v[0] - v[2], t2 = v[1] + v[3], d = v[1] - v[3];     // i d = (-d.im, d.re)
            v[0] = t0 + t2;
            v[2] = t0 - t2;
            v[1] = C2{t1.re - d.im, t1.im + d.re};
            v[3] = C2{t1.re + d.im, t1.im - d.re};
        }
#pragma unroll
        for (int r = 0; r < R; ++r) st_pt(base + pf((e0 + (r << STL)) * 4), v[r]);
    }
}
__host__ __device__ constexpr int rl_of(int l) { return l >= 2 ? 2 : 1; }         // radix 4 where possible
// Position of natural index a in the input order of the decimation-in-time passes (digit reversal for the
// radix sequence the passes use, taken from the top sub-transform length down).
__device__ __forceinline__ int dit_in_pos(int LS, int a) {
    int pos = 0;
    for (int cur = LS; cur > 0;) {
        const int rl = rl_of(cur);
        cur -= rl;
        pos += (a & ((1 << rl) - 1)) << cur;
        a >>= rl;
    }
    return pos;
}

template <typename KV>
__global__ void __launch_bounds__(kFftThreads) compress_fft_kernel(Dims s, CacheDev c, const KV* __restrict__ K,
                                                                   const KV* __restrict__ V, int64_t sb, int64_t st, int64_t sh,
                                                                   int L, int LS) {
    extern __shared__ __align__(16) unsigned char fsm[];
    const int S = 1 << LS;
    float* fbuf = reinterpret_cast<float*>(fsm);                           // [S] points of 4 floats, padded
    float2* tws = reinterpret_cast<float2*>(fbuf + pf(S * 4) + 8);         // e^{2 pi i t / S}
    uint16_t* rev = reinterpret_cast<uint16_t*>(tws + S);
    float* zacc = reinterpret_cast<float*>(rev + S + 8);                   // [k][8]: (A.re x2, A.im x2, B.re x2, B.im x2)
    const int tid = threadIdx.x;
    const int quad = blockIdx.x, h = blockIdx.y, b = blockIdx.z >> 1, side = blockIdx.z & 1;
    const int ncomp = side == 0 ? s.dck : s.dcv;
    if (4 * quad >= ncomp) return;
    const int n_init = min(L, s.l_init);
    const int n_local = min(L - n_init, s.l_local);
    const int n_mid = L - n_init - n_local;
    const int log2P = 31 - __clz(s.P);
    const int32_t* idc = (side == 0 ? c.idx_comp_k : c.idx_comp_v) + (size_t)h * ncomp + 4 * quad;
    const int nd = min(4, ncomp - 4 * quad);                               // (ncomp is a multiple of 8: always 4)
    int dim[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) dim[i] = i < nd ? idc[i] : idc[0];
    const KV* X = (side == 0 ? K : V) + (size_t)b * sb + (size_t)h * sh + (size_t)n_init * st;

    for (int i = tid; i < S; i += kFftThreads) {
        tws[i] = cis_frac((float)i / (float)S);
        rev[i] = (uint16_t)dit_in_pos(LS, i);
    }
    for (int i = tid; i < 8 * s.k; i += kFftThreads) zacc[i] = 0.f;
    __syncthreads();

#pragma unroll 1
    for (int cls = 0; cls < s.P && cls < n_mid; ++cls) {
        const int n_c = (n_mid - cls + s.P - 1) >> log2P;
        // gather: token a of the class at its digit-reversed place; (re0, re1, im0, im1) = dims (0, 2, 1, 3) of the quad
#pragma unroll 1
        for (int a = tid; a < S; a += kFftThreads) {
            float x0 = 0.f, x1 = 0.f, x2 = 0.f, x3 = 0.f;
            if (a < n_c) {
                const KV* row = X + (size_t)(cls + (a << log2P)) * st;
                x0 = ld_f(row + dim[0]); x1 = ld_f(row + dim[1]); x2 = ld_f(row + dim[2]); x3 = ld_f(row + dim[3]);
            }
            *reinterpret_cast<float4*>(fbuf + pf(rev[a] * 4)) = make_float4(x0, x2, x1, x3);
        }
        __syncthreads();
        // sub-transform lengths grow from the smallest up to S
        {
            int n = 0;
            for (int ll = LS; ll > 0; ll -= rl_of(ll)) ++n;
#pragma unroll 1
            for (int i = n - 1; i >= 0; --i) {
                int ll = LS;
                for (int j = 0; j < i; ++j) ll -= rl_of(ll);
                if (rl_of(ll) == 2) dit_pass<2>(fbuf, tws, LS, ll, tid);
                else dit_pass<1>(fbuf, tws, LS, ll, tid);
                __syncthreads();
            }
        }
        // bins (m, S - m) -> spectra of the real columns, rotated by the class phase, added to the accumulator
#pragma unroll 1
        for (int pr = tid; pr < S / 2; pr += kFftThreads) {
            const int m = pr, mc = pr == 0 ? S / 2 : S - pr;
            if (m >= s.k && mc >= s.k) continue;
            const C2 ya = ld_pt(fbuf + pf(m * 4)), yb = ld_pt(fbuf + pf(mc * 4));
            const float2 twm = cis_frac((float)((m * cls) & (s.T - 1)) / (float)s.T), twc = cis_frac((float)((mc * cls) & (s.T - 1)) / (float)s.T);
            const P2 half = pk(0.5f, 0.5f), zero = pk(0.f, 0.f);
            C2 zAm, zBm, zAc, zBc;
            if (pr != 0) {
                // first columns: y0 = (ya + conj(yb)) / 2, second columns: y1 = (ya - conj(yb)) / (2 i); bin mc holds the conjugates
                const C2 y0 = C2{(ya.re + yb.re) * half, (ya.im - yb.im) * half};
                const C2 y1 = C2{(ya.im + yb.im) * half, (yb.re - ya.re) * half};
                zAm = cmulw(y0, twm.x, twm.y);
                zBm = cmulw(y1, twm.x, twm.y);
                zAc = cmulw(C2{y0.re, zero - y0.im}, twc.x, twc.y);
                zBc = cmulw(C2{y1.re, zero - y1.im}, twc.x, twc.y);
            } else {
                // bins 0 and S/2 are real for a real column: (re, im) of the packed value are the two columns
                zAm = cmulw(C2{ya.re, zero}, twm.x, twm.y);
                zBm = cmulw(C2{ya.im, zero}, twm.x, twm.y);
                zAc = cmulw(C2{yb.re, zero}, twc.x, twc.y);
                zBc = cmulw(C2{yb.im, zero}, twc.x, twc.y);
            }
            auto add = [&](int n, const C2& A, const C2& B) {
                float a0, a1, a2, a3, b0, b1, b2, b3;
                unpk(A.re, a0, a1); unpk(A.im, a2, a3); unpk(B.re, b0, b1); unpk(B.im, b2, b3);
                float4* z = reinterpret_cast<float4*>(zacc + 8 * n);
                float4 u = z[0], w = z[1];
                u.x += a0; u.y += a1; u.z += a2; u.w += a3;
                w.x += b0; w.y += b1; w.z += b2; w.w += b3;
                z[0] = u; z[1] = w;
            };
            if (m < s.k) add(m, zAm, zBm);
            if (mc < s.k) add(mc, zAc, zBc);
        }
        __syncthreads();
    }
    // coefficient rows 2n (cos sums = Re Z_n) and 2n + 1 (sin sums = Im Z_n), columns 4 quad .. 4 quad + 3
    float* coef = coef_rows(side == 0 ? c.coef_k : c.coef_v, s, b, h, ncomp) + 4 * quad;
#pragma unroll 1
    for (int n = tid; n < s.k; n += kFftThreads) {
        const float* z = zacc + 8 * n;                    // A = columns (0, 2), B = columns (1, 3)
        *reinterpret_cast<float4*>(coef + (size_t)(2 * n) * ncomp) = make_float4(z[0], z[4], z[1], z[5]);
        *reinterpret_cast<float4*>(coef + (size_t)(2 * n + 1) * ncomp) = make_float4(z[2], z[6], z[3], z[7]);
    }
}

template <typename KV>
cudaError_t launch_fft_t(const Dims& s, const CacheDev& c, const void* K, const void* V, int64_t sb, int64_t st, int64_t sh, int L,
                         int LS, cudaStream_t stream) {
    const int S = 1 << LS;
    const size_t smem = 4 * (size_t)(pf(S * 4) + 8) + 8 * (size_t)S + 2 * (size_t)(S + 8) + 32 * (size_t)s.k + 64;
    cudaError_t err = ensure_dynamic_smem(compress_fft_kernel<KV>, smem);
    if (err != cudaSuccess) return err;
    const int max_comp = s.dck > s.dcv ? s.dck : s.dcv;
    compress_fft_kernel<KV><<<dim3(max_comp / 4, s.Hkv, s.B * 2), kFftThreads, smem, stream>>>(
        s, c, static_cast<const KV*>(K), static_cast<const KV*>(V), sb, st, sh, L, LS);
    return cudaGetLastError();
}

}  // namespace

// True if the transform path serves this layout: power-of-two period and class count, S = T / P a power of two in
// [32, 2048] with S >= k (every frequency has a bin of its own), shared memory within the limit.
bool compress_fft_supported(const Dims& s, int* log2S) {
    if (s.T < 2 || (s.T & (s.T - 1)) || s.P < 1 || (s.P & (s.P - 1)) || s.T % s.P) return false;
    const int S = s.T / s.P;
    int ls = 0;
    while ((1 << ls) < S) ++ls;
    if ((1 << ls) != S || ls < 5 || ls > 11 || s.k > S) return false;
    if (s.dck % 4 || s.dcv % 4 || (s.dck == 0 && s.dcv == 0)) return false;
    const size_t smem = 4 * (size_t)(pf(S * 4) + 8) + 8 * (size_t)S + 2 * (size_t)(S + 8) + 32 * (size_t)s.k + 64;
    if (smem > 200 * 1024) return false;
    *log2S = ls;
    return true;
}

// Coefficients only (the caller runs the partition / gather kernel; the coefficients need no zeroing: every row is stored).
cudaError_t launch_compress_fft(const Dims& s, const CacheDev& c, int dtype, const void* K, const void* V, int64_t sb, int64_t st,
                                int64_t sh, int L, int log2S, cudaStream_t stream) {
    if (dtype == FA_BF16) return launch_fft_t<__nv_bfloat16>(s, c, K, V, sb, st, sh, L, log2S, stream);
    return launch_fft_t<float>(s, c, K, V, sb, st, sh, L, log2S, stream);
}

}  // namespace fa
