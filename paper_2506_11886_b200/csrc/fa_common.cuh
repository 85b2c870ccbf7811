// Shared declarations of the CUDA library: derived layout numbers, element
// loads/stores, basis phase, launch plans.  Product code only; the CPU oracle
// shares nothing with this file.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fa.h"

namespace fa {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegBig = -1.0e30f;   // "no token yet" running max (finite, so differences stay finite)
constexpr int kNumSmsDefault = 148;     // B200; used only when no device can be asked (sm_count())
constexpr int kBarSlots = 256;          // (b, KV head, pass) triples that can own barrier counters in the first 4 KiB of a workspace
constexpr int kStateStride = 8;        // int32 words of cache state per batch row

// Layout numbers every kernel needs, passed by value.
struct Dims {
    int B, Hq, Hkv, G, d;
    int nfk, nfv, dck, dcv;     // |D^ku|, |D^vu|, |D^kc|, |D^vc|
    int M, k, T;                // Eq.4
    int l_init, l_local, max_mid;
    int P, S_cap;               // residue classes and slots per class of K^mu / V^mu
    int norm;
    float scale;
};

inline Dims make_dims(const fa_layout& l) {
    Dims s;
    s.B = l.batch; s.Hq = l.n_q_heads; s.Hkv = l.n_kv_heads; s.G = l.n_q_heads / l.n_kv_heads; s.d = l.head_dim;
    s.nfk = l.n_full_k; s.nfv = l.n_full_v; s.dck = l.head_dim - l.n_full_k; s.dcv = l.head_dim - l.n_full_v;
    s.M = l.n_coef; s.k = l.n_coef / 2; s.T = l.period;
    s.l_init = l.l_init; s.l_local = l.l_local; s.max_mid = l.max_mid;
    s.P = l.mid_classes; s.S_cap = (l.max_mid + l.mid_classes - 1) / l.mid_classes;
    s.norm = l.norm; s.scale = l.softmax_scale;
    return s;
}

// Device view of fa_cache (same fields, typed for kernels).
struct CacheDev {
    const int32_t *idx_full_k, *idx_comp_k, *idx_full_v, *idx_comp_v;
    void *k_init, *v_init, *k_local, *v_local, *k_mid, *v_mid;
    float *coef_k, *coef_v;
    int32_t *state, *status;
};

inline CacheDev make_cache(const fa_cache& c) {
    CacheDev o;
    o.idx_full_k = c.idx_full_k; o.idx_comp_k = c.idx_comp_k; o.idx_full_v = c.idx_full_v; o.idx_comp_v = c.idx_comp_v;
    o.k_init = c.k_init; o.v_init = c.v_init; o.k_local = c.k_local; o.v_local = c.v_local;
    o.k_mid = c.k_mid; o.v_mid = c.v_mid; o.coef_k = c.coef_k; o.coef_v = c.coef_v;
    o.state = c.state; o.status = c.status;
    return o;
}

// Plan of one fa_decode_attention call; a pure function of the layout so that
// fa_workspace_bytes and the launch agree.
struct DecodePlan {
    int algo;          // FA_DECODE_DIRECT or FA_DECODE_FFT
    int gh;            // query heads of one KV head handled together by one CTA (<= 4)
    int n_pass;        // ceil(G / gh)
    int n_split;       // CTAs that share the middle tokens of one (b, KV head, pass)
    int n_wsplit;      // CTAs that hold only window tokens (0: the windows are spread over the n_split CTAs)
    int n_part;        // n_split + n_wsplit: partial results per query head
    int fused;         // 1: the main kernel also forms u and merges the partial results (cooperative launch)
    int n_slice;       // CTAs that share the coefficient rows of one (b, KV head) in the epilogue
    int rows_pro;      // coefficient rows per prologue CTA
    int fft_log2;      // log2 of the transform length (FFT path)
    int nb;            // classes transformed together by one CTA (FFT path)
    int occ;           // CTAs per SM the main kernel is built for (FFT path: 1, or 2 with a shorter ring)
    int split;         // 1: the split build of the fused kernel (a tile group of warps beside the transform group)
    // workspace offsets in bytes
    size_t off_bar, off_u, off_ml, off_o, off_z, off_oc, off_om, off_cnt, total;
};

// V^mu of bf16 caches is stored with its 16-byte chunks (8 dims) permuted inside each row:
// chunk c of slot a sits at chunk c ^ v_swz(a, chunks per row).  A bulk copy of a class then
// lands in shared memory in an image whose 8x8 matrix loads (ldmatrix) of eight consecutive
// slots hit eight different bank groups.  fp32 caches are stored plainly.
__host__ __device__ inline int v_swz(int a, int nchunks) {
    switch (nchunks) {
        case 2: return (a >> 2) & 1;
        case 4: return (a >> 1) & 3;
        case 6: return (a >> 2) & 1;
        case 8: return a & 7;
        default: return 0;
    }
}
// Element offset of dim slot e of V^mu row (slot) a inside its row of nfv elements.
__host__ __device__ inline int v_mid_col(int a, int e, int nfv, int dtype) {
    if (dtype != FA_BF16) return e;
    return ((((e >> 3) ^ v_swz(a, nfv >> 3)) << 3) | (e & 7));
}

fa_status plan_decode(const fa_layout& l, DecodePlan* plan);
int sm_count();                          // SMs of the current device, cached per device
bool cooperative_launch_supported();     // of the current device, cached per device
fa_status check_layout(const fa_layout* l);

// Kernel launchers (defined next to their kernels).  All return the launch error, if any.
cudaError_t launch_validate(const Dims&, const CacheDev&, cudaStream_t);
cudaError_t launch_compress(const Dims&, const CacheDev&, int dtype, const void* K, const void* V, int64_t sb,
                            int64_t st, int64_t sh, int L, bool with_coef, bool ordered, bool mid_rows, bool zero_coef, cudaStream_t,
                            bool chained = false);
bool compress_tc_gathers(const Dims& s);
// The same path on CTA pairs (fa_compress_tc2.cu): needs an even number of 128-row tiles.
bool compress_tc2_supported(const Dims& s);
bool compress_tc2_gathers(const Dims& s);
cudaError_t launch_compress_tc2(const Dims&, const CacheDev&, const void* K, const void* V, int64_t sb, int64_t st, int64_t sh,
                                int L, bool ordered, bool gather, cudaStream_t);
// Tensor-core reconstruction of the dimension selection (fa_select_tc.cu).
bool reconstruct_tc_supported(const Dims& s, int dtype, const void* K, const void* V, int64_t sb, int64_t st, int64_t sh, int n_mid);
size_t reconstruct_tc_scratch_bytes(const Dims& s);
cudaError_t launch_reconstruct_tc(const Dims& s, const float* coef_k, const float* coef_v, const void* K, const void* V, int64_t sb,
                                  int64_t st, int64_t sh, int n_init, int n_mid, float* sq, int32_t* status, void* scratch,
                                  cudaStream_t stream);
bool compress_fft_supported(const Dims&, int* log2S);
cudaError_t launch_compress_fft(const Dims&, const CacheDev&, int dtype, const void* K, const void* V, int64_t sb, int64_t st,
                                int64_t sh, int L, int log2S, cudaStream_t);
bool compress_tc_supported(const Dims&, int dtype, int64_t sb, int64_t st, int64_t sh);
cudaError_t launch_compress_tc(const Dims&, const CacheDev&, const void* K, const void* V, int64_t sb, int64_t st, int64_t sh,
                               int L, bool ordered, bool gather, cudaStream_t);
cudaError_t launch_append(const Dims&, const CacheDev&, int dtype, const void* k_new, const void* v_new, cudaStream_t);
cudaError_t launch_decode_prologue(const Dims&, const CacheDev&, int dtype, const DecodePlan&, const void* q, char* ws,
                                   cudaStream_t);
cudaError_t launch_decode_direct(const Dims&, const CacheDev&, int dtype, const DecodePlan&, const void* q, char* ws,
                                 cudaStream_t);
// k_new / v_new non-null: a fused step (the push of Eq.5 rides on the decode launch; fused plans with one pass only).
cudaError_t launch_decode_fft(const Dims&, const CacheDev&, int dtype, const DecodePlan&, const void* q, void* out, char* ws,
                              const void* k_new, const void* v_new, cudaStream_t);
size_t decode_fft_smem_bytes(const Dims&, int log2S, int gh, int nb, int occ = 1, int split = 0);
bool decode_fft_fused_fits(const Dims&, int log2S, int gh, int nb, int n_part, int occ = 1, int split = 0);
bool decode_fft_launchable(const Dims&, const DecodePlan&);
cudaError_t launch_decode_epilogue(const Dims&, const CacheDev&, int dtype, const DecodePlan&, void* out, char* ws,
                                   cudaStream_t);

// Raises a kernel's dynamic shared memory limit when a launch needs more than it has been
// given so far on the current device (no CUDA call at all in the steady state, so launches
// stay capturable in CUDA graphs after a warm-up call).
cudaError_t ensure_dynamic_smem_impl(const void* kernel, size_t bytes);
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, size_t bytes) {
    return ensure_dynamic_smem_impl(reinterpret_cast<const void*>(kernel), bytes);
}

#ifdef __CUDACC__
// ---- element access ---------------------------------------------------------
__device__ __forceinline__ float ld_f(const float* p) { return *p; }
__device__ __forceinline__ float ld_f(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st_f(float* p, float v) { *p = v; }
__device__ __forceinline__ void st_f(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Reconstruction weight of coefficient row m (Eq.6).
__device__ __forceinline__ float recon_weight(int norm, int m, int k, int T) {
    if (norm == FA_NORM_PAPER) return 1.0f / (float)k;
    if (m == 0) return 1.0f / (float)T;
    if (m == 1) return 0.0f;
    return 2.0f / (float)T;
}

// Eq.4: cos and sin of 2 pi n j / T, with n * j reduced modulo T in integers first.
__device__ __forceinline__ void basis_cs(int n, int j, int T, float* c, float* s) {
    long long r = ((long long)n * (long long)j) % (long long)T;
    sincospif(2.0f * (float)r / (float)T, s, c);
}

// Address of row (class c, slot a) of K^mu / V^mu of (b, h).
template <typename KV>
__device__ __forceinline__ KV* mid_row(void* base, const Dims& s, int b, int h, int c, int a, int nfull) {
    size_t row = (((size_t)b * s.Hkv + h) * s.P + c) * (size_t)s.S_cap + a;
    return reinterpret_cast<KV*>(base) + row * (size_t)nfull;
}
template <typename KV>
__device__ __forceinline__ KV* win_row(void* base, const Dims& s, int b, int h, int rows, int r) {
    size_t row = ((size_t)b * s.Hkv + h) * (size_t)rows + r;
    return reinterpret_cast<KV*>(base) + row * (size_t)s.d;
}
__device__ __forceinline__ float* coef_rows(float* base, const Dims& s, int b, int h, int ncomp) {
    return base + (((size_t)b * s.Hkv + h) * (size_t)s.M) * (size_t)ncomp;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
#endif  // __CUDACC__

}  // namespace fa
