// fa_select_dims (Sec. 3.4): which dimensions of K and of V to keep per token and which to hold as
// Fourier coefficients.  Every dimension of the middle segment is compressed (Eq.3) and reconstructed
// (Eq.6 weights); the dimensions with the largest mean squared reconstruction error are kept.
//   1. coefficients of all d dims: fa_compress on a scratch cache whose layout compresses everything
//      (the tensor-core kernel already multiplies all dims), carved from the workspace;
//   2. the middle tokens rebuilt, x~[j][e] = sum_m w_m F[m][j] C[m][e], and the squared error summed per dim:
//      for bf16 tensors on the tensor cores (reconstruct_tc_kernel, fa_select_tc.cu), otherwise mse_kernel
//      (fp32, 64 middle tokens per CTA, basis by rotation recurrence re-seeded exactly every 16 frequencies);
//   3. select_kernel: mean over the batch rows, rank by (error, index), write the sorted index sets.
#include <cstring>

#include "fa_common.cuh"

namespace fa {

fa_status check_layout(const fa_layout* l);

namespace {

constexpr int kMseTokens = 64;      // middle tokens per CTA
constexpr int kMseRows = 32;        // coefficient rows staged per round (16 frequencies)

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

__global__ void iota_rows_kernel(int32_t* p, int rows, int d) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < rows * d) p[i] = i % d;
}

// grid (ceil(n_mid / 64), Hkv * 2, B), 256 threads = 64 tokens x 4 groups of d/4 dims.
// coef: [B][Hkv][M][d] of the side; X: prefill tensor of the side; sq: [B][Hkv][2][d] sums of squared errors.
template <typename KV, int DPT>
__global__ void __launch_bounds__(256) mse_kernel(Dims s, const float* __restrict__ coef_k, const float* __restrict__ coef_v,
                                                  const KV* __restrict__ K, const KV* __restrict__ V, int64_t sb, int64_t st,
                                                  int64_t sh, int n_init, int n_mid, float* __restrict__ sq) {
    __shared__ __align__(16) float c_s[kMseRows * 256];
    __shared__ float err_s[256];
    const int tid = threadIdx.x, tj = tid & (kMseTokens - 1), dg = tid / kMseTokens;
    const int h = blockIdx.y >> 1, side = blockIdx.y & 1, b = blockIdx.z;
    const int j = blockIdx.x * kMseTokens + tj;
    const bool live = j < n_mid;
    const int d = s.d, e0 = dg * DPT;
    const float* coef = (side == 0 ? coef_k : coef_v) + ((size_t)b * s.Hkv + h) * (size_t)s.M * d;
    err_s[tid] = 0.f;
    float acc[DPT];
#pragma unroll
    for (int i = 0; i < DPT; ++i) acc[i] = 0.f;
    float dc, ds;                                    // rotation by one frequency for this token
    basis_cs(1, live ? j : 0, s.T, &dc, &ds);
    for (int m0 = 0; m0 < s.M; m0 += kMseRows) {
        const int rows = min(kMseRows, s.M - m0);
        __syncthreads();
        for (int i = tid; i < rows * (d >> 2); i += 256)
            reinterpret_cast<float4*>(c_s)[i] = __ldg(reinterpret_cast<const float4*>(coef + (size_t)m0 * d) + i);
        __syncthreads();
        float c, sn;
        basis_cs(m0 >> 1, live ? j : 0, s.T, &c, &sn);       // exact re-seed
        for (int r = 0; r < rows; r += 2) {
            const float wc = recon_weight(s.norm, m0 + r, s.k, s.T) * c, ws = recon_weight(s.norm, m0 + r + 1, s.k, s.T) * sn;
            const float* rc = c_s + r * d + e0;
            const float* rs = rc + d;
#pragma unroll
            for (int i = 0; i < DPT; i += 4) {
                const float4 a = *reinterpret_cast<const float4*>(rc + i), q = *reinterpret_cast<const float4*>(rs + i);
                acc[i] = fmaf(wc, a.x, fmaf(ws, q.x, acc[i]));
                acc[i + 1] = fmaf(wc, a.y, fmaf(ws, q.y, acc[i + 1]));
                acc[i + 2] = fmaf(wc, a.z, fmaf(ws, q.z, acc[i + 2]));
                acc[i + 3] = fmaf(wc, a.w, fmaf(ws, q.w, acc[i + 3]));
            }
            const float c2 = fmaf(c, dc, -sn * ds);
            sn = fmaf(c, ds, sn * dc);
            c = c2;
        }
    }
    __syncthreads();
    if (live) {
        const KV* x = (side == 0 ? K : V) + (size_t)b * sb + (size_t)(n_init + j) * st + (size_t)h * sh + e0;
#pragma unroll
        for (int i = 0; i < DPT; ++i) {
            const float df = acc[i] - ld_f(x + i);
            atomicAdd(err_s + e0 + i, df * df);
        }
    }
    __syncthreads();
    if (tid < d) atomicAdd(sq + (((size_t)b * s.Hkv + h) * 2 + side) * d + tid, err_s[tid]);
}

// grid (Hkv, 2), d threads (<= 256).  Normalises the sums to mean squared errors, averages them over
// the batch rows and ranks the dims: the d - n_full with the smallest (error, index) are compressed.
__global__ void select_kernel(Dims s, float* __restrict__ sq, int n_mid, int32_t* idx_full_k, int32_t* idx_comp_k,
                              int32_t* idx_full_v, int32_t* idx_comp_v) {
    __shared__ float m_s[256];
    __shared__ int comp_s[256];
    const int h = blockIdx.x, side = blockIdx.y, e = threadIdx.x, d = s.d;
    const int n_full = side == 0 ? s.nfk : s.nfv;
    float mean = 0.f;
    if (e < d) {
        for (int b = 0; b < s.B; ++b) {
            float* p = sq + (((size_t)b * s.Hkv + h) * 2 + side) * d + e;
            const float v = n_mid > 0 ? *p / (float)n_mid : 0.f;
            *p = v;
            mean += v;
        }
        mean /= (float)s.B;
        m_s[e] = mean;
    }
    __syncthreads();
    if (e < d) {
        int rank = 0;
        for (int i = 0; i < d; ++i) rank += (m_s[i] < mean || (m_s[i] == mean && i < e)) ? 1 : 0;
        comp_s[e] = rank < d - n_full;
    }
    __syncthreads();
    if (e == 0) {
        int32_t* full = (side == 0 ? idx_full_k : idx_full_v) + (size_t)h * n_full;
        int32_t* comp = (side == 0 ? idx_comp_k : idx_comp_v) + (size_t)h * (d - n_full);
        int a = 0, c = 0;
        for (int i = 0; i < d; ++i) {
            if (comp_s[i]) comp[c++] = i;
            else full[a++] = i;
        }
    }
}

struct Scratch {
    fa_layout layout;
    fa_cache cache;
    float* sq;
    char* wc16;                 // weighted coefficients in bf16, the B operand of the tensor-core reconstruction
    char* ws_compress;
    size_t ws_compress_bytes;
    size_t total;
};

// Lays the scratch cache (everything compressed) and the error sums out in a workspace.
fa_status plan_scratch(const fa_layout& l, char* base, Scratch* out) {
    Scratch sc;
    std::memset(&sc, 0, sizeof(sc));
    sc.layout = l;
    sc.layout.n_full_k = 0;
    sc.layout.n_full_v = 0;
    fa_cache_sizes sz;
    fa_status st = fa_cache_sizes_of(&sc.layout, &sz);
    if (st != FA_OK) return st;
    size_t off = 0;
    auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off = align_up(off + bytes, 256); return p; };
    sc.cache.idx_comp_k = reinterpret_cast<const int32_t*>(take(sz.idx_comp_k));
    sc.cache.idx_comp_v = reinterpret_cast<const int32_t*>(take(sz.idx_comp_v));
    sc.cache.k_init = take(sz.k_init);
    sc.cache.v_init = take(sz.v_init);
    sc.cache.k_local = take(sz.k_local);
    sc.cache.v_local = take(sz.v_local);
    sc.cache.coef_k = reinterpret_cast<float*>(take(sz.coef_k));
    sc.cache.coef_v = reinterpret_cast<float*>(take(sz.coef_v));
    sc.cache.state = reinterpret_cast<int32_t*>(take(sz.state));
    sc.cache.status = reinterpret_cast<int32_t*>(take(sz.status));
    sc.sq = reinterpret_cast<float*>(take(sizeof(float) * (size_t)l.batch * l.n_kv_heads * 2 * l.head_dim));
    sc.wc16 = take(reconstruct_tc_scratch_bytes(make_dims(l)));
    size_t wsb = 0;
    st = fa_workspace_bytes(&sc.layout, &wsb);
    if (st != FA_OK) return st;
    sc.ws_compress = take(wsb);
    sc.ws_compress_bytes = wsb;
    sc.total = off;
    *out = sc;
    return FA_OK;
}

template <typename KV>
cudaError_t launch_mse(const Dims& s, const fa_cache& c, const void* K, const void* V, int64_t sb, int64_t st, int64_t sh,
                       int n_init, int n_mid, float* sq, cudaStream_t cs) {
    const dim3 grid((n_mid + kMseTokens - 1) / kMseTokens, s.Hkv * 2, s.B);
    const KV* k = static_cast<const KV*>(K);
    const KV* v = static_cast<const KV*>(V);
    switch (s.d) {
        case 64: mse_kernel<KV, 16><<<grid, 256, 0, cs>>>(s, c.coef_k, c.coef_v, k, v, sb, st, sh, n_init, n_mid, sq); break;
        case 128: mse_kernel<KV, 32><<<grid, 256, 0, cs>>>(s, c.coef_k, c.coef_v, k, v, sb, st, sh, n_init, n_mid, sq); break;
        case 256: mse_kernel<KV, 64><<<grid, 256, 0, cs>>>(s, c.coef_k, c.coef_v, k, v, sb, st, sh, n_init, n_mid, sq); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace
}  // namespace fa

using namespace fa;

extern "C" {

fa_status fa_select_workspace_bytes(const fa_layout* layout, size_t* out) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    if (!out) return FA_ERR_INVALID_ARG;
    if (layout->head_dim != 64 && layout->head_dim != 128 && layout->head_dim != 256) return FA_ERR_UNSUPPORTED;
    Scratch sc;
    st = plan_scratch(*layout, nullptr, &sc);
    if (st != FA_OK) return st;
    *out = sc.total;
    return FA_OK;
}

fa_status fa_select_dims(const fa_layout* layout, const void* K, const void* V, int64_t stride_b, int64_t stride_t,
                         int64_t stride_h, int32_t L, int32_t* idx_full_k, int32_t* idx_comp_k, int32_t* idx_full_v,
                         int32_t* idx_comp_v, float* mse, void* ws, size_t ws_bytes, void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    if (layout->head_dim != 64 && layout->head_dim != 128 && layout->head_dim != 256) return FA_ERR_UNSUPPORTED;
    if (L < 0 || (L > 0 && (!K || !V))) return FA_ERR_INVALID_ARG;
    if ((layout->n_full_k > 0 && !idx_full_k) || (layout->n_full_k < layout->head_dim && !idx_comp_k)) return FA_ERR_INVALID_ARG;
    if ((layout->n_full_v > 0 && !idx_full_v) || (layout->n_full_v < layout->head_dim && !idx_comp_v)) return FA_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return FA_ERR_WORKSPACE;
    Scratch sc;
    st = plan_scratch(*layout, static_cast<char*>(ws), &sc);
    if (st != FA_OK) return st;
    if (ws_bytes < sc.total) return FA_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const Dims s = make_dims(*layout);
    const int n_ids = s.Hkv * s.d;
    iota_rows_kernel<<<(n_ids + 255) / 256, 256, 0, cs>>>(const_cast<int32_t*>(sc.cache.idx_comp_k), s.Hkv, s.d);
    iota_rows_kernel<<<(n_ids + 255) / 256, 256, 0, cs>>>(const_cast<int32_t*>(sc.cache.idx_comp_v), s.Hkv, s.d);
    if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
    if (cudaMemsetAsync(sc.cache.status, 0, 16, cs) != cudaSuccess) return FA_ERR_CUDA;
    if (cudaMemsetAsync(sc.ws_compress, 0, sc.ws_compress_bytes < 4096 ? sc.ws_compress_bytes : 4096, cs) != cudaSuccess) return FA_ERR_CUDA;
    st = fa_compress(&sc.layout, &sc.cache, K, V, stride_b, stride_t, stride_h, L, sc.ws_compress, sc.ws_compress_bytes, stream);
    if (st != FA_OK) return st;
    const int n_init = L < s.l_init ? L : s.l_init;
    const int n_local = (L - n_init) < s.l_local ? (L - n_init) : s.l_local;
    const int n_mid = L - n_init - n_local;
    const size_t sq_bytes = sizeof(float) * (size_t)s.B * s.Hkv * 2 * s.d;
    if (cudaMemsetAsync(sc.sq, 0, sq_bytes, cs) != cudaSuccess) return FA_ERR_CUDA;
    if (n_mid > 0 && reconstruct_tc_supported(s, layout->kv_dtype, K, V, stride_b, stride_t, stride_h, n_mid)) {
        if (launch_reconstruct_tc(s, sc.cache.coef_k, sc.cache.coef_v, K, V, stride_b, stride_t, stride_h, n_init, n_mid, sc.sq,
                                  sc.cache.status, sc.wc16, cs) != cudaSuccess)
            return FA_ERR_CUDA;
    } else if (n_mid > 0) {
        cudaError_t err = layout->kv_dtype == FA_BF16
                              ? launch_mse<__nv_bfloat16>(s, sc.cache, K, V, stride_b, stride_t, stride_h, n_init, n_mid, sc.sq, cs)
                              : launch_mse<float>(s, sc.cache, K, V, stride_b, stride_t, stride_h, n_init, n_mid, sc.sq, cs);
        if (err != cudaSuccess) return FA_ERR_CUDA;
    }
    select_kernel<<<dim3(s.Hkv, 2), 256, 0, cs>>>(s, sc.sq, n_mid, idx_full_k, idx_comp_k, idx_full_v, idx_comp_v);
    if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
    if (mse && cudaMemcpyAsync(mse, sc.sq, sq_bytes, cudaMemcpyDeviceToDevice, cs) != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

}  // extern "C"
