// fa_append (Eq.5): push one token; when the local window is full its oldest
// row leaves, its kept dims join K^mu / V^mu and its compressed dims are added
// to every coefficient row with basis column j = n_mid.  One kernel:
//   grid (row tiles, Hkv, B).  Each CTA updates its rows of C^K and C^V;
//   CTA x == 0 also writes the leaving row's kept dims to the middle.  The last
//   CTA of a batch row to finish (atomic ticket, no waiting) overwrites the
//   ring slot with the new token and advances the counters, so no CTA can see
//   a half-updated state.
#include "fa_common.cuh"

namespace fa {

constexpr int kAppendRows = 64;   // coefficient rows per CTA

template <typename KV>
__global__ void __launch_bounds__(256) append_kernel(Dims s, CacheDev c, const KV* __restrict__ k_new,
                                                     const KV* __restrict__ v_new) {
    __shared__ float x_s[2][256];        // the row that leaves (or is stored), both sides, natural dim order
    __shared__ int last_s;
    const int h = blockIdx.y, b = blockIdx.z;
    const int n_init = c.state[kStateStride * b + 0], n_local = c.state[kStateStride * b + 1], n_mid = c.state[kStateStride * b + 2];
    const int head = c.state[kStateStride * b + 3];
    const bool to_init = n_init < s.l_init;
    const bool evict = !to_init && n_local == s.l_local;
    const bool full = evict && (n_mid >= s.max_mid || n_mid >= s.T);
    if (full) {
        if (threadIdx.x == 0 && blockIdx.x == 0 && h == 0) atomicExch(c.status, (int)FA_ERR_CAPACITY);
        return;                          // every CTA of this batch row takes the same exit
    }
    if (evict) {
        // the row that leaves: oldest ring row, or the new token itself if there is no local window
        for (int i = threadIdx.x; i < 2 * s.d; i += blockDim.x) {
            int side = i / s.d, e = i - side * s.d;
            float v;
            if (s.l_local == 0) {
                v = ld_f((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + h) * s.d + e);
            } else {
                v = ld_f(win_row<KV>(side == 0 ? c.k_local : c.v_local, s, b, h, s.l_local, head) + e);
            }
            x_s[side][e] = v;
        }
        __syncthreads();
        const int j = n_mid;
        if (blockIdx.x == 0) {
            for (int i = threadIdx.x; i < s.nfk + s.nfv; i += blockDim.x) {
                int side = i < s.nfk ? 0 : 1;
                int e = side == 0 ? i : i - s.nfk;
                int nfull = side == 0 ? s.nfk : s.nfv;
                const int32_t* idf = (side == 0 ? c.idx_full_k : c.idx_full_v) + (size_t)h * nfull;
                KV* dst = mid_row<KV>(side == 0 ? c.k_mid : c.v_mid, s, b, h, j % s.P, j / s.P, nfull);
                st_f(dst + e, x_s[side][idf[e]]);
            }
        }
        // coefficient rows [m0, m1) of both sides
        const int m0 = blockIdx.x * kAppendRows;
        const int m1 = min(s.M, m0 + kAppendRows);
        for (int side = 0; side < 2; ++side) {
            int nfull = side == 0 ? s.nfk : s.nfv;
            int ncomp = s.d - nfull;
            if (ncomp == 0) continue;
            const int32_t* idc = (side == 0 ? c.idx_comp_k : c.idx_comp_v) + (size_t)h * ncomp;
            float* coef = coef_rows(side == 0 ? c.coef_k : c.coef_v, s, b, h, ncomp);
            int vec_per_row = ncomp >> 2;                   // ncomp is a multiple of 8
            int total = (m1 - m0) * vec_per_row;
            for (int i = threadIdx.x; i < total; i += blockDim.x) {
                int r = i / vec_per_row, v4 = i - r * vec_per_row;
                int m = m0 + r;
                float cs, sn;
                basis_cs(m >> 1, j, s.T, &cs, &sn);
                float f = (m & 1) ? sn : cs;
                float4* p = reinterpret_cast<float4*>(coef + (size_t)m * ncomp) + v4;
                float4 cur = *p;
                int e = 4 * v4;
                cur.x = fmaf(f, x_s[side][idc[e + 0]], cur.x);
                cur.y = fmaf(f, x_s[side][idc[e + 1]], cur.y);
                cur.z = fmaf(f, x_s[side][idc[e + 2]], cur.z);
                cur.w = fmaf(f, x_s[side][idc[e + 3]], cur.w);
                *p = cur;
            }
        }
    }
    // ticket: the last CTA of this batch row stores the new token and advances the counters
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        int done = atomicAdd(c.state + kStateStride * b + 4, 1);
        last_s = (done == (int)(gridDim.x * gridDim.y) - 1);
    }
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    for (int i = threadIdx.x; i < 2 * s.Hkv * s.d; i += blockDim.x) {
        int side = i / (s.Hkv * s.d);
        int rem = i - side * (s.Hkv * s.d);
        int hh = rem / s.d, e = rem - hh * s.d;
        const KV* src = (side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + hh) * s.d;
        if (to_init) {
            win_row<KV>(side == 0 ? c.k_init : c.v_init, s, b, hh, s.l_init, n_init)[e] = src[e];
        } else if (s.l_local > 0) {
            int slot = evict ? head : (head + n_local) % s.l_local;
            win_row<KV>(side == 0 ? c.k_local : c.v_local, s, b, hh, s.l_local, slot)[e] = src[e];
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (to_init) c.state[kStateStride * b + 0] = n_init + 1;
        else if (evict) {
            c.state[kStateStride * b + 2] = n_mid + 1;
            if (s.l_local > 0) c.state[kStateStride * b + 3] = (head + 1) % s.l_local;
        } else c.state[kStateStride * b + 1] = n_local + 1;
        c.state[kStateStride * b + 4] = 0;        // ticket counter ready for the next call
    }
}

template <typename KV>
static cudaError_t launch_append_t(const Dims& s, const CacheDev& c, const void* k_new, const void* v_new,
                                   cudaStream_t st) {
    int tiles = (s.M + kAppendRows - 1) / kAppendRows;
    append_kernel<KV><<<dim3(tiles, s.Hkv, s.B), 256, 0, st>>>(s, c, static_cast<const KV*>(k_new),
                                                               static_cast<const KV*>(v_new));
    return cudaGetLastError();
}

cudaError_t launch_append(const Dims& s, const CacheDev& c, int dtype, const void* k_new, const void* v_new,
                          cudaStream_t st) {
    if (dtype == FA_BF16) return launch_append_t<__nv_bfloat16>(s, c, k_new, v_new, st);
    return launch_append_t<float>(s, c, k_new, v_new, st);
}

}  // namespace fa
