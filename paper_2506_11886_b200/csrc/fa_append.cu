// fa_append (Eq.5): push one token; when the local window is full its oldest
// row leaves, its kept dims join K^mu / V^mu and its compressed dims are added
// to every coefficient row with basis column j = n_mid.  One kernel:
//   grid (row tiles, Hkv, B).  Each CTA updates kAppendRows rows of C^K and C^V
//   (every float4 read-modify-write independent of the others, all loads issued
//   before the first store); CTA x == 0 also writes the leaving row's kept dims
//   to the middle.  The last CTA of a batch row to finish (atomic ticket, no
//   waiting) overwrites the ring slot with the new token and advances the
//   counters, so no CTA can see a half-updated state.
#include "fa_common.cuh"
#include "fa_decode_ws.cuh"

namespace fa {

constexpr int kAppendRows = 32;   // coefficient rows per CTA (halved when more than 128 dims are compressed)
constexpr int kAppendVec = 4;     // float4 read-modify-writes per thread and side (dims <= 128 compressed)

template <typename KV>
__global__ void __launch_bounds__(256) append_kernel(Dims s, CacheDev c, const KV* __restrict__ k_new,
                                                     const KV* __restrict__ v_new, int rows_per_cta) {
    __shared__ float x_s[2][256];        // the row that leaves, both sides, natural dim order
    __shared__ __align__(16) float xc_s[2][256];   // the same gathered at D^kc / D^vc
    __shared__ float f_s[kAppendRows];   // basis column j for the rows of this CTA
    __shared__ int last_s;
    const int h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
    // programmatic dependent launch: the next kernel may be scheduled now; this one first waits for
    // everything its predecessor in the stream wrote
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int n_init = c.state[kStateStride * b + 0], n_local = c.state[kStateStride * b + 1];
    const int n_mid = c.state[kStateStride * b + 2], head = c.state[kStateStride * b + 3];
    const bool to_init = n_init < s.l_init;
    const bool evict = !to_init && n_local == s.l_local;
    const bool full = evict && (n_mid >= s.max_mid || n_mid >= s.T);
    if (full) {
        if (tid == 0 && blockIdx.x == 0 && h == 0) atomicExch(c.status, (int)FA_ERR_CAPACITY);
        return;                          // every CTA of this batch row takes the same exit
    }
    if (evict) {
        const int j = n_mid;
        const int m0 = blockIdx.x * rows_per_cta;
        const int rows = min(rows_per_cta, s.M - m0);
        // start the coefficient loads first: they do not depend on anything computed here
        float4 cur[2][kAppendVec];
        float4* ptr[2][kAppendVec];
#pragma unroll
        for (int side = 0; side < 2; ++side) {
            const int ncomp = side == 0 ? s.dck : s.dcv;
            const int vpr = ncomp >> 2;
            float* coef = ncomp ? coef_rows(side == 0 ? c.coef_k : c.coef_v, s, b, h, ncomp) + (size_t)m0 * ncomp : nullptr;
#pragma unroll
            for (int u = 0; u < kAppendVec; ++u) {
                const int i = tid + 256 * u;
                ptr[side][u] = (ncomp && i < rows * vpr) ? reinterpret_cast<float4*>(coef) + i : nullptr;
                if (ptr[side][u]) cur[side][u] = *ptr[side][u];
            }
        }
        // the row that leaves: oldest ring row, or the new token itself if there is no local window
        for (int i = tid; i < 2 * s.d; i += 256) {
            const int side = i / s.d, e = i - side * s.d;
            float v;
            if (s.l_local == 0) v = ld_f((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + h) * s.d + e);
            else v = ld_f(win_row<KV>(side == 0 ? c.k_local : c.v_local, s, b, h, s.l_local, head) + e);
            x_s[side][e] = v;
        }
        if (tid < rows) {
            float cs, sn;
            const int m = m0 + tid;
            basis_cs(m >> 1, j, s.T, &cs, &sn);
            f_s[tid] = (m & 1) ? sn : cs;
        }
        __syncthreads();
        for (int i = tid; i < s.dck + s.dcv; i += 256) {
            const int side = i < s.dck ? 0 : 1;
            const int e = side == 0 ? i : i - s.dck;
            const int32_t* idc = side == 0 ? c.idx_comp_k + (size_t)h * s.dck : c.idx_comp_v + (size_t)h * s.dcv;
            xc_s[side][e] = x_s[side][idc[e]];
        }
        if (blockIdx.x == 0) {
            for (int i = tid; i < s.nfk + s.nfv; i += 256) {
                const int side = i < s.nfk ? 0 : 1;
                const int e = side == 0 ? i : i - s.nfk;
                const int nfull = side == 0 ? s.nfk : s.nfv;
                const int32_t* idf = (side == 0 ? c.idx_full_k : c.idx_full_v) + (size_t)h * nfull;
                KV* dst = mid_row<KV>(side == 0 ? c.k_mid : c.v_mid, s, b, h, j % s.P, j / s.P, nfull);
                const int col = side == 1 ? v_mid_col(j / s.P, e, nfull, sizeof(KV) == 2 ? FA_BF16 : FA_F32) : e;
                st_f(dst + col, x_s[side][idf[e]]);
            }
        }
        __syncthreads();
#pragma unroll
        for (int side = 0; side < 2; ++side) {
            const int ncomp = side == 0 ? s.dck : s.dcv;
            const int vpr = ncomp >> 2;
#pragma unroll
            for (int u = 0; u < kAppendVec; ++u) {
                if (!ptr[side][u]) continue;
                const int i = tid + 256 * u;
                const int r = i / vpr, v4 = i - r * vpr;
                const float f = f_s[r];
                const float4 x = *reinterpret_cast<const float4*>(&xc_s[side][4 * v4]);
                float4 o = cur[side][u];
                o.x = fmaf(f, x.x, o.x);
                o.y = fmaf(f, x.y, o.y);
                o.z = fmaf(f, x.z, o.z);
                o.w = fmaf(f, x.w, o.w);
                *ptr[side][u] = o;
            }
        }
    }
    // ticket: the last CTA of this batch row stores the new token and advances the counters
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int done = atomicAdd(c.state + kStateStride * b + 4, 1);
        last_s = (done == (int)(gridDim.x * gridDim.y) - 1);
    }
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    for (int i = tid; i < 2 * s.Hkv * s.d; i += 256) {
        const int side = i / (s.Hkv * s.d);
        const int rem = i - side * (s.Hkv * s.d);
        const int hh = rem / s.d, e = rem - hh * s.d;
        const KV* src = (side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + hh) * s.d;
        if (to_init) {
            win_row<KV>(side == 0 ? c.k_init : c.v_init, s, b, hh, s.l_init, n_init)[e] = src[e];
        } else if (s.l_local > 0) {
            const int slot = evict ? head : (head + n_local) % s.l_local;
            win_row<KV>(side == 0 ? c.k_local : c.v_local, s, b, hh, s.l_local, slot)[e] = src[e];
        }
    }
    __syncthreads();
    if (tid == 0) {
        if (to_init) c.state[kStateStride * b + 0] = n_init + 1;
        else if (evict) {
            c.state[kStateStride * b + 2] = n_mid + 1;
            if (s.l_local > 0) c.state[kStateStride * b + 3] = (head + 1) % s.l_local;
        } else c.state[kStateStride * b + 1] = n_local + 1;
        c.state[kStateStride * b + 4] = 0;        // ticket counter ready for the next call
    }
}

// First half of a fused decode step (Eq.5 without the coefficient update): one CTA per (batch row, KV head) moves
// the row that leaves the local window (kept dims to K^mu / V^mu), stores the new token and advances
// the counters, and leaves the compressed dims of the leaving row with its basis column j in the
// workspace.  The decode kernel of the same step adds f_j x^T to the coefficient rows as it streams
// them, so the coefficients are read and written once per step instead of twice.
template <typename KV>
__global__ void __launch_bounds__(256) append_lite_kernel(Dims s, CacheDev c, DecodePlan p, const KV* __restrict__ k_new,
                                                          const KV* __restrict__ v_new, char* wsp) {
    __shared__ float x_s[2][256];        // the row that leaves, both sides, natural dim order
    __shared__ int last_s;
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    // wait for everything before this kernel, THEN let the decode kernel of the step start: it reads
    // coefficient rows before its own wait, and nothing but this kernel may still be running then
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    Ws ws = ws_view(wsp, p);
    const int n_init = c.state[kStateStride * b + 0], n_local = c.state[kStateStride * b + 1];
    const int n_mid = c.state[kStateStride * b + 2], head = c.state[kStateStride * b + 3];
    const bool to_init = n_init < s.l_init;
    const bool evict = !to_init && n_local == s.l_local;
    const bool full = evict && (n_mid >= s.max_mid || n_mid >= s.T);
    if (full) {
        if (tid == 0 && h == 0) { atomicExch(c.status, (int)FA_ERR_CAPACITY); ws.pend_j[b] = -1; }
        return;                          // every CTA of this batch row takes the same exit
    }
    // the new token of this head (up to two elements per thread), loaded together with the leaving row
    KV new_e[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int i = tid + 256 * u;
        if (i < 2 * s.d) {
            const int side = i / s.d, e = i - side * s.d;
            new_e[u] = ((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + h) * s.d)[e];
        }
    }
    if (evict) {
        const int j = n_mid;
        for (int i = tid; i < 2 * s.d; i += 256) {
            const int side = i / s.d, e = i - side * s.d;
            float v;
            if (s.l_local == 0) v = ld_f((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + h) * s.d + e);
            else v = ld_f(win_row<KV>(side == 0 ? c.k_local : c.v_local, s, b, h, s.l_local, head) + e);
            x_s[side][e] = v;
        }
        __syncthreads();
        for (int i = tid; i < s.nfk + s.nfv; i += 256) {
            const int side = i < s.nfk ? 0 : 1;
            const int e = side == 0 ? i : i - s.nfk;
            const int nfull = side == 0 ? s.nfk : s.nfv;
            const int32_t* idf = (side == 0 ? c.idx_full_k : c.idx_full_v) + (size_t)h * nfull;
            KV* dst = mid_row<KV>(side == 0 ? c.k_mid : c.v_mid, s, b, h, j % s.P, j / s.P, nfull);
            const int col = side == 1 ? v_mid_col(j / s.P, e, nfull, sizeof(KV) == 2 ? FA_BF16 : FA_F32) : e;
            st_f(dst + col, x_s[side][idf[e]]);
        }
        float* pend = ws.pend + ((size_t)b * s.Hkv + h) * (s.dck + s.dcv);
        for (int i = tid; i < s.dck + s.dcv; i += 256) {
            const int side = i < s.dck ? 0 : 1;
            const int e = side == 0 ? i : i - s.dck;
            const int32_t* idc = side == 0 ? c.idx_comp_k + (size_t)h * s.dck : c.idx_comp_v + (size_t)h * s.dcv;
            pend[i] = x_s[side][idc[e]];
        }
    }
    // the new token of this head: next init row, or the ring slot behind the newest local row (the slot
    // just read and vacated when the window is full)
    if (evict) __syncthreads();          // every thread has read the slot that is overwritten next
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int i = tid + 256 * u;
        if (i >= 2 * s.d) continue;
        const int side = i / s.d, e = i - side * s.d;
        if (to_init) {
            win_row<KV>(side == 0 ? c.k_init : c.v_init, s, b, h, s.l_init, n_init)[e] = new_e[u];
        } else if (s.l_local > 0) {
            const int slot = evict ? head : (head + n_local) % s.l_local;
            win_row<KV>(side == 0 ? c.k_local : c.v_local, s, b, h, s.l_local, slot)[e] = new_e[u];
        }
    }
    // ticket: the last head of this batch row to finish advances the counters (nobody reads them after this point)
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const int done = atomicAdd(c.state + kStateStride * b + 4, 1);
        last_s = (done == (int)gridDim.x - 1);
    }
    __syncthreads();
    if (!last_s || tid != 0) return;
    if (to_init) c.state[kStateStride * b + 0] = n_init + 1;
    else if (evict) {
        c.state[kStateStride * b + 2] = n_mid + 1;
        if (s.l_local > 0) c.state[kStateStride * b + 3] = (head + 1) % s.l_local;
    } else c.state[kStateStride * b + 1] = n_local + 1;
    c.state[kStateStride * b + 4] = 0;            // ticket counter ready for the next call
    ws.pend_j[b] = evict ? n_mid : -1;
}

template <typename KV>
static cudaError_t launch_append_t(const Dims& s, const CacheDev& c, const void* k_new, const void* v_new,
                                   cudaStream_t st) {
    const int max_comp = s.dck > s.dcv ? s.dck : s.dcv;
    const int rows = max_comp > 128 ? kAppendRows / 2 : kAppendRows;     // rows * max_comp / 4 <= 256 * kAppendVec
    const int tiles = (s.M + rows - 1) / rows;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles, s.Hkv, s.B);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, append_kernel<KV>, s, c, static_cast<const KV*>(k_new), static_cast<const KV*>(v_new), rows);
}

template <typename KV>
static cudaError_t launch_append_lite_t(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* k_new, const void* v_new,
                                        char* ws, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(s.Hkv, s.B);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, append_lite_kernel<KV>, s, c, p, static_cast<const KV*>(k_new), static_cast<const KV*>(v_new), ws);
}

cudaError_t launch_append_lite(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, const void* k_new, const void* v_new,
                               char* ws, cudaStream_t st) {
    if (dtype == FA_BF16) return launch_append_lite_t<__nv_bfloat16>(s, c, p, k_new, v_new, ws, st);
    return launch_append_lite_t<float>(s, c, p, k_new, v_new, ws, st);
}

cudaError_t launch_append(const Dims& s, const CacheDev& c, int dtype, const void* k_new, const void* v_new,
                          cudaStream_t st) {
    if (dtype == FA_BF16) return launch_append_t<__nv_bfloat16>(s, c, k_new, v_new, st);
    return launch_append_t<float>(s, c, k_new, v_new, st);
}

}  // namespace fa
