// fa_decode_attention (Eq.6 re-associated), the two small-side products around the token loop:
//   prologue   u_g[m] = scale * log2(e) * w_m * sum_e C^K[m][e] q_g[D^kc[e]]
//   epilogue   merge the token splits, o^c[e] = sum_m w_m z[m] C^V[m][e], normalise, scatter.
// Both read their coefficient matrix exactly once; each CTA brings a tile of rows into shared
// memory with 16-byte asynchronous copies (all in flight together) and works from there.  All
// loads of partial results are issued in independent batches so that a call costs a few memory
// round trips, not one per split.  The three kernels of a decode call are chained with
// programmatic dependent launch: each lets its successor start at once, and the successor waits
// (griddepcontrol.wait) only where it first touches what its predecessor wrote.
#include "fa_common.cuh"
#include "fa_decode_ws.cuh"

namespace fa {

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- prologue --
// grid (ceil(M / rows_pro), Hkv, B), 256 threads.
template <typename KV>
__global__ void __launch_bounds__(256) decode_prologue_kernel(Dims s, CacheDev c, DecodePlan p, const KV* __restrict__ q,
                                                              char* wsp) {
    extern __shared__ __align__(16) float sm_pro[];
    pdl_launch_dependents();
    Ws ws = ws_view(wsp, p);
    const int h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
    if (blockIdx.x == 0 && tid == 0) ws.cnt[b * s.Hkv + h] = 0;
    if (s.dck == 0) return;
    const int stride = s.dck + 4;                      // row stride of the tile: 16-byte aligned, bank-skewed
    const int qstride = s.dck + 1;
    float* tile = sm_pro;                              // [rows_pro][stride]
    float* qc_s = tile + p.rows_pro * stride;          // [G][qstride] gathered query
    const int m0 = blockIdx.x * p.rows_pro;
    const int rows = min(p.rows_pro, s.M - m0);
    const float* coef = coef_rows(c.coef_k, s, b, h, s.dck) + (size_t)m0 * s.dck;
    const int vpr = s.dck >> 2;
    for (int i = tid; i < rows * vpr; i += 256) {
        int r = i / vpr, v4 = i - r * vpr;
        cp_async16(tile + r * stride + 4 * v4, coef + (size_t)r * s.dck + 4 * v4);
    }
    const int32_t* idc = c.idx_comp_k + (size_t)h * s.dck;
    for (int i = tid; i < s.G * s.dck; i += 256) {
        int g = i / s.dck, e = i - g * s.dck;
        qc_s[g * qstride + e] = ld_f(q + ((size_t)b * s.Hq + h * s.G + g) * s.d + idc[e]);
    }
    cp_async_wait_all();
    __syncthreads();
    for (int t = tid; t < rows * s.G; t += 256) {
        const int g = t % s.G, r = t / s.G;
        const float* row = tile + r * stride;
        const float* qq = qc_s + g * qstride;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        for (int e = 0; e < s.dck; e += 4) {
            a0 = fmaf(row[e], qq[e], a0);
            a1 = fmaf(row[e + 1], qq[e + 1], a1);
            a2 = fmaf(row[e + 2], qq[e + 2], a2);
            a3 = fmaf(row[e + 3], qq[e + 3], a3);
        }
        const int m = m0 + r;
        ws.u[((size_t)b * s.Hq + h * s.G + g) * s.M + m] =
            recon_weight(s.norm, m, s.k, s.T) * s.scale * kLog2e * ((a0 + a1) + (a2 + a3));
    }
}

// ---------------------------------------------------------------- epilogue --
// grid (n_slice, Hkv, B), 256 threads.  Each CTA merges the split statistics of its KV head,
// forms the weighted z of its slice of coefficient rows and multiplies by those rows of C^V;
// the last CTA of a (b, h) to finish (atomic ticket, nobody waits) adds the slices in a fixed
// order, normalises and writes the output rows.
template <typename KV>
__global__ void __launch_bounds__(256) decode_epilogue_kernel(Dims s, CacheDev c, DecodePlan p, KV* __restrict__ out,
                                                              char* wsp) {
    extern __shared__ __align__(16) float sm_epi[];
    __shared__ int last_s;
    Ws ws = ws_view(wsp, p);
    const int slice = blockIdx.x, h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
    const int rows_max = (s.M + p.n_slice - 1) / p.n_slice;
    const int m0 = slice * rows_max;
    const int rows = max(0, min(rows_max, s.M - m0));
    const int stride = s.dcv + 4;
    const int ns = p.n_part;
    float* alpha_s = sm_epi;                               // [G][n_split]: first the maxima, then exp2(m - max)
    float* l_s = alpha_s + s.G * ns;                       // [G][n_split]
    float* linv_s = l_s + s.G * ns;                        // [G]
    float* zw_s = linv_s + s.G;                            // [G][rows_max]
    int* inv_s = reinterpret_cast<int*>(zw_s + s.G * rows_max);   // [d] dim -> slot in D^vc, or -1
    float* tile = reinterpret_cast<float*>(inv_s + s.d);   // [rows_max][stride]
    tile = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(tile) + 15) & ~uintptr_t(15));

    // the coefficient tile does not depend on the main kernel: start it before waiting for it
    if (s.dcv > 0) {
        const float* cv = coef_rows(c.coef_v, s, b, h, s.dcv) + (size_t)m0 * s.dcv;
        const int vpr = s.dcv >> 2;
        for (int i = tid; i < rows * vpr; i += 256) {
            int r = i / vpr, v4 = i - r * vpr;
            cp_async16(tile + r * stride + 4 * v4, cv + (size_t)r * s.dcv + 4 * v4);
        }
    }
    for (int e = tid; e < s.d; e += 256) inv_s[e] = -1;
    pdl_wait();                                            // partial results of the main kernel are complete

    // split statistics: one (head, split) pair per thread, then a tiny reduction per head
    for (int i = tid; i < s.G * ns; i += 256) {
        const int g = i / ns, sp = i - g * ns;
        const float2 ml = *reinterpret_cast<const float2*>(ws.ml + (((size_t)b * s.Hq + h * s.G + g) * ns + sp) * 2);
        alpha_s[i] = ml.x;
        l_s[i] = ml.y;
    }
    __syncthreads();
    if (tid < s.G) {
        float mx = kNegBig;
        for (int sp = 0; sp < ns; ++sp) mx = fmaxf(mx, alpha_s[tid * ns + sp]);
        float L = 0.f;
        for (int sp = 0; sp < ns; ++sp) {
            const float a = exp2f(alpha_s[tid * ns + sp] - mx);
            alpha_s[tid * ns + sp] = a;
            L = fmaf(a, l_s[tid * ns + sp], L);
        }
        linv_s[tid] = L > 0.f ? 1.0f / L : 0.f;
    }
    __syncthreads();
    if (s.dcv > 0) {
        for (int t = tid; t < s.G * rows; t += 256) {
            const int g = t / rows, r = t - g * rows;
            const float* z = ws.z + ((size_t)b * s.Hq + h * s.G + g) * ns * s.M + m0 + r;
            const float* al = alpha_s + g * ns;
            float v0 = 0.f, v1 = 0.f;
            int sp = 0;
            for (; sp + 8 <= ns; sp += 8) {                // eight independent loads in flight
                float zz[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) zz[i] = z[(size_t)(sp + i) * s.M];
#pragma unroll
                for (int i = 0; i < 8; i += 2) { v0 = fmaf(al[sp + i], zz[i], v0); v1 = fmaf(al[sp + i + 1], zz[i + 1], v1); }
            }
            for (; sp < ns; ++sp) v0 = fmaf(al[sp], z[(size_t)sp * s.M], v0);
            zw_s[g * rows_max + r] = (v0 + v1) * recon_weight(s.norm, m0 + r, s.k, s.T);
        }
        cp_async_wait_all();
        __syncthreads();
        for (int t = tid; t < s.G * s.dcv; t += 256) {
            const int g = t / s.dcv, e = t - g * s.dcv;
            const float* zw = zw_s + g * rows_max;
            float a0 = 0.f, a1 = 0.f;
            int r = 0;
            for (; r + 2 <= rows; r += 2) {
                a0 = fmaf(zw[r], tile[r * stride + e], a0);
                a1 = fmaf(zw[r + 1], tile[(r + 1) * stride + e], a1);
            }
            if (r < rows) a0 = fmaf(zw[r], tile[r * stride + e], a0);
            ws.oc[(((size_t)b * s.Hq + h * s.G + g) * p.n_slice + slice) * s.dcv + e] = a0 + a1;
        }
    }
    // ticket
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int done = atomicAdd(ws.cnt + b * s.Hkv + h, 1);
        last_s = (done == (int)gridDim.x - 1);
    }
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    const int32_t* idc_v = c.idx_comp_v + (size_t)h * s.dcv;
    for (int e = tid; e < s.dcv; e += 256) inv_s[idc_v[e]] = e;
    __syncthreads();
    for (int t = tid; t < s.G * s.d; t += 256) {
        const int g = t / s.d, e = t - g * s.d;
        const size_t qh = (size_t)b * s.Hq + h * s.G + g;
        const float* al = alpha_s + g * ns;
        const float* o = ws.o + qh * ns * s.d + e;
        float v0 = 0.f, v1 = 0.f;
        int sp = 0;
        for (; sp + 8 <= ns; sp += 8) {
            float oo[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) oo[i] = o[(size_t)(sp + i) * s.d];
#pragma unroll
            for (int i = 0; i < 8; i += 2) { v0 = fmaf(al[sp + i], oo[i], v0); v1 = fmaf(al[sp + i + 1], oo[i + 1], v1); }
        }
        for (; sp < ns; ++sp) v0 = fmaf(al[sp], o[(size_t)sp * s.d], v0);
        const int slot = inv_s[e];
        if (slot >= 0) {
            const float* oc = ws.oc + qh * p.n_slice * s.dcv + slot;
            float w0 = 0.f, w1 = 0.f;
            int sl = 0;
            for (; sl + 8 <= p.n_slice; sl += 8) {
                float cc[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) cc[i] = __ldcg(oc + (size_t)(sl + i) * s.dcv);
#pragma unroll
                for (int i = 0; i < 8; i += 2) { w0 += cc[i]; w1 += cc[i + 1]; }
            }
            for (; sl < p.n_slice; ++sl) w0 += __ldcg(oc + (size_t)sl * s.dcv);
            v0 += w0;
            v1 += w1;
        }
        st_f(out + qh * s.d + e, (v0 + v1) * linv_s[g]);
    }
}

// ---------------------------------------------------------------- launchers --
// Launch with the programmatic-stream-serialization attribute: the kernel may start while its
// predecessor in the stream still runs; it synchronises with griddepcontrol.wait.
template <typename... Params, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

template <typename KV>
static cudaError_t launch_prologue_t(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* q, char* ws,
                                     cudaStream_t st) {
    const int tiles = s.dck > 0 ? (s.M + p.rows_pro - 1) / p.rows_pro : 1;
    const size_t smem = sizeof(float) * ((size_t)p.rows_pro * (s.dck + 4) + (size_t)s.G * (s.dck + 1));
    cudaError_t err = ensure_dynamic_smem(decode_prologue_kernel<KV>, smem);
    if (err != cudaSuccess) return err;
    decode_prologue_kernel<KV><<<dim3(tiles, s.Hkv, s.B), 256, smem, st>>>(s, c, p, static_cast<const KV*>(q), ws);
    return cudaGetLastError();
}

cudaError_t launch_decode_prologue(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, const void* q,
                                   char* ws, cudaStream_t st) {
    if (dtype == FA_BF16) return launch_prologue_t<__nv_bfloat16>(s, c, p, q, ws, st);
    return launch_prologue_t<float>(s, c, p, q, ws, st);
}

template <typename KV>
static cudaError_t launch_epilogue_t(const Dims& s, const CacheDev& c, const DecodePlan& p, void* out, char* ws,
                                     cudaStream_t st) {
    const int rows = (s.M + p.n_slice - 1) / p.n_slice;
    const size_t smem = sizeof(float) * (2 * (size_t)s.G * p.n_part + s.G + (size_t)s.G * rows + s.d + 4 + (size_t)rows * (s.dcv + 4));
    cudaError_t err = ensure_dynamic_smem(decode_epilogue_kernel<KV>, smem);
    if (err != cudaSuccess) return err;
    return launch_pdl(decode_epilogue_kernel<KV>, dim3(p.n_slice, s.Hkv, s.B), dim3(256), smem, st, true, s, c, p,
                      static_cast<KV*>(out), ws);
}

cudaError_t launch_decode_epilogue(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, void* out, char* ws,
                                   cudaStream_t st) {
    if (dtype == FA_BF16) return launch_epilogue_t<__nv_bfloat16>(s, c, p, out, ws, st);
    return launch_epilogue_t<float>(s, c, p, out, ws, st);
}

}  // namespace fa
