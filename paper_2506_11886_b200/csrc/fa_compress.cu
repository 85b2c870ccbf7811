// fa_compress, CUDA-core path (Eq.1-4): partition + gather, then the
// projection C = F X^mn as an fp32 tile product with the basis generated on
// the fly.  Serves fp32 caches and is the fallback of the tensor-core path.
#include "fa_common.cuh"

namespace fa {

// ---- index-set check (Eq.2: D^u and D^c partition the head dims) ------------
__global__ void validate_kernel(Dims s, CacheDev c) {
    int h = blockIdx.x;
    int side = blockIdx.y;
    __shared__ int seen[256];
    __shared__ int bad;
    int nfull = side == 0 ? s.nfk : s.nfv;
    int ncomp = s.d - nfull;
    const int32_t* idf = (side == 0 ? c.idx_full_k : c.idx_full_v) + (size_t)h * nfull;
    const int32_t* idc = (side == 0 ? c.idx_comp_k : c.idx_comp_v) + (size_t)h * ncomp;
    for (int i = threadIdx.x; i < s.d; i += blockDim.x) seen[i] = 0;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < s.d; i += blockDim.x) {
        bool full = i < nfull;
        const int32_t* a = full ? idf : idc;
        int pos = full ? i : i - nfull;
        int v = a[pos];
        if (v < 0 || v >= s.d) { atomicExch(&bad, 1); continue; }
        if (pos > 0 && a[pos - 1] >= v) atomicExch(&bad, 1);
        atomicAdd(&seen[v], 1);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < s.d; i += blockDim.x)
        if (seen[i] != 1) atomicExch(&bad, 1);
    __syncthreads();
    if (threadIdx.x == 0 && bad) atomicExch(c.status, (int)FA_ERR_INDEX);
}

cudaError_t launch_validate(const Dims& s, const CacheDev& c, cudaStream_t st) {
    validate_kernel<<<dim3(s.Hkv, 2), 128, 0, st>>>(s, c);
    return cudaGetLastError();
}

// ---- Eq.1-2: windows, kept dims, counters -----------------------------------
// grid (chunks of 64 tokens, Hkv, B * 2 sides).  Every row of the input, of the windows and of the
// kept-dim rows starts on a 16-byte boundary and is a whole number of 16-byte chunks (the C ABI asks
// for 16-byte aligned K, V and strides that are multiples of 8 elements; head_dim and the kept-dim
// counts are multiples of 8).  The CTA stages its 64 input rows in shared memory with one 16-byte load
// per chunk, then one thread per output chunk either copies it (window rows) or gathers its dims
// through the index set (kept-dim rows; for V^mu of bf16 caches the chunk it writes is the permuted one).
constexpr int kRowsPerCta = 64;

template <typename KV>
__global__ void __launch_bounds__(256) partition_gather_kernel(Dims s, CacheDev c, const KV* __restrict__ K,
                                                                   const KV* __restrict__ V, int64_t sb, int64_t st,
                                                                   int64_t sh, int L, int mid_rows, int skip_a, int skip_c, int zero_coef) {
    constexpr int EPC = 16 / (int)sizeof(KV);            // elements per chunk
    extern __shared__ __align__(16) unsigned char gsm[];
    // the contraction kernel behind this one may start at once (programmatic dependent launch): it waits for this
    // grid only in front of its reductions into the coefficients cleared here
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    KV* rows_s = reinterpret_cast<KV*>(gsm);                                         // [64][d]
    int32_t* idf_s = reinterpret_cast<int32_t*>(gsm + (size_t)kRowsPerCta * s.d * sizeof(KV));   // [nfull]
    const int h = blockIdx.y, b = blockIdx.z >> 1, side = blockIdx.z & 1;
    const int n_init = min(L, s.l_init);
    const int n_local = min(L - n_init, s.l_local);
    const int n_mid = L - n_init - n_local;
    if (blockIdx.x == 0 && blockIdx.y == 0 && side == 0 && threadIdx.x == 0) {
        c.state[kStateStride * b + 0] = n_init;
        c.state[kStateStride * b + 1] = n_local;
        c.state[kStateStride * b + 2] = n_mid;
        c.state[kStateStride * b + 3] = 0;          // ring starts at physical row 0
        c.state[kStateStride * b + 4] = 0;          // append ticket
    }
    const int nfull = side == 0 ? s.nfk : s.nfv;
    if (zero_coef && s.d > nfull) {
        // the contraction kernels behind this one ADD their partial sums: the CTAs of a (b, head, side) clear its coefficients
        float4* cz = reinterpret_cast<float4*>(coef_rows(side == 0 ? c.coef_k : c.coef_v, s, b, h, s.d - nfull));
        const int n4 = s.M * (s.d - nfull) / 4;
        for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x) cz[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const KV* X = (side == 0 ? K : V) + (size_t)b * sb + (size_t)h * sh;
    const int32_t* idf = (side == 0 ? c.idx_full_k : c.idx_full_v) + (size_t)h * nfull;
    void* w_init = side == 0 ? c.k_init : c.v_init;
    void* w_local = side == 0 ? c.k_local : c.v_local;
    void* w_mid = side == 0 ? c.k_mid : c.v_mid;
    // without the kept-dim rows (the tensor-core kernel writes them) the chunks [skip_a, skip_c) of middle tokens only are not launched
    const int chunk = (int)blockIdx.x < skip_a ? (int)blockIdx.x : (int)blockIdx.x + (skip_c - skip_a);
    const int t0 = chunk * kRowsPerCta, nrow = min(L - t0, kRowsPerCta);
    const int cpr = s.d / EPC;                            // chunks per input row
    for (int i = threadIdx.x; i < nfull; i += blockDim.x) idf_s[i] = idf[i];
    for (int i = threadIdx.x; i < nrow * cpr; i += blockDim.x) {
        const int r = i / cpr, ch = i - r * cpr;
        reinterpret_cast<uint4*>(rows_s)[i] = __ldg(reinterpret_cast<const uint4*>(X + (size_t)(t0 + r) * st) + ch);
    }
    __syncthreads();
    // window rows: chunk for chunk
    for (int i = threadIdx.x; i < nrow * cpr; i += blockDim.x) {
        const int r = i / cpr, ch = i - r * cpr, t = t0 + r;
        KV* dst = nullptr;
        if (t < n_init) dst = win_row<KV>(w_init, s, b, h, s.l_init, t);
        else if (t >= L - n_local) dst = win_row<KV>(w_local, s, b, h, s.l_local, t - (L - n_local));
        if (dst) reinterpret_cast<uint4*>(dst)[ch] = reinterpret_cast<const uint4*>(rows_s)[i];
    }
    // kept-dim rows of the middle
    if (!mid_rows) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    const int cpo = nfull / EPC;                          // chunks per output row
    for (int i = threadIdx.x; i < nrow * cpo; i += blockDim.x) {
        const int r = i / cpo, ch = i - r * cpo, t = t0 + r;
        if (t < n_init || t >= L - n_local) continue;
        const int j = t - n_init, cls = j % s.P, slot = j / s.P;
        // output chunk ch holds the logical chunk ch ^ swizzle (the permutation is an involution)
        const int lch = (side == 1 && sizeof(KV) == 2) ? (ch ^ v_swz(slot, nfull >> 3)) : ch;
        const KV* row = rows_s + r * s.d;
        __align__(16) KV vals[EPC];
#pragma unroll
        for (int e = 0; e < EPC; ++e) vals[e] = row[idf_s[lch * EPC + e]];
        KV* dst = mid_row<KV>(w_mid, s, b, h, cls, slot, nfull);
        reinterpret_cast<uint4*>(dst)[ch] = *reinterpret_cast<const uint4*>(vals);
    }
    // In a chain of launches that overlap one another (the partition kernels of several layers, each launched
    // programmatically behind the one before), the end of this grid then implies the end of all before it.  Launched
    // the plain way this returns at once.
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---- Eq.3-4: C[m][e] += sum_j F[m][j] X[n_init + j][D^c[e]] ------------------
// grid (row tiles of 32 coefficient rows, token splits, B * Hkv * 2 sides).
// Per 64-token chunk the CTA stages the gathered columns and a 64 x 32 basis
// tile in shared memory; thread (rg, lane) accumulates rows 4 rg..4 rg + 3 of
// the tile for columns lane, lane + 32, ...  Partial sums of the token splits
// are added to the zeroed coefficients with atomics.
constexpr int kTM = 32, kTJ = 64;

template <typename KV>
__global__ void __launch_bounds__(256) compress_coef_kernel(Dims s, CacheDev c, const KV* __restrict__ K,
                                                            const KV* __restrict__ V, int64_t sb, int64_t st, int64_t sh,
                                                            int L, int chunks_per_split) {
    extern __shared__ float smem[];
    int side = blockIdx.z & 1;
    int bh = blockIdx.z >> 1;
    int b = bh / s.Hkv, h = bh % s.Hkv;
    int nfull = side == 0 ? s.nfk : s.nfv;
    int ncomp = s.d - nfull;
    if (ncomp == 0) return;
    int n_init = min(L, s.l_init);
    int n_local = min(L - n_init, s.l_local);
    int n_mid = L - n_init - n_local;
    const KV* X = (side == 0 ? K : V) + (size_t)b * sb + (size_t)h * sh;
    const int32_t* idc = (side == 0 ? c.idx_comp_k : c.idx_comp_v) + (size_t)h * ncomp;
    float* coef = coef_rows(side == 0 ? c.coef_k : c.coef_v, s, b, h, ncomp);

    float* X_s = smem;                       // [kTJ][ncomp]
    float* F_s = smem + kTJ * ncomp;         // [kTJ][kTM]
    int m0 = blockIdx.x * kTM;
    int rg = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int ncol = (ncomp + 31) / 32;            // <= 8
    float acc[4][8];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[r][i] = 0.f;

    int j_begin = blockIdx.y * chunks_per_split * kTJ;
    int j_end = min(n_mid, j_begin + chunks_per_split * kTJ);
    for (int j0 = j_begin; j0 < j_end; j0 += kTJ) {
        int nj = min(kTJ, j_end - j0);
        __syncthreads();
        for (int i = threadIdx.x; i < kTJ * ncomp; i += blockDim.x) {
            int jj = i / ncomp, e = i - jj * ncomp;
            X_s[i] = jj < nj ? ld_f(X + (size_t)(n_init + j0 + jj) * st + idc[e]) : 0.f;
        }
        // basis tile: thread -> (token jj, frequency pair nn) ; rows 2 nn (cos), 2 nn + 1 (sin)
        for (int i = threadIdx.x; i < kTJ * (kTM / 2); i += blockDim.x) {
            int jj = i / (kTM / 2), nn = i % (kTM / 2);
            int n = m0 / 2 + nn;
            float cs = 0.f, sn = 0.f;
            if (jj < nj && n < s.k) basis_cs(n, j0 + jj, s.T, &cs, &sn);
            F_s[jj * kTM + 2 * nn] = cs;
            F_s[jj * kTM + 2 * nn + 1] = sn;
        }
        __syncthreads();
        for (int jj = 0; jj < nj; ++jj) {
            float4 f = *reinterpret_cast<const float4*>(F_s + jj * kTM + 4 * rg);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (i < ncol) {
                    int e = lane + 32 * i;
                    float x = e < ncomp ? X_s[jj * ncomp + e] : 0.f;
                    acc[0][i] = fmaf(f.x, x, acc[0][i]);
                    acc[1][i] = fmaf(f.y, x, acc[1][i]);
                    acc[2][i] = fmaf(f.z, x, acc[2][i]);
                    acc[3][i] = fmaf(f.w, x, acc[3][i]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        int m = m0 + 4 * rg + r;
        if (m >= s.M) continue;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            int e = lane + 32 * i;
            if (i < ncol && e < ncomp) atomicAdd(coef + (size_t)m * ncomp + e, acc[r][i]);
        }
    }
}

template <typename KV>
static cudaError_t launch_compress_t(const Dims& s, const CacheDev& c, const void* K, const void* V, int64_t sb,
                                     int64_t st, int64_t sh, int L, bool with_coef, bool ordered, bool mid_rows, bool zero_coef, bool chained,
                                     cudaStream_t stream) {
    int chunks_rows = (L + kRowsPerCta - 1) / kRowsPerCta;
    if (chunks_rows < 1) chunks_rows = 1;
    int skip_a = 0, skip_c = 0;
    if (!mid_rows) {
        const int ni = L < s.l_init ? L : s.l_init, nl = (L - ni) < s.l_local ? (L - ni) : s.l_local;
        skip_a = (ni + kRowsPerCta - 1) / kRowsPerCta;          // first chunk past the initial window
        skip_c = (L - nl) / kRowsPerCta;                        // first chunk with a token of the local window
        if (skip_a < 1) skip_a = 1;                             // chunk 0 always runs: it writes the counters
        if (skip_c < skip_a) skip_c = skip_a;
    }
    constexpr int EPC = 16 / (int)sizeof(KV);
    if (s.d % EPC || s.nfk % EPC || s.nfv % EPC || sb % EPC || st % EPC || sh % EPC || (reinterpret_cast<uintptr_t>(K) & 15) ||
        (reinterpret_cast<uintptr_t>(V) & 15))
        return cudaErrorInvalidValue;
    const int nf = s.nfk > s.nfv ? s.nfk : s.nfv;
    const size_t gsmem = (size_t)kRowsPerCta * s.d * sizeof(KV) + sizeof(int32_t) * (size_t)nf;
    cudaError_t err = ensure_dynamic_smem(partition_gather_kernel<KV>, gsmem);
    if (err != cudaSuccess) return err;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(chunks_rows - (skip_c - skip_a), s.Hkv, s.B * 2);
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = gsmem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // chained: may run beside the partition kernel in front of it
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = chained ? 1 : 0;
        err = cudaLaunchKernelEx(&cfg, partition_gather_kernel<KV>, s, c, static_cast<const KV*>(K), static_cast<const KV*>(V), sb, st, sh, L,
                                 mid_rows ? 1 : 0, skip_a, skip_c, zero_coef ? 1 : 0);
    }
    if (err != cudaSuccess) return err;
    int n_init = L < s.l_init ? L : s.l_init;
    int n_local = (L - n_init) < s.l_local ? (L - n_init) : s.l_local;
    int n_mid = L - n_init - n_local;
    int max_comp = s.dck > s.dcv ? s.dck : s.dcv;
    if (n_mid == 0 || max_comp == 0 || !with_coef) return cudaSuccess;
    int row_tiles = (s.M + kTM - 1) / kTM;
    int chunks = (n_mid + kTJ - 1) / kTJ;
    int ctas_fixed = row_tiles * s.B * s.Hkv * 2;
    int n_tsplit = (4 * sm_count() + ctas_fixed - 1) / ctas_fixed;
    if (n_tsplit > chunks) n_tsplit = chunks;
    if (n_tsplit < 1 || ordered) n_tsplit = 1;               // one split: every coefficient is added to zero exactly once
    int cps = (chunks + n_tsplit - 1) / n_tsplit;
    n_tsplit = (chunks + cps - 1) / cps;
    size_t smem = sizeof(float) * ((size_t)kTJ * max_comp + (size_t)kTJ * kTM);
    err = ensure_dynamic_smem(compress_coef_kernel<KV>, smem);
    if (err != cudaSuccess) return err;
    compress_coef_kernel<KV><<<dim3(row_tiles, n_tsplit, s.B * s.Hkv * 2), 256, smem, stream>>>(
        s, c, static_cast<const KV*>(K), static_cast<const KV*>(V), sb, st, sh, L, cps);
    return cudaGetLastError();
}

// with_coef = false runs only the partition / gather kernel (the tensor-core or the transform path computes the
// coefficients); mid_rows = false leaves the kept-dim rows of the middle out too (windows and counters only);
// zero_coef clears the coefficients in the same launch (for the contraction kernels, which add to them).
cudaError_t launch_compress(const Dims& s, const CacheDev& c, int dtype, const void* K, const void* V, int64_t sb,
                            int64_t st, int64_t sh, int L, bool with_coef, bool ordered, bool mid_rows, bool zero_coef,
                            cudaStream_t stream, bool chained) {
    if (dtype == FA_BF16) return launch_compress_t<__nv_bfloat16>(s, c, K, V, sb, st, sh, L, with_coef, ordered, mid_rows, zero_coef, chained, stream);
    return launch_compress_t<float>(s, c, K, V, sb, st, sh, L, with_coef, ordered, mid_rows, zero_coef, chained, stream);
}

}  // namespace fa
