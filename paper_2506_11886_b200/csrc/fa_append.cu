// fa_append (Eq.5): push one token; when the local window is full its oldest
// row leaves, its kept dims join K^mu / V^mu and its compressed dims are added
// to every coefficient row with basis column j = n_mid.  One kernel:
//   grid (row tiles, Hkv, B).  Each CTA updates kAppendRows rows of C^K and C^V:
//   the rows are contiguous, so one bulk copy per side brings them to shared
//   memory (issued before anything else, completion on an mbarrier), the rank-1
//   update runs there and one bulk copy per side takes them back; CTA x == 0 also
//   writes the leaving row's kept dims to the middle.  The last CTA of a batch row to finish (atomic ticket, no
//   waiting) overwrites the ring slot with the new token and advances the
//   counters, so no CTA can see a half-updated state.
#include "fa_common.cuh"
#include "fa_decode_ws.cuh"

namespace fa {

constexpr int kAppendRows = 32;   // coefficient rows per chunk
constexpr int kAppendChunks = 8;  // chunks per CTA, at most (double-buffered)
constexpr uint32_t kAppendSpin = 1u << 22;

namespace {
__device__ __forceinline__ uint32_t sm_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
}  // namespace

// A CTA's life is a chain of dependent memory round trips (counters, leaving row, ticket), so what counts
// is how many bytes are in flight per SM: the coefficient rows travel as bulk copies whose round trip
// overlaps the counters', several CTAs to an SM.
template <typename KV>
__global__ void __launch_bounds__(256) append_kernel(Dims s, CacheDev c, const KV* __restrict__ k_new,
                                                     const KV* __restrict__ v_new, int n_chunks) {
    // one or two buffers of [kAppendRows][dck] of C^K, then [kAppendRows][dcv] of C^V
    extern __shared__ __align__(128) float coef_s[];
    __shared__ float x_s[2][256];        // the row that leaves, both sides, natural dim order
    __shared__ __align__(16) float xc_s[2][256];   // the same gathered at D^kc / D^vc
    __shared__ float f_s[kAppendRows * kAppendChunks];   // basis column j for the rows of this CTA
    __shared__ __align__(8) uint64_t bar_s[2];
    __shared__ int last_s;
    const int h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
    // programmatic dependent launch: the next kernel may be scheduled now; this one first waits for
    // everything its predecessor in the stream wrote
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // The coefficient rows set off first: their addresses depend on the grid alone, so their round trip
    // overlaps the one of the counters.  Every path below waits for them before the CTA ends.
    // A CTA owns n_chunks chunks of kAppendRows rows; chunk i travels through buffer i & 1 (load, update, store), the
    // load of chunk i + 2 following the store of chunk i, so that a CTA pays its chain of counters, leaving row and
    // ticket once for all its rows.
    const int m0 = blockIdx.x * n_chunks * kAppendRows;
    const int rows_cta = max(0, min(n_chunks * kAppendRows, s.M - m0));
    const int n_ch = (rows_cta + kAppendRows - 1) / kAppendRows;
    const int buf_floats = kAppendRows * (s.dck + s.dcv);
    const bool any_coef = s.dck + s.dcv > 0 && n_ch > 0;
    auto chunk_rows = [&](int ch) { return min(kAppendRows, rows_cta - ch * kAppendRows); };
    // (thread 0) bulk loads of chunk ch into its buffer, completion on the buffer's barrier
    auto load_chunk = [&](int ch) {
        const int bf = ch & 1, rows = chunk_rows(ch), r0 = m0 + ch * kAppendRows;
        float* ck_s = coef_s + (size_t)bf * buf_floats;
        float* cv_s = ck_s + (size_t)kAppendRows * s.dck;
        const uint32_t bytes_k = (uint32_t)(rows * s.dck * 4), bytes_v = (uint32_t)(rows * s.dcv * 4);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sm_addr(&bar_s[bf])), "r"(bytes_k + bytes_v) : "memory");
        if (bytes_k)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sm_addr(ck_s)),
                         "l"(__cvta_generic_to_global(coef_rows(c.coef_k, s, b, h, s.dck) + (size_t)r0 * s.dck)), "r"(bytes_k),
                         "r"(sm_addr(&bar_s[bf]))
                         : "memory");
        if (bytes_v)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sm_addr(cv_s)),
                         "l"(__cvta_generic_to_global(coef_rows(c.coef_v, s, b, h, s.dcv) + (size_t)r0 * s.dcv)), "r"(bytes_v),
                         "r"(sm_addr(&bar_s[bf]))
                         : "memory");
    };
    if (tid == 0 && any_coef) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_addr(&bar_s[0])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_addr(&bar_s[1])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        load_chunk(0);
        if (n_ch > 1) load_chunk(1);
    }
    // Bounded wait for chunk ch (one thread polls, then the CTA meets); false after a time-out.
    auto chunk_landed = [&](int ch) -> bool {
        __shared__ int ok_s;
        if (tid == 0) {
            int ok = 1;
            if (any_coef) {
                ok = 0;
                const uint32_t parity = (uint32_t)(ch >> 1) & 1u;
                for (uint32_t i = 0; i < kAppendSpin && !ok; ++i) {
                    uint32_t done;
                    asm volatile(
                        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                        : "=r"(done)
                        : "r"(sm_addr(&bar_s[ch & 1])), "r"(parity)
                        : "memory");
                    ok = (int)done;
                }
                if (!ok) atomicExch(c.status, (int)FA_ERR_TIMEOUT);
            }
            ok_s = ok;
        }
        __syncthreads();
        const bool ok = ok_s != 0;
        __syncthreads();                 // ok_s may be written again
        return ok;
    };
    // the loads issued so far have landed: nothing may still be writing this CTA's shared memory when it ends
    auto rows_landed = [&]() -> bool {
        bool ok = chunk_landed(0);
        if (n_ch > 1) ok = chunk_landed(1) && ok;
        return ok;
    };
    const int n_init = c.state[kStateStride * b + 0], n_local = c.state[kStateStride * b + 1];
    const int n_mid = c.state[kStateStride * b + 2], head = c.state[kStateStride * b + 3];
    const bool to_init = n_init < s.l_init;
    const bool evict = !to_init && n_local == s.l_local;
    const bool full = evict && (n_mid >= s.max_mid || n_mid >= s.T);
    if (full) {
        if (tid == 0 && blockIdx.x == 0 && h == 0) atomicExch(c.status, (int)FA_ERR_CAPACITY);
        rows_landed();                   // nothing may still be writing this CTA's shared memory when it ends
        return;                          // every CTA of this batch row takes the same exit
    }
    if (!evict) rows_landed();
    if (evict) {
        const int j = n_mid;
        // the row that leaves: oldest ring row, or the new token itself if there is no local window
        for (int i = tid; i < 2 * s.d; i += 256) {
            const int side = i / s.d, e = i - side * s.d;
            float v;
            if (s.l_local == 0) v = ld_f((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + h) * s.d + e);
            else v = ld_f(win_row<KV>(side == 0 ? c.k_local : c.v_local, s, b, h, s.l_local, head) + e);
            x_s[side][e] = v;
        }
        for (int r = tid; r < rows_cta; r += 256) {
            float cs, sn;
            const int m = m0 + r;
            basis_cs(m >> 1, j, s.T, &cs, &sn);
            f_s[r] = (m & 1) ? sn : cs;
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
        __syncthreads();                 // f_s and xc_s are complete
        bool live = true;
#pragma unroll 1
        for (int ch = 0; ch < n_ch; ++ch) {
            live = chunk_landed(ch) && live;
            const int rows = chunk_rows(ch), r0 = m0 + ch * kAppendRows;
            float* ck_s = coef_s + (size_t)(ch & 1) * buf_floats;
            float* cv_s = ck_s + (size_t)kAppendRows * s.dck;
            if (live) {
#pragma unroll
                for (int side = 0; side < 2; ++side) {
                    const int ncomp = side == 0 ? s.dck : s.dcv;
                    const int vpr = ncomp >> 2;
                    float4* rows4 = reinterpret_cast<float4*>(side == 0 ? ck_s : cv_s);
#pragma unroll 4
                    for (int i = tid; i < rows * vpr; i += 256) {
                        const int r = i / vpr, v4 = i - r * vpr;
                        const float f = f_s[ch * kAppendRows + r];
                        const float4 x = *reinterpret_cast<const float4*>(&xc_s[side][4 * v4]);
                        float4 o = rows4[i];
                        o.x = fmaf(f, x.x, o.x);
                        o.y = fmaf(f, x.y, o.y);
                        o.z = fmaf(f, x.z, o.z);
                        o.w = fmaf(f, x.w, o.w);
                        rows4[i] = o;
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // these stores, then the bulk copies that read them
            __syncthreads();
            if (tid == 0 && any_coef) {
                const uint32_t bytes_k = (uint32_t)(rows * s.dck * 4), bytes_v = (uint32_t)(rows * s.dcv * 4);
                if (live) {
                    if (bytes_k)
                        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(__cvta_generic_to_global(
                                         coef_rows(c.coef_k, s, b, h, s.dck) + (size_t)r0 * s.dck)),
                                     "r"(sm_addr(ck_s)), "r"(bytes_k)
                                     : "memory");
                    if (bytes_v)
                        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(__cvta_generic_to_global(
                                         coef_rows(c.coef_v, s, b, h, s.dcv) + (size_t)r0 * s.dcv)),
                                     "r"(sm_addr(cv_s)), "r"(bytes_v)
                                     : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                // the buffer goes to chunk ch + 2 once the store has read it; the last stores are waited for before the CTA ends
                if (ch + 2 < n_ch || ch + 1 >= n_ch) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                if (ch + 2 < n_ch && live) load_chunk(ch + 2);
            }
        }
    }
    // ticket: the last CTA of this batch row stores the new token and advances the counters.  What the
    // ticket orders is every CTA's read of the leaving row (consumed above) before the overwrite of its
    // ring slot; the coefficient stores need no fence here, the end of the kernel publishes them.
    __syncthreads();
    if (tid == 0) {
        const int done = atomicAdd(c.state + kStateStride * b + 4, 1);
        last_s = (done == (int)(gridDim.x * gridDim.y) - 1);
    }
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    // The new token of every head of this batch row, in 16-byte chunks, all loads of a round before its
    // stores: this CTA runs alone at the end of the kernel, so its round trips are the kernel's tail.
    if (to_init || s.l_local > 0) {
        constexpr int EPC = 16 / (int)sizeof(KV);
        const int cpr = s.d / EPC, nchunk = 2 * s.Hkv * cpr;
        const int slot = to_init ? n_init : (evict ? head : (head + n_local) % s.l_local);
#pragma unroll 1
        for (int base = 0; base < nchunk; base += 256 * 4) {
            uint4 v[4];
            uint4* dst[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = base + tid + 256 * u;
                dst[u] = nullptr;
                if (i < nchunk) {
                    const int side = i / (s.Hkv * cpr), rem = i - side * (s.Hkv * cpr);
                    const int hh = rem / cpr, ch = rem - hh * cpr;
                    v[u] = reinterpret_cast<const uint4*>((side == 0 ? k_new : v_new) + ((size_t)b * s.Hkv + hh) * s.d)[ch];
                    void* w = to_init ? (side == 0 ? c.k_init : c.v_init) : (side == 0 ? c.k_local : c.v_local);
                    dst[u] = reinterpret_cast<uint4*>(win_row<KV>(w, s, b, hh, to_init ? s.l_init : s.l_local, slot)) + ch;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (dst[u]) *dst[u] = v[u];
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

template <typename KV>
static cudaError_t launch_append_t(const Dims& s, const CacheDev& c, const void* k_new, const void* v_new,
                                   cudaStream_t st) {
    // Chunks of kAppendRows rows per CTA: one while the grid fits the device about four CTAs to an SM, more (up to
    // kAppendChunks, through two buffers) when it would not: a CTA then pays its chain of dependent round trips
    // (counters, leaving row, ticket) once for all its chunks, and the grid runs as one wave.
    const int chunks_all = (s.M + kAppendRows - 1) / kAppendRows;
    const long long ctas1 = (long long)chunks_all * s.Hkv * s.B, slots = 4LL * sm_count();
    int n_chunks = (int)((ctas1 + slots - 1) / slots);
    if (n_chunks > kAppendChunks) n_chunks = kAppendChunks;
    if (n_chunks > chunks_all) n_chunks = chunks_all;
    if (n_chunks < 1) n_chunks = 1;
    const int tiles = (chunks_all + n_chunks - 1) / n_chunks;
    const size_t smem = sizeof(float) * (size_t)kAppendRows * (s.dck + s.dcv) * (n_chunks > 1 ? 2 : 1);
    cudaError_t err = ensure_dynamic_smem(append_kernel<KV>, smem);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles, s.Hkv, s.B);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, append_kernel<KV>, s, c, static_cast<const KV*>(k_new), static_cast<const KV*>(v_new), n_chunks);
}

cudaError_t launch_append(const Dims& s, const CacheDev& c, int dtype, const void* k_new, const void* v_new,
                          cudaStream_t st) {
    if (dtype == FA_BF16) return launch_append_t<__nv_bfloat16>(s, c, k_new, v_new, st);
    return launch_append_t<float>(s, c, k_new, v_new, st);
}

}  // namespace fa
