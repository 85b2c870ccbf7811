// Host side of the C ABI declared in include/fa.h: argument checks, buffer
// sizes, launch plans.  Every entry point validates on the host, then launches
// on the caller's stream; nothing here allocates device memory.
#include <cstring>
#include <mutex>

#include "fa_common.cuh"

namespace fa {

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline size_t elt_bytes(int dtype) { return dtype == FA_BF16 ? 2 : 4; }

fa_status check_layout(const fa_layout* l) {
    if (!l) return FA_ERR_INVALID_ARG;
    if (l->batch < 1 || l->n_q_heads < 1 || l->n_kv_heads < 1 || l->head_dim < 8) return FA_ERR_INVALID_ARG;
    if (l->n_q_heads % l->n_kv_heads != 0) return FA_ERR_INVALID_ARG;
    if (l->n_full_k < 0 || l->n_full_k > l->head_dim || l->n_full_v < 0 || l->n_full_v > l->head_dim)
        return FA_ERR_INVALID_ARG;
    if (l->n_coef < 2 || (l->n_coef & 1) || l->period < 2 || l->n_coef > l->period) return FA_ERR_INVALID_ARG;
    if (l->l_init < 0 || l->l_local < 0 || l->max_mid < 0 || l->max_mid > l->period) return FA_ERR_INVALID_ARG;
    if (l->mid_classes < 1) return FA_ERR_INVALID_ARG;
    if (l->kv_dtype != FA_F32 && l->kv_dtype != FA_BF16) return FA_ERR_INVALID_ARG;
    if (l->norm != FA_NORM_ORTHO && l->norm != FA_NORM_PAPER) return FA_ERR_INVALID_ARG;
    if (l->decode_algo < FA_DECODE_AUTO || l->decode_algo > FA_DECODE_FFT_SPLIT) return FA_ERR_INVALID_ARG;
    if (!(l->softmax_scale > 0.0f)) return FA_ERR_INVALID_ARG;
    // what the kernels implement
    if (l->head_dim % 8 != 0 || l->head_dim > 256) return FA_ERR_UNSUPPORTED;
    if (l->n_full_k % 8 != 0 || l->n_full_v % 8 != 0) return FA_ERR_UNSUPPORTED;
    if (l->n_q_heads / l->n_kv_heads > 16) return FA_ERR_UNSUPPORTED;
    if (l->n_coef > 4096) return FA_ERR_UNSUPPORTED;
    return FA_OK;
}

// Host-side caches of this library (what the driver granted or answered so far) are small tables
// behind this one mutex, keyed by device where the answer depends on it: two host threads may make
// their first calls at the same time.
static std::mutex g_host_mu;

// Number of SMs of the current device (148 when no device can be asked, e.g. on a host without a GPU:
// the sizes computed from it are then those of a B200).
int sm_count() {
    constexpr int kMaxDev = 64;
    static int cached[kMaxDev] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) { cudaGetLastError(); return kNumSmsDefault; }
    std::lock_guard<std::mutex> lock(g_host_mu);
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { cudaGetLastError(); n = kNumSmsDefault; }
        cached[dev] = n;
    }
    return cached[dev];
}

// True if the current device supports cooperative launches (asked once per device).
bool cooperative_launch_supported() {
    constexpr int kMaxDev = 64;
    static signed char cached[kMaxDev] = {0};          // 0 unknown, 1 yes, -1 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) { cudaGetLastError(); return false; }
    std::lock_guard<std::mutex> lock(g_host_mu);
    if (cached[dev] == 0) {
        int coop = 0;
        const bool ok = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && coop;
        if (!ok) cudaGetLastError();
        cached[dev] = ok ? 1 : -1;
    }
    return cached[dev] > 0;
}

// (kernel, device) -> largest dynamic shared memory size granted so far.
cudaError_t ensure_dynamic_smem_impl(const void* kernel, size_t bytes) {
    struct Entry { const void* fn; int dev; size_t bytes; };
    static Entry table[256];
    static int used = 0;
    if (bytes <= 32 * 1024) return cudaSuccess;       // (static shared memory counts against the 48 KB that need no opt-in)
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    std::lock_guard<std::mutex> lock(g_host_mu);
    Entry* hit = nullptr;
    for (int i = 0; i < used; ++i)
        if (table[i].fn == kernel && table[i].dev == dev) { hit = &table[i]; break; }
    if (hit && bytes <= hit->bytes) return cudaSuccess;
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (err != cudaSuccess) return err;
    if (hit) hit->bytes = bytes;
    else if (used < 256) table[used++] = Entry{kernel, dev, bytes};
    return cudaSuccess;
}

static int ilog2_exact(int v) {
    int l = 0;
    while ((1 << l) < v) ++l;
    return ((1 << l) == v) ? l : -1;
}

// True if the residue-class transform kernel can serve this layout: power-of-two period split
// into P classes of S = T / P slots, S a power of two in [32, 2048]; at most 64 kept dims per
// side, head_dim <= 128, and the kernel's shared memory must fit.
static bool fft_ok(const fa_layout& l, int gh, int* log2S) {
    if (l.kv_dtype != FA_BF16) return false;                                   // tensor-core dot products: bf16 caches
    if (l.head_dim == l.n_full_k && l.head_dim == l.n_full_v) return false;   // nothing compressed
    if (ilog2_exact(l.period) < 0 || l.period % l.mid_classes != 0) return false;
    int S = l.period / l.mid_classes;
    int ls = ilog2_exact(S);
    if (ls < 5 || ls > 10) return false;
    if (l.n_coef / 2 > S) return false;                                        // every frequency needs its own bin
    if (l.n_full_k > 64 || l.n_full_v > 64 || l.head_dim > 128) return false;
    if ((long long)l.l_init + l.l_local > (1 << 22)) return false;                // 32-bit split arithmetic in the kernel
    if (decode_fft_smem_bytes(make_dims(l), ls, gh, 1) > 227 * 1024) return false;
    *log2S = ls;
    return true;
}

fa_status plan_decode(const fa_layout& l, DecodePlan* p) {
    Dims s = make_dims(l);
    std::memset(p, 0, sizeof(*p));
    const int kNumSms = sm_count();
    int log2S = 0;
    const int gh_fft = s.G >= 3 ? 4 : 2;
    const bool can_fft = fft_ok(l, gh_fft, &log2S);
    const bool want_fft = l.decode_algo == FA_DECODE_FFT || l.decode_algo == FA_DECODE_FFT_SPLIT;
    if (want_fft && !can_fft) return FA_ERR_UNSUPPORTED;
    p->algo = (l.decode_algo == FA_DECODE_DIRECT || !can_fft) ? FA_DECODE_DIRECT : FA_DECODE_FFT;
    p->fft_log2 = log2S;
    if (p->algo == FA_DECODE_FFT) {
        p->gh = gh_fft;
        p->n_pass = (s.G + p->gh - 1) / p->gh;
        const int jobs = s.B * s.Hkv * p->n_pass;
        // One CTA per SM (a ring of stages and a whole batch of classes per CTA).  When every
        // (b, KV head, pass) can have a CTA resident at once, the kernel is fused: it forms u itself
        // and merges its own partial results, its CTAs waiting for one another (cooperative
        // launch).  A head gets floor(SMs / heads) CTAs; the window tokens either share the class
        // CTAs or get CTAs of their own, whichever keeps the largest CTA's bytes smallest.  With more
        // heads than SMs a head gets one CTA, which waits for nobody: a plain launch that runs in waves.
        const long long win_bytes = 2LL * (s.l_init + s.l_local) * s.d;
        const long long class_bytes = (long long)(s.T / s.P) * (s.nfk + s.nfv);
        // classes transformed together: enough butterflies for all consumer threads, within shared memory
        auto pick_nb = [&](int n_split, int occ = 1) {
            const int S = s.T / s.P;
            // (one query head per KV head: a transform carries two classes, so twice the classes fill the same buffers)
            const int pairs = (s.G == 1 && p->gh == 2) ? 2 : 1;
            int nb = pairs * 2048 / S;
            if (nb < 1) nb = 1;
            if (nb > 8 * pairs * pairs) nb = 8 * pairs * pairs;
            const int per_cta = (s.P + n_split - 1) / n_split;
            if (nb > per_cta) nb = per_cta;
            const size_t limit = occ == 2 ? 113 * 1024 : 227 * 1024;      // two CTAs share the SM's 228 KB, 1 KB reserved each
            while (nb > 1 && decode_fft_smem_bytes(s, log2S, p->gh, nb, occ) > limit) --nb;
            return nb;
        };
        p->fused = 0;
        p->n_wsplit = 0;
        p->occ = 1;
        p->split = 0;
        // Short transforms leave room for two CTAs on an SM (a shorter ring, a register cap): one CTA's
        // dependent phases hide behind the other's, and a head gets twice the CTAs (or, with more heads
        // than SMs, the waves are twice as wide).  Tried first; one CTA per SM otherwise.
        for (int occ = log2S <= 8 ? 2 : 1; occ >= 1 && !p->fused && l.decode_algo != FA_DECODE_FFT_SPLIT; --occ) {
            const size_t smem_limit = occ == 2 ? 113 * 1024 : 227 * 1024;
            const int slots = kNumSms * occ;
            const int per_job = jobs < slots ? slots / jobs : 1;
            // Fewer CTAs per head than the device offers when the merge scratch of the fused kernel could
            // not hold the partial results of that many parts (one KV head alone could have them all).
            for (int pj = per_job; pj >= 1 && !p->fused; pj = pj > 24 ? 24 : pj - 1) {
                int best_ns = 0, best_nw = 0;
                long long best_cost = -1;
                // nw = 0: the window tokens are spread over the class CTAs (few CTAs per head); else CTAs of their own
                for (int nw = 0; nw <= 8 && nw < pj; ++nw) {
                    int ns = pj - nw;
                    if (ns > s.P) ns = s.P;
                    const long long cc = (long long)((s.P + ns - 1) / ns) * class_bytes + (nw == 0 ? (win_bytes + ns - 1) / ns : 0);
                    const long long wc = nw ? (win_bytes + nw - 1) / nw : 0;
                    const long long cost = cc > wc ? cc : wc;
                    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_ns = ns; best_nw = nw; }
                    if (win_bytes == 0) break;
                }
                // fewest class CTAs that reach the same classes per CTA
                const int per_cta = (s.P + best_ns - 1) / best_ns;
                best_ns = (s.P + per_cta - 1) / per_cta;
                const int nb = pick_nb(best_ns, occ);
                if (occ == 2 && nb < (per_cta < 4 ? per_cta : 4)) break;                   // too few classes per transform batch: not worth it
                if (decode_fft_smem_bytes(s, log2S, p->gh, nb, occ) <= smem_limit &&
                    decode_fft_fused_fits(s, log2S, p->gh, nb, best_ns + best_nw, occ)) {
                    p->fused = 1;
                    p->n_split = best_ns;
                    p->n_wsplit = best_nw;
                    p->nb = nb;
                    p->occ = occ;
                }
            }
        }
        // Three-kernel form.  Classes are indivisible: pick the split count that minimises
        // waves * (classes per CTA + a CTA's fixed cost, about two classes' worth), smallest count on ties.
        int best = 1;
        long long best_cost = -1;
        for (int n = 1; n <= s.P && n <= 64; ++n) {
            long long waves = ((long long)jobs * n + kNumSms - 1) / kNumSms;
            long long cost = waves * ((s.P + n - 1) / n + 2);
            if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = n; }
        }
        // More heads than SMs: the lone CTAs of the fused kernel run in whole waves.  AUTO keeps it unless
        // the balanced split is ahead by the same cost model (the last wave nearly empty) by more than
        // the margin that the three launches and the round trip of u and the partial results cost.
        // (Heads that are all resident at once, two to an SM, stay fused: a lone CTA takes as long with a neighbour on
        // its SM as without, measured 116-118 us for 160 to 256 heads of the MHA serving shape against 138 us split.)
        if (p->fused && jobs > kNumSms * p->occ && l.decode_algo == FA_DECODE_AUTO &&
            20LL * ((jobs + kNumSms * p->occ - 1) / (kNumSms * p->occ)) * (s.P + 2) * p->occ > 23 * best_cost)
            p->fused = 0;
        if (!p->fused) {
            p->n_wsplit = 0;
            p->occ = 1;
            p->n_split = best;
            p->nb = pick_nb(best);
        }
        // Split build of the fused kernel (one CTA per SM): six more warps (the tile group) form the kept-dim products
        // of a batch of classes beside the eight transform warps: the scores under the batch's spectra and score
        // transform, the V products under its probability transform and fold.  Measured: it pays for the longest
        // transforms when a CTA has several batches (their products then hide completely); with one batch per CTA
        // the score products already run under the wait for the head's u rows and six warps form them slower than
        // eight, and the shorter transforms lose more to the tile group's issue slots than the V products cost.
        if (p->fused && p->occ == 1 && log2S == 10 && !(s.G == 1 && p->gh == 2)) {
            const int per_cta = (s.P + p->n_split - 1) / p->n_split;
            // its shorter ring leaves room for a larger batch
            int nb = per_cta < 2 ? per_cta : 2;
            while (nb > p->nb && decode_fft_smem_bytes(s, log2S, p->gh, nb, 1, 1) > 227 * 1024) --nb;
            if (nb < p->nb) nb = p->nb;
            if (per_cta >= 2 * p->nb && decode_fft_smem_bytes(s, log2S, p->gh, nb, 1, 1) <= 227 * 1024 &&
                decode_fft_fused_fits(s, log2S, p->gh, nb, p->n_split + p->n_wsplit, 1, 1)) {
                p->split = 1;
                p->nb = nb;
            }
        }
    } else {
        p->gh = s.G >= 4 ? 4 : (s.G >= 2 ? 2 : 1);
        if (s.G == 3) p->gh = 4;
        p->n_pass = (s.G + p->gh - 1) / p->gh;
        // split the tokens of one (b, KV head, pass) over CTAs so that the grid fills the GPU about twice
        int jobs = s.B * s.Hkv * p->n_pass;
        int want = (2 * kNumSms + jobs - 1) / jobs;
        long long tokens = (long long)s.max_mid + s.l_init + s.l_local;
        int max_by_work = (int)((tokens + 255) / 256);            // at least one 256-token tile each
        if (want > max_by_work) want = max_by_work;
        if (want > 64) want = 64;
        if (want < 1) want = 1;
        p->n_split = want;
    }
    p->n_part = p->n_split + p->n_wsplit;
    p->rows_pro = 32;
    p->n_slice = s.dcv > 0 ? (s.M + 63) / 64 : 1;
    size_t off = 0;
    p->off_bar = off; off = align_up(off + sizeof(int32_t) * 4 * (size_t)kBarSlots, 256);   // same place and size for every layout
    p->off_u = off;   off = align_up(off + sizeof(float) * (size_t)s.B * s.Hq * s.M, 256);
    p->off_ml = off;  off = align_up(off + sizeof(float) * (size_t)s.B * s.Hq * p->n_part * 2, 256);
    p->off_o = off;   off = align_up(off + sizeof(float) * (size_t)s.B * s.Hq * p->n_part * s.d, 256);
    p->off_z = off;   off = align_up(off + sizeof(float) * (size_t)s.B * s.Hq * p->n_part * s.M, 256);
    const int n_oc = p->n_slice > p->n_part ? p->n_slice : p->n_part;
    p->off_oc = off;  off = align_up(off + sizeof(float) * (size_t)s.B * s.Hq * n_oc * (s.dcv > 0 ? s.dcv : 1), 256);
    p->off_om = off;  off = align_up(off + sizeof(float) * (size_t)s.B * s.Hq * s.d, 256);
    p->off_cnt = off; off = align_up(off + sizeof(int32_t) * (size_t)s.B * s.Hkv, 256);
    p->total = off;
    return FA_OK;
}

// Copies the step's host inputs into the staging buffer with one launch: pinned host memory is
// readable by the device, and one kernel costs less than three copy operations in the stream.
__global__ void stage_inputs_kernel(const uint4* __restrict__ q, const uint4* __restrict__ k, const uint4* __restrict__ v,
                                    uint4* q_d, uint4* k_d, uint4* v_d, int nq, int nk) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nq) q_d[i] = q[i];
    else if (i < nq + nk) k_d[i - nq] = k[i - nq];
    else if (i < nq + 2 * nk) v_d[i - nq - nk] = v[i - nq - nk];
}

// Device-side address of a host buffer the device can read directly (pinned / registered), or nullptr.
static const void* device_view_of_host(const void* p) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer) return nullptr;
    return a.devicePointer;
}

static fa_status check_cache(const fa_layout* l, const fa_cache* c) {
    if (!c) return FA_ERR_INVALID_ARG;
    Dims s = make_dims(*l);
    const void* need[] = {c->state, c->status};
    for (const void* p : need) if (!p || !aligned16(p)) return FA_ERR_INVALID_ARG;
    if (s.nfk > 0 && (!c->idx_full_k || (s.max_mid > 0 && !c->k_mid))) return FA_ERR_INVALID_ARG;
    if (s.nfv > 0 && (!c->idx_full_v || (s.max_mid > 0 && !c->v_mid))) return FA_ERR_INVALID_ARG;
    if (s.dck > 0 && (!c->idx_comp_k || !c->coef_k)) return FA_ERR_INVALID_ARG;
    if (s.dcv > 0 && (!c->idx_comp_v || !c->coef_v)) return FA_ERR_INVALID_ARG;
    if (s.l_init > 0 && (!c->k_init || !c->v_init)) return FA_ERR_INVALID_ARG;
    if (s.l_local > 0 && (!c->k_local || !c->v_local)) return FA_ERR_INVALID_ARG;
    const void* al[] = {c->k_init, c->v_init, c->k_local, c->v_local, c->k_mid, c->v_mid, c->coef_k, c->coef_v,
                        c->idx_full_k, c->idx_comp_k, c->idx_full_v, c->idx_comp_v};
    for (const void* p : al) if (p && !aligned16(p)) return FA_ERR_INVALID_ARG;
    return FA_OK;
}

}  // namespace fa

using namespace fa;

extern "C" {

fa_status fa_cache_sizes_of(const fa_layout* layout, fa_cache_sizes* out) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    if (!out) return FA_ERR_INVALID_ARG;
    Dims s = make_dims(*layout);
    size_t eb = elt_bytes(layout->kv_dtype);
    size_t bh = (size_t)s.B * s.Hkv;
    out->idx_full_k = sizeof(int32_t) * (size_t)s.Hkv * s.nfk;
    out->idx_comp_k = sizeof(int32_t) * (size_t)s.Hkv * s.dck;
    out->idx_full_v = sizeof(int32_t) * (size_t)s.Hkv * s.nfv;
    out->idx_comp_v = sizeof(int32_t) * (size_t)s.Hkv * s.dcv;
    out->k_init = out->v_init = bh * s.l_init * s.d * eb;
    out->k_local = out->v_local = bh * s.l_local * s.d * eb;
    out->k_mid = bh * (size_t)s.P * s.S_cap * s.nfk * eb;
    out->v_mid = bh * (size_t)s.P * s.S_cap * s.nfv * eb;
    out->coef_k = bh * (size_t)s.M * s.dck * sizeof(float);
    out->coef_v = bh * (size_t)s.M * s.dcv * sizeof(float);
    out->state = sizeof(int32_t) * kStateStride * (size_t)s.B;
    out->status = sizeof(int32_t) * 4;
    return FA_OK;
}

fa_status fa_workspace_bytes(const fa_layout* layout, size_t* out) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    if (!out) return FA_ERR_INVALID_ARG;
    DecodePlan p;
    st = plan_decode(*layout, &p);
    if (st != FA_OK) return st;
    *out = p.total;
    if (p.fused) {                       // room for the three-kernel form too, should a cooperative launch not fit
        fa_layout split = *layout;
        split.decode_algo = FA_DECODE_FFT_SPLIT;
        DecodePlan p2;
        if (plan_decode(split, &p2) == FA_OK && p2.total > *out) *out = p2.total;
    }
    return FA_OK;
}

fa_status fa_workspace_init(void* ws, size_t ws_bytes, void* stream) {
    if (!ws || !aligned16(ws) || ws_bytes < 4096) return FA_ERR_WORKSPACE;
    if (cudaMemsetAsync(ws, 0, 4096, static_cast<cudaStream_t>(stream)) != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

fa_status fa_cache_reset(const fa_layout* layout, fa_cache* cache, void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    fa_cache_sizes sz;
    fa_cache_sizes_of(layout, &sz);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(cache->state, 0, sz.state, s) != cudaSuccess) return FA_ERR_CUDA;
    if (cudaMemsetAsync(cache->status, 0, sz.status, s) != cudaSuccess) return FA_ERR_CUDA;
    if (sz.coef_k && cudaMemsetAsync(cache->coef_k, 0, sz.coef_k, s) != cudaSuccess) return FA_ERR_CUDA;
    if (sz.coef_v && cudaMemsetAsync(cache->coef_v, 0, sz.coef_v, s) != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

fa_status fa_poll_status(const fa_cache* cache, void* stream) {
    if (!cache || !cache->status) return FA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, cache->status, sizeof(word), cudaMemcpyDeviceToHost, s) != cudaSuccess) return FA_ERR_CUDA;
    if (cudaMemsetAsync(cache->status, 0, sizeof(word), s) != cudaSuccess) return FA_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return FA_ERR_CUDA;
    if (word < FA_OK || word > FA_ERR_INDEX) return FA_ERR_CUDA;
    return static_cast<fa_status>(word);
}

fa_status fa_validate(const fa_layout* layout, const fa_cache* cache, void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (launch_validate(make_dims(*layout), make_cache(*cache), s) != cudaSuccess) return FA_ERR_CUDA;
    return fa_poll_status(cache, stream);
}

fa_status fa_compress_ex(const fa_layout* layout, fa_cache* cache, const void* K, const void* V, int64_t stride_b,
                         int64_t stride_t, int64_t stride_h, int32_t L, uint32_t flags, void* ws, size_t ws_bytes, void* stream) {
    (void)ws; (void)ws_bytes;
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    if (L < 0 || (flags & ~(uint32_t)(FA_COMPRESS_ORDERED | FA_COMPRESS_FFT))) return FA_ERR_INVALID_ARG;
    if (L > 0 && (!K || !V || !aligned16(K) || !aligned16(V))) return FA_ERR_INVALID_ARG;
    if (L > 0 && (stride_t < layout->head_dim || stride_h < layout->head_dim || stride_b < 0)) return FA_ERR_INVALID_ARG;
    if ((stride_b | stride_t | stride_h) & 7) return FA_ERR_INVALID_ARG;
    Dims s = make_dims(*layout);
    int n_init = L < s.l_init ? L : s.l_init;
    int n_local = (L - n_init) < s.l_local ? (L - n_init) : s.l_local;
    if (L - n_init - n_local > s.max_mid) return FA_ERR_CAPACITY;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int64_t sbb = s.B > 1 ? stride_b : 0;
    const bool ordered = (flags & FA_COMPRESS_ORDERED) != 0;
    if (flags & FA_COMPRESS_FFT) {
        // transform path: one store per coefficient, nothing to clear
        int log2S = 0;
        if (!compress_fft_supported(s, &log2S)) return FA_ERR_UNSUPPORTED;
        if (launch_compress(s, make_cache(*cache), layout->kv_dtype, K, V, stride_b, stride_t, stride_h, L, false, true, true, false, cs) != cudaSuccess)
            return FA_ERR_CUDA;
        if (L > 0 && launch_compress_fft(s, make_cache(*cache), layout->kv_dtype, K, V, sbb, stride_t, stride_h, L, log2S, cs) != cudaSuccess)
            return FA_ERR_CUDA;
        if (L == 0) {
            fa_cache_sizes sz0;
            fa_cache_sizes_of(layout, &sz0);
            if (sz0.coef_k && cudaMemsetAsync(cache->coef_k, 0, sz0.coef_k, cs) != cudaSuccess) return FA_ERR_CUDA;
            if (sz0.coef_v && cudaMemsetAsync(cache->coef_v, 0, sz0.coef_v, cs) != cudaSuccess) return FA_ERR_CUDA;
        }
        return FA_OK;
    }
    // The tensor-core path rounds the basis to bf16 (relative error 2^-9 per term); summed over n middle
    // tokens the coefficient error relative to the largest coefficient falls like 1 / sqrt(n): short
    // middles (where the tensor cores would idle anyway) take the fp32 kernel to stay within 1e-3.
    const int n_mid_host = L - n_init - n_local;
    const bool tc = L > 0 && n_mid_host >= 1024 && compress_tc_supported(s, layout->kv_dtype, sbb, stride_t, stride_h);
    // tensor-core path: its kernel also writes the kept-dim rows of the middle from the boxes it loads; the partition
    // kernel is left with the windows and the counters
    bool tc2 = tc && compress_tc2_supported(s);             // CTA pairs where the row tiles pair up
    bool tc_rows = tc && (tc2 ? compress_tc2_gathers(s) : compress_tc_gathers(s));
    if (launch_compress(s, make_cache(*cache), layout->kv_dtype, K, V, stride_b, stride_t, stride_h, L, !tc, ordered, !tc_rows, true, cs) != cudaSuccess)
        return FA_ERR_CUDA;
    if (tc2 && launch_compress_tc2(s, make_cache(*cache), K, V, sbb, stride_t, stride_h, L, ordered, tc_rows, cs) != cudaSuccess) {
        // the cluster launch was refused (e.g. a partitioned device): the single-CTA kernel does the same work; if it
        // cannot write the kept-dim rows itself, the partition kernel runs once more with them
        cudaGetLastError();
        tc2 = false;
        if (tc_rows && !compress_tc_gathers(s)) {
            tc_rows = false;
            if (launch_compress(s, make_cache(*cache), layout->kv_dtype, K, V, stride_b, stride_t, stride_h, L, false, ordered, true, true, cs) != cudaSuccess)
                return FA_ERR_CUDA;
        }
    }
    if (tc && !tc2 && launch_compress_tc(s, make_cache(*cache), K, V, sbb, stride_t, stride_h, L, ordered, tc_rows, cs) != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

namespace {
// The argument checks of fa_compress_ex for one layer (no launch).
fa_status check_compress_args(const fa_layout* layout, const fa_cache* cache, const void* K, const void* V, int64_t stride_b,
                              int64_t stride_t, int64_t stride_h, int32_t L, uint32_t flags) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    if (L < 0 || (flags & ~(uint32_t)(FA_COMPRESS_ORDERED | FA_COMPRESS_FFT))) return FA_ERR_INVALID_ARG;
    if (L > 0 && (!K || !V || !aligned16(K) || !aligned16(V))) return FA_ERR_INVALID_ARG;
    if (L > 0 && (stride_t < layout->head_dim || stride_h < layout->head_dim || stride_b < 0)) return FA_ERR_INVALID_ARG;
    if ((stride_b | stride_t | stride_h) & 7) return FA_ERR_INVALID_ARG;
    const Dims s = make_dims(*layout);
    const int n_init = L < s.l_init ? L : s.l_init;
    const int n_local = (L - n_init) < s.l_local ? (L - n_init) : s.l_local;
    if (L - n_init - n_local > s.max_mid) return FA_ERR_CAPACITY;
    return FA_OK;
}
// True if fa_compress_ex would run this layer as the partition kernel (windows, counters, coefficients cleared) and the
// CTA-pair contraction, which also writes the kept-dim rows: the form that a call over several layers can overlap.
bool compress_is_pair_form(const fa_layout* layout, int64_t stride_b, int64_t stride_t, int64_t stride_h, int32_t L, uint32_t flags) {
    if (flags & FA_COMPRESS_FFT) return false;
    const Dims s = make_dims(*layout);
    const int n_init = L < s.l_init ? L : s.l_init;
    const int n_local = (L - n_init) < s.l_local ? (L - n_init) : s.l_local;
    const int64_t sbb = s.B > 1 ? stride_b : 0;
    return L > 0 && L - n_init - n_local >= 1024 && compress_tc_supported(s, layout->kv_dtype, sbb, stride_t, stride_h) &&
           compress_tc2_supported(s) && compress_tc2_gathers(s);
}
}  // namespace

fa_status fa_compress_layers(int32_t n_layers, const fa_layout* layouts, fa_cache* caches, const void* const* K,
                             const void* const* V, int64_t stride_b, int64_t stride_t, int64_t stride_h, int32_t L,
                             uint32_t flags, void* ws, size_t ws_bytes, void* stream) {
    if (n_layers < 0 || (n_layers > 0 && (!layouts || !caches || !K || !V))) return FA_ERR_INVALID_ARG;
    // every layer's arguments are checked before anything is enqueued
    bool pair_form = n_layers > 1;
    for (int i = 0; i < n_layers; ++i) {
        const fa_status st = check_compress_args(&layouts[i], &caches[i], K[i], V[i], stride_b, stride_t, stride_h, L, flags);
        if (st != FA_OK) return st;
        pair_form = pair_form && compress_is_pair_form(&layouts[i], stride_b, stride_t, stride_h, L, flags);
        // the overlapped form runs the layers' kernels side by side: their caches must not be one another's
        for (int j = 0; j < i && pair_form; ++j)
            if (caches[j].coef_k == caches[i].coef_k || caches[j].state == caches[i].state) pair_form = false;
    }
    if (!pair_form) {
        for (int i = 0; i < n_layers; ++i) {
            const fa_status st = fa_compress_ex(&layouts[i], &caches[i], K[i], V[i], stride_b, stride_t, stride_h, L, flags, ws, ws_bytes, stream);
            if (st != FA_OK) return st;
        }
        return FA_OK;
    }
    // All partition kernels first, each launched programmatically behind the one before (they touch different caches and
    // run side by side; each ends by waiting for its predecessor, so the end of the last implies the end of all); then
    // the contractions, likewise: the CTAs of layer i + 1 take the SMs that the first CTAs of layer i to finish
    // leave, and wait for layer i (hence for everything before it) only in front of their reductions.
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const bool ordered = (flags & FA_COMPRESS_ORDERED) != 0;
    for (int i = 0; i < n_layers; ++i) {
        const Dims s = make_dims(layouts[i]);
        if (launch_compress(s, make_cache(caches[i]), layouts[i].kv_dtype, K[i], V[i], stride_b, stride_t, stride_h, L, false, ordered, false,
                            true, cs, i > 0) != cudaSuccess)
            return FA_ERR_CUDA;
    }
    for (int i = 0; i < n_layers; ++i) {
        const Dims s = make_dims(layouts[i]);
        const int64_t sbb = s.B > 1 ? stride_b : 0;
        if (launch_compress_tc2(s, make_cache(caches[i]), K[i], V[i], sbb, stride_t, stride_h, L, ordered, true, cs) != cudaSuccess) {
            // the cluster launch was refused: finish this and the remaining layers one by one (each call redoes its layer in full)
            cudaGetLastError();
            for (int j = i; j < n_layers; ++j) {
                const fa_status st = fa_compress_ex(&layouts[j], &caches[j], K[j], V[j], stride_b, stride_t, stride_h, L, flags, ws, ws_bytes, stream);
                if (st != FA_OK) return st;
            }
            return FA_OK;
        }
    }
    return FA_OK;
}

fa_status fa_compress(const fa_layout* layout, fa_cache* cache, const void* K, const void* V, int64_t stride_b,
                      int64_t stride_t, int64_t stride_h, int32_t L, void* ws, size_t ws_bytes, void* stream) {
    return fa_compress_ex(layout, cache, K, V, stride_b, stride_t, stride_h, L, 0u, ws, ws_bytes, stream);
}

fa_status fa_compress_ragged(const fa_layout* layout, fa_cache* cache, const void* K, const void* V, int64_t stride_b,
                             int64_t stride_t, int64_t stride_h, const int32_t* lengths, void* ws, size_t ws_bytes,
                             void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    if (!lengths || stride_b < 0) return FA_ERR_INVALID_ARG;
    // every batch row is a one-row cache of its own: same index sets and status word, its own slices
    fa_layout one = *layout;
    one.batch = 1;
    fa_cache_sizes sz;
    st = fa_cache_sizes_of(&one, &sz);
    if (st != FA_OK) return st;
    const size_t eb = elt_bytes(layout->kv_dtype);
    for (int b = 0; b < layout->batch; ++b) {
        if (lengths[b] < 0) return FA_ERR_INVALID_ARG;
        fa_cache row = *cache;
        auto at = [&](void* p, size_t bytes) -> void* { return p ? static_cast<char*>(p) + (size_t)b * bytes : nullptr; };
        row.k_init = at(cache->k_init, sz.k_init);     row.v_init = at(cache->v_init, sz.v_init);
        row.k_local = at(cache->k_local, sz.k_local);  row.v_local = at(cache->v_local, sz.v_local);
        row.k_mid = at(cache->k_mid, sz.k_mid);        row.v_mid = at(cache->v_mid, sz.v_mid);
        row.coef_k = static_cast<float*>(at(cache->coef_k, sz.coef_k));
        row.coef_v = static_cast<float*>(at(cache->coef_v, sz.coef_v));
        row.state = static_cast<int32_t*>(at(cache->state, sz.state));
        const char* Kb = static_cast<const char*>(K) + (size_t)b * (size_t)stride_b * eb;
        const char* Vb = static_cast<const char*>(V) + (size_t)b * (size_t)stride_b * eb;
        st = fa_compress(&one, &row, lengths[b] ? Kb : (K ? Kb : nullptr), lengths[b] ? Vb : (V ? Vb : nullptr), stride_b, stride_t,
                         stride_h, lengths[b], ws, ws_bytes, stream);
        if (st != FA_OK) return st;
    }
    return FA_OK;
}

fa_status fa_append(const fa_layout* layout, fa_cache* cache, const void* k_new, const void* v_new, void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return FA_ERR_INVALID_ARG;
    if (launch_append(make_dims(*layout), make_cache(*cache), layout->kv_dtype, k_new, v_new,
                      static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return FA_ERR_CUDA;
    return FA_OK;
}

fa_status fa_decode_attention(const fa_layout* layout, const fa_cache* cache, const void* q, void* out, void* ws,
                              size_t ws_bytes, void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    if (!q || !out || !aligned16(q) || !aligned16(out)) return FA_ERR_INVALID_ARG;
    DecodePlan p;
    st = plan_decode(*layout, &p);
    if (st != FA_OK) return st;
    if (!ws || !aligned16(ws) || ws_bytes < p.total) return FA_ERR_WORKSPACE;
    Dims s = make_dims(*layout);
    CacheDev c = make_cache(*cache);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    char* w = static_cast<char*>(ws);
    if (p.fused) {
        const cudaError_t err = launch_decode_fft(s, c, layout->kv_dtype, p, q, out, w, nullptr, nullptr, cs);
        if (err == cudaSuccess) return FA_OK;
        if (err != cudaErrorCooperativeLaunchTooLarge) return FA_ERR_CUDA;
        // the device cannot hold all CTAs at once right now (SMs taken by another client): three kernels instead
        cudaGetLastError();
        fa_layout split = *layout;
        split.decode_algo = FA_DECODE_FFT_SPLIT;
        return fa_decode_attention(&split, cache, q, out, ws, ws_bytes, stream);
    }
    if (launch_decode_prologue(s, c, layout->kv_dtype, p, q, w, cs) != cudaSuccess) return FA_ERR_CUDA;
    if (p.algo == FA_DECODE_FFT) {
        if (launch_decode_fft(s, c, layout->kv_dtype, p, q, out, w, nullptr, nullptr, cs) != cudaSuccess) return FA_ERR_CUDA;
    } else {
        if (launch_decode_direct(s, c, layout->kv_dtype, p, q, w, cs) != cudaSuccess) return FA_ERR_CUDA;
    }
    if (launch_decode_epilogue(s, c, layout->kv_dtype, p, out, w, cs) != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

}  // extern "C"

constexpr int kStepFusedMinParts = 8;

// fa_decode_step.  Where the decode call is the fused kernel with one pass and many parts per head, the push
// rides on that launch; otherwise the two calls are made one after the other.
static fa_status decode_step_impl(const fa_layout* layout, fa_cache* cache, const void* q, const void* k_new, const void* v_new,
                                  void* out, void* ws, size_t ws_bytes, void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    st = check_cache(layout, cache);
    if (st != FA_OK) return st;
    if (!q || !out || !aligned16(q) || !aligned16(out)) return FA_ERR_INVALID_ARG;
    if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return FA_ERR_INVALID_ARG;
    DecodePlan p;
    st = plan_decode(*layout, &p);
    if (st != FA_OK) return st;
    if (!ws || !aligned16(ws) || ws_bytes < p.total) return FA_ERR_WORKSPACE;
    Dims s = make_dims(*layout);
    // The push rides on the decode launch where a head has many parts (each then updates a small slice of the
    // coefficient rows as it streams them for u and for the output product).  With few parts per head the
    // stand-alone append kernel, which spreads the coefficient update over the whole device, is faster
    // (measured: batch 8 MHA 22 us against 35 us inside the decode kernel, batch 4 at 128K 22 against 64).
    // Whether the device can hold all parts at once is asked before anything is enqueued: nothing to undo.
    if (p.fused && p.n_pass == 1 && p.n_part >= kStepFusedMinParts && cooperative_launch_supported() && decode_fft_launchable(s, p)) {
        const cudaError_t err = launch_decode_fft(s, make_cache(*cache), layout->kv_dtype, p, q, out, static_cast<char*>(ws), k_new, v_new,
                                                  static_cast<cudaStream_t>(stream));
        if (err == cudaSuccess) return FA_OK;
        if (err != cudaErrorCooperativeLaunchTooLarge) return FA_ERR_CUDA;
        cudaGetLastError();                                  // refused before anything ran (SMs taken by another client): the two calls
    }
    st = fa_append(layout, cache, k_new, v_new, stream);
    if (st != FA_OK) return st;
    return fa_decode_attention(layout, cache, q, out, ws, ws_bytes, stream);
}

extern "C" {

fa_status fa_decode_step(const fa_layout* layout, fa_cache* cache, const void* q, const void* k_new, const void* v_new,
                         void* out, void* ws, size_t ws_bytes, void* stream) {
    return decode_step_impl(layout, cache, q, k_new, v_new, out, ws, ws_bytes, stream);
}

fa_status fa_decode_step_layers(int32_t n_layers, const fa_layout* layouts, fa_cache* caches, const void* const* q,
                                const void* const* k_new, const void* const* v_new, void* const* out, void* ws,
                                size_t ws_bytes, void* stream) {
    if (n_layers < 0 || (n_layers > 0 && (!layouts || !caches || !q || !k_new || !v_new || !out))) return FA_ERR_INVALID_ARG;
    // every layer's arguments are checked before anything is enqueued: a bad layer leaves all caches untouched
    for (int i = 0; i < n_layers; ++i) {
        fa_status st = check_layout(&layouts[i]);
        if (st != FA_OK) return st;
        st = check_cache(&layouts[i], &caches[i]);
        if (st != FA_OK) return st;
        const void* ptrs[] = {q[i], k_new[i], v_new[i], out[i]};
        for (const void* p : ptrs) if (!p || !aligned16(p)) return FA_ERR_INVALID_ARG;
        DecodePlan p;
        st = plan_decode(layouts[i], &p);
        if (st != FA_OK) return st;
        if (!ws || !aligned16(ws) || ws_bytes < p.total) return FA_ERR_WORKSPACE;
    }
    for (int i = 0; i < n_layers; ++i) {
        const fa_status st = decode_step_impl(&layouts[i], &caches[i], q[i], k_new[i], v_new[i], out[i], ws, ws_bytes, stream);
        if (st != FA_OK) return st;
    }
    return FA_OK;
}

size_t fa_step_staging_bytes(const fa_layout* layout) {
    if (check_layout(layout) != FA_OK) return 0;
    size_t eb = elt_bytes(layout->kv_dtype);
    size_t qb = align_up((size_t)layout->batch * layout->n_q_heads * layout->head_dim * eb, 256);
    size_t kb = align_up((size_t)layout->batch * layout->n_kv_heads * layout->head_dim * eb, 256);
    return 2 * qb + 2 * kb;
}

fa_status fa_decode_step_host(const fa_layout* layout, fa_cache* cache, const void* q_host, const void* k_new_host,
                              const void* v_new_host, void* out_host, void* staging, void* ws, size_t ws_bytes,
                              void* stream) {
    fa_status st = check_layout(layout);
    if (st != FA_OK) return st;
    if (!q_host || !out_host || !staging || !aligned16(staging)) return FA_ERR_INVALID_ARG;
    if ((k_new_host == nullptr) != (v_new_host == nullptr)) return FA_ERR_INVALID_ARG;
    size_t eb = elt_bytes(layout->kv_dtype);
    size_t q_bytes = (size_t)layout->batch * layout->n_q_heads * layout->head_dim * eb;
    size_t k_bytes = (size_t)layout->batch * layout->n_kv_heads * layout->head_dim * eb;
    size_t qb = align_up(q_bytes, 256), kb = align_up(k_bytes, 256);
    char* base = static_cast<char*>(staging);
    char *q_d = base, *o_d = base + qb, *k_d = base + 2 * qb, *v_d = base + 2 * qb + kb;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const void *q_v = nullptr, *k_v = nullptr, *v_v = nullptr;
    if (k_new_host && q_bytes % 16 == 0 && k_bytes % 16 == 0 && aligned16(q_host) && aligned16(k_new_host) && aligned16(v_new_host)) {
        q_v = device_view_of_host(q_host);
        k_v = device_view_of_host(k_new_host);
        v_v = device_view_of_host(v_new_host);
    }
    // a pinned result buffer is written by the decode kernel itself (posted writes over the bus)
    void* out_v = aligned16(out_host) ? const_cast<void*>(device_view_of_host(out_host)) : nullptr;
    if (out_v) o_d = static_cast<char*>(out_v);
    if (q_v && k_v && v_v) {
        // pinned inputs: one staging kernel reads them over the bus (measured faster than three copy
        // operations, and than letting every CTA of the step read the host buffers in place)
        const int nq = (int)(q_bytes / 16), nk = (int)(k_bytes / 16);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((nq + 2 * nk + 255) / 256);
        cfg.blockDim = dim3(256);
        cfg.stream = cs;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, stage_inputs_kernel, static_cast<const uint4*>(q_v), static_cast<const uint4*>(k_v),
                               static_cast<const uint4*>(v_v), reinterpret_cast<uint4*>(q_d), reinterpret_cast<uint4*>(k_d),
                               reinterpret_cast<uint4*>(v_d), nq, nk) != cudaSuccess)
            return FA_ERR_CUDA;
        st = fa_decode_step(layout, cache, q_d, k_d, v_d, o_d, ws, ws_bytes, stream);
    } else if (k_new_host) {
        if (cudaMemcpyAsync(q_d, q_host, q_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return FA_ERR_CUDA;
        if (cudaMemcpyAsync(k_d, k_new_host, k_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return FA_ERR_CUDA;
        if (cudaMemcpyAsync(v_d, v_new_host, k_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return FA_ERR_CUDA;
        st = fa_decode_step(layout, cache, q_d, k_d, v_d, o_d, ws, ws_bytes, stream);
    } else {
        if (cudaMemcpyAsync(q_d, q_host, q_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return FA_ERR_CUDA;
        st = fa_decode_attention(layout, cache, q_d, o_d, ws, ws_bytes, stream);
    }
    if (st != FA_OK) return st;
    if (!out_v && cudaMemcpyAsync(out_host, o_d, q_bytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

int fa_launch_count(const fa_layout* layout, int what) {
    if (check_layout(layout) != FA_OK) return 0;
    switch (what) {
        case 0: return 2;   // partition/gather + coefficient kernel (memsets not counted)
        case 1: return 1;
        case 2: {           // one fused kernel, or prologue + main + epilogue
            DecodePlan p;
            if (plan_decode(*layout, &p) != FA_OK) return 0;
            return p.fused ? 1 : 3;
        }
        case 3: {           // fa_decode_step: the fused decode kernel alone, or fa_append + fa_decode_attention
            DecodePlan p;
            if (plan_decode(*layout, &p) != FA_OK) return 0;
            return (p.fused && p.n_pass == 1 && p.n_part >= kStepFusedMinParts) ? 1 : 1 + (p.fused ? 1 : 3);
        }
        case 4: {           // plan query: the split build of the fused decode kernel
            DecodePlan p;
            if (plan_decode(*layout, &p) != FA_OK) return 0;
            return (p.fused && p.split) ? 1 : 0;
        }
        case 5: {           // plan query: residue classes per batch of the transform kernel (0: the direct kernel)
            DecodePlan p;
            if (plan_decode(*layout, &p) != FA_OK) return 0;
            return p.algo == FA_DECODE_FFT ? p.nb : 0;
        }
        case 6: {           // plan query: CTAs per (batch, KV head, pass) of the decode kernel
            DecodePlan p;
            if (plan_decode(*layout, &p) != FA_OK) return 0;
            return p.n_part;
        }
        default: return 0;
    }
}

const char* fa_status_string(fa_status s) {
    switch (s) {
        case FA_OK: return "ok";
        case FA_ERR_INVALID_ARG: return "invalid argument";
        case FA_ERR_UNSUPPORTED: return "unsupported layout";
        case FA_ERR_CAPACITY: return "middle segment is full";
        case FA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case FA_ERR_CUDA: return "CUDA runtime error";
        case FA_ERR_TIMEOUT: return "bounded device wait timed out";
        case FA_ERR_INDEX: return "index sets are not a sorted disjoint cover of the head dims";
    }
    return "unknown status";
}

int fa_version(void) { return 100; }

}  // extern "C"
