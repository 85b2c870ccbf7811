// fa_select_dims, tensor-core reconstruction (Sec. 3.4) for bf16 prefill tensors on sm_100a: the middle tokens
// rebuilt from the coefficients of every dimension, X~ = F^T (W C), as a dense [L_mid x M] x [M x N]
// contraction on the 5th-generation tensor cores (tcgen05.mma, bf16 x bf16 -> fp32 accumulators in tensor
// memory), and the squared error against the prefill summed per dimension as the accumulators are read back.
//
// It mirrors the compression kernel with the roles of tokens and coefficient rows exchanged.  One CTA owns 128
// middle tokens of HP KV heads, K and V together (N = 2 d columns per head); the coefficient axis is the
// contraction axis, cut into blocks of 64 rows.  Per block and pipeline stage:
//   * warp 0 (one lane) loads the [64 rows x 64 dims] boxes of the weighted coefficients W C (rounded to bf16 by
//     weighted_coef_kernel, laid out [B][M][H_kv][d] so that they tile like a prefill tensor) with TMA;
//   * warps 2-9 generate the 128 x 64 tile of F^T: a thread owns one token and 16 frequencies, starts from the
//     exact integer phase of its first two frequencies and rotates by two frequencies at a time (packed fp32 pairs);
//   * warp 1 (one lane) issues four tcgen05.mma (K = 16 each) per head and commits the stage back.
// The basis and W C enter the tensor core as bf16 (as the basis of the compression does), so a dimension that the
// coefficients rebuild exactly still shows an error of about 1e-6 of its energy; errors above that floor are
// those of the fp32 path.  Every wait is bounded; tensor memory is freed on every path.
#include "fa_umma.cuh"

namespace fa {
namespace {

using bf16 = __nv_bfloat16;
using namespace umma;

constexpr int kRT = 128;          // tokens per CTA (accumulator rows)
constexpr int kRK = 64;           // coefficient rows per pipeline stage
constexpr int kGenWarpsR = 8;      // basis generators (and epilogue)
constexpr int kThreadsR = 64 + 32 * kGenWarpsR;

// wk / wv [B][M][Hkv][d] = bf16(w_m * C[b][h][m][e]) from the fp32 coefficients [B][Hkv][M][d] of a cache that
// compresses every dimension.
__global__ void weighted_coef_kernel(Dims s, const float* __restrict__ coef_k, const float* __restrict__ coef_v,
                                     bf16* __restrict__ wk, bf16* __restrict__ wv) {
    const int d4 = s.d >> 2;
    const size_t n = (size_t)s.B * s.M * s.Hkv * d4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < 2 * n; i += (size_t)gridDim.x * blockDim.x) {
        const int side = i >= n;
        size_t r = side ? i - n : i;
        const int v = (int)(r % d4); r /= d4;
        const int h = (int)(r % s.Hkv); r /= s.Hkv;
        const int m = (int)(r % s.M);
        const int b = (int)(r / s.M);
        const float w = recon_weight(s.norm, m, s.k, s.T);
        const float4 x = *reinterpret_cast<const float4*>((side ? coef_v : coef_k) + ((((size_t)b * s.Hkv + h) * s.M + m) * s.d) + 4 * v);
        const __nv_bfloat162 lo = __floats2bfloat162_rn(w * x.x, w * x.y), hi = __floats2bfloat162_rn(w * x.z, w * x.w);
        uint2 o;
        o.x = *reinterpret_cast<const uint32_t*>(&lo);
        o.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>((side ? wv : wk) + ((((size_t)b * s.M + m) * s.Hkv + h) * s.d) + 4 * v) = o;
    }
}

// D = head dim (64 or 128): N = 2 D accumulator columns per KV head; HP heads share one CTA and one generated
// basis tile (HP * N <= 512 tensor-memory columns).  grid (ceil(n_mid / 128), Hkv / HP, B).
// K, V: the prefill tensors (element strides sb, st, sh); sq [B][Hkv][2][D]: sums of squared errors (zeroed by the caller).
template <int D, int HP>
__global__ void __launch_bounds__(kThreadsR, 1) reconstruct_tc_kernel(const __grid_constant__ CUtensorMap tmWK,
                                                                      const __grid_constant__ CUtensorMap tmWV, Dims s,
                                                                      const bf16* __restrict__ K, const bf16* __restrict__ V,
                                                                      int64_t sb, int64_t st, int64_t sh, int n_init, int n_mid,
                                                                      float* __restrict__ sq, int32_t* status) {
    constexpr int N = 2 * D;
    constexpr int kABytes = kRT * kRK * 2;                 // 16 KB basis tile
    constexpr int kBoxBytes = kRK * 64 * 2;                // 8 KB per [64 rows x 64 dims] box
    constexpr int kBBytes1 = (N / 64) * kBoxBytes;          // one head
    constexpr int kBBytes = HP * kBBytes1;
    constexpr int kStageBytesR = kABytes + kBBytes;
    constexpr int kStagesR = (200 * 1024) / kStageBytesR < 4 ? (200 * 1024) / kStageBytesR : 4;
    constexpr uint32_t kTmemCols = HP * N;
    // bf16 x bf16 -> fp32, A K-major, B MN-major, N and M of the instruction
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kRT >> 4) << 24);
    extern __shared__ unsigned char smem_unaligned[];
    unsigned char* smem = smem_unaligned + ((1024u - (smem_u32(smem_unaligned) & 1023u)) & 1023u);
    unsigned char* stage0 = smem;                          // kStagesR x (A | B boxes), 1024-byte aligned
    // one barrier per stage for the basis tile (the generator warps) and the boxes (the producer's expect_tx): the
    // thread that issues the MMAs pays for every barrier it passes
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStagesR * kStageBytesR);
    uint64_t* empty = full + kStagesR;
    uint64_t* acc_ready = empty + kStagesR;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_ready + 1);
    volatile int* fail = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* err_s = reinterpret_cast<float*>(tmem_slot + 4);   // [HP][2][D] squared errors of this CTA's tokens

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j_tile = blockIdx.x * kRT, h0 = blockIdx.y * HP, b = blockIdx.z;
    const int nkb = s.M / kRK;

    if (tid == 0) {
        for (int i = 0; i < kStagesR; ++i) { mbar_init(full + i, kGenWarpsR + 1); mbar_init(empty + i, 1); }
        mbar_init(acc_ready, 1);
        *fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < HP * N; i += kThreadsR) err_s[i] = 0.f;
    if (warp == 1) {                                       // tensor memory: HP * N fp32 columns x 128 lanes
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer: B operand = 64 rows of W C, K dims then V dims, per head ----------------
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int stg = kb % kStagesR;
                if (kb >= kStagesR && !mbar_wait(empty + stg, ((kb / kStagesR) - 1) & 1, fail, status)) break;
                unsigned char* bdst = stage0 + (size_t)stg * kStageBytesR + kABytes;
                mbar_expect_tx(full + stg, (uint32_t)kBBytes);
#pragma unroll
                for (int hh = 0; hh < HP; ++hh)
#pragma unroll
                    for (int bx = 0; bx < N / 64; ++bx) {
                        const CUtensorMap* tm = bx < D / 64 ? &tmWK : &tmWV;
                        const int dim0 = (bx % (D / 64)) * 64;
                        tma_load_4d(bdst + hh * kBBytes1 + bx * kBoxBytes, tm, dim0, h0 + hh, kb * kRK, b, full + stg);
                    }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int stg = kb % kStagesR;
                const uint32_t par = (kb / kStagesR) & 1;
                if (!mbar_wait(full + stg, par, fail, status)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(stage0 + (size_t)stg * kStageBytesR);
                const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                for (int ks = 0; ks < kRK / 16; ++ks) {
                    // A: K-major, rows of 128 bytes (64 coefficient rows of one token), 8-token groups 1024 bytes apart
                    const uint64_t adesc = umma_desc(a_addr + ks * 32, 1, 1024 >> 4);
                    // B: MN-major, 64 dims per 128-byte row, 8-row groups 1024 bytes apart, next 64 dims one box further
#pragma unroll
                    for (int hh = 0; hh < HP; ++hh) {
                        const uint64_t bdesc = umma_desc(b_addr + hh * kBBytes1 + ks * 2048, kBoxBytes >> 4, 1024 >> 4);
                        umma_bf16(tmem_base + hh * N, adesc, bdesc, kIdesc, (kb > 0 || ks > 0) ? 1u : 0u);
                    }
                }
                umma_commit(empty + stg);                  // frees the stage when these MMAs have read it
            }
            umma_commit(acc_ready);
        }
    } else {
        // ---------------- basis generators: A operand = F^T for this CTA's tokens ----------------
        const int t = tid - 64;                            // 0 .. 255
        const int r = t >> 1, hq = t & 1;                  // token row of the tile, half of the 32 frequencies of a block
        const unsigned j = (unsigned)(j_tile + r);
        const float inv_T = 1.0f / (float)s.T;
        auto angle = [&](unsigned phase) {                 // 2 pi phase / T in [-pi, pi)
            const float f = (float)phase * inv_T;
            return 6.283185307179586f * (f - (f >= 0.5f ? 1.0f : 0.0f));
        };
        // rotation by two frequencies for this token, as splat pairs
        unsigned long long CS2, SN2, NSN2;
        {
            const float a = angle((2u * j) % (unsigned)s.T);
            const float c2 = __cosf(a), s2 = __sinf(a);
            asm("mov.b64 %0, {%1,%1};" : "=l"(CS2) : "f"(c2));
            asm("mov.b64 %0, {%1,%1};" : "=l"(SN2) : "f"(s2));
            asm("mov.b64 %0, {%1,%1};" : "=l"(NSN2) : "f"(-s2));
        }
        const uint32_t row_off = (uint32_t)((r >> 3) * 1024 + (r & 7) * 128);
        for (int kb = 0; kb < nkb; ++kb) {
            const int stg = kb % kStagesR;
            if (kb >= kStagesR && !mbar_wait(empty + stg, ((kb / kStagesR) - 1) & 1, fail, status)) break;
            unsigned char* a_dst = stage0 + (size_t)stg * kStageBytesR;
            const unsigned n0 = (unsigned)(kb * (kRK / 2) + 16 * hq);   // first frequency of this thread's run
            // packed phasors of frequencies (n0, n0 + 1): C = (cos, cos), S = (sin, sin), exact integer phases
            unsigned long long C, S;
            {
                const float aa = angle((n0 * j) % (unsigned)s.T);          // the products stay below 2^32 (checked on the host)
                const float ab = angle(((n0 + 1) * j) % (unsigned)s.T);
                asm("mov.b64 %0, {%1,%2};" : "=l"(C) : "f"(__cosf(aa)), "f"(__cosf(ab)));
                asm("mov.b64 %0, {%1,%2};" : "=l"(S) : "f"(__sinf(aa)), "f"(__sinf(ab)));
            }
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {               // 4 frequencies (cos, sin interleaved) = one 16-byte chunk of the row
                uint32_t w[4];
#pragma unroll
                for (int i2 = 0; i2 < 2; ++i2) {
                    float c0, c1, s0, s1;
                    asm("mov.b64 {%0,%1}, %2;" : "=f"(c0), "=f"(c1) : "l"(C));
                    asm("mov.b64 {%0,%1}, %2;" : "=f"(s0), "=f"(s1) : "l"(S));
                    const __nv_bfloat162 pa = __floats2bfloat162_rn(c0, s0);   // rows 2 n, 2 n + 1
                    const __nv_bfloat162 pb = __floats2bfloat162_rn(c1, s1);   // rows 2 n + 2, 2 n + 3
                    w[2 * i2] = *reinterpret_cast<const uint32_t*>(&pa);
                    w[2 * i2 + 1] = *reinterpret_cast<const uint32_t*>(&pb);
                    // advance both phasors by two frequencies: C' = C cs2 - S sn2, S' = S cs2 + C sn2
                    unsigned long long tC, tS, nC, nS;
                    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(tC) : "l"(C), "l"(CS2));
                    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(tS) : "l"(S), "l"(CS2));
                    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(nC) : "l"(S), "l"(NSN2), "l"(tC));
                    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(nS) : "l"(C), "l"(SN2), "l"(tS));
                    C = nC;
                    S = nS;
                }
                const int chunk = 4 * hq + ch;
                *reinterpret_cast<uint4*>(a_dst + row_off + ((chunk ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic stores -> visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(full + stg);
        }
        // ---------------- epilogue: (accumulator - prefill)^2 summed over the tokens, per dim ----------------
        const bool ok = mbar_wait(acc_ready, 0, fail, status);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            const int lane_grp = warp & 3;                 // a warp reads tensor-memory lanes 32 (warp % 4) ...
            const int col_half = (warp - 2) >> 2;          // two warps share a lane group: one column half each
            constexpr int kHalf = (int)kTmemCols / 2;
            const int jt = j_tile + lane_grp * 32 + lane;  // this thread's token
            const bool live = jt < n_mid;
#pragma unroll 1
            for (int col0 = col_half * kHalf; col0 < (col_half + 1) * kHalf; col0 += 32) {
                const int hh = col0 / N, hcol0 = col0 - hh * N;
                const bool is_k = hcol0 < D;               // a block of 32 columns lies within K's dims or within V's
                const int dim0 = is_k ? hcol0 : hcol0 - D;
                float v[32];
                tmem_ld32(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)col0, v);
                if (live) {
                    const bf16* x = (is_k ? K : V) + (size_t)b * sb + (size_t)(n_init + jt) * st + (size_t)(h0 + hh) * sh + dim0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(x) + q);
                        const uint32_t wds[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float lo = __uint_as_float(wds[i] << 16), hi = __uint_as_float(wds[i] & 0xffff0000u);
                            const float d0 = v[8 * q + 2 * i] - lo, d1 = v[8 * q + 2 * i + 1] - hi;
                            v[8 * q + 2 * i] = d0 * d0;
                            v[8 * q + 2 * i + 1] = d1 * d1;
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0.f;
                }
                // sum over the 32 tokens of the warp: after the five exchange steps lane l holds column col0 + l
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) {
                    const bool up = (lane & off) != 0;
#pragma unroll
                    for (int i = 0; i < off; ++i) {
                        const float send = up ? v[i] : v[i + off];
                        const float keep = up ? v[i + off] : v[i];
                        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                    }
                }
                atomicAdd(err_s + col0 + lane, v[0]);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    for (int i = tid; i < HP * N; i += kThreadsR) {
        const int hh = i / N, side = (i - hh * N) / D, e = i % D;
        atomicAdd(sq + (((size_t)b * s.Hkv + h0 + hh) * 2 + side) * D + e, err_s[i]);
    }
}

// 4-D view (dim, head, row, batch) of the weighted coefficients [B][M][Hkv][d]; box = 64 dims x 64 rows.
bool make_coef_map(CUtensorMap* tm, const void* base, const Dims& s) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)s.d, (cuuint64_t)s.Hkv, (cuuint64_t)s.M, (cuuint64_t)s.B};
    cuuint64_t strides[3] = {(cuuint64_t)s.d * 2, (cuuint64_t)s.Hkv * s.d * 2, (cuuint64_t)s.M * s.Hkv * s.d * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)kRK, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int HP>
cudaError_t launch_rec_t(const CUtensorMap& tmWK, const CUtensorMap& tmWV, const Dims& s, const void* K, const void* V, int64_t sb,
                         int64_t st, int64_t sh, int n_init, int n_mid, float* sq, int32_t* status, cudaStream_t stream) {
    constexpr int N = 2 * D;
    constexpr size_t stage = (size_t)kRT * kRK * 2 + (size_t)HP * (N / 64) * kRK * 64 * 2;
    constexpr size_t n_stages = (200 * 1024) / stage < 4 ? (200 * 1024) / stage : 4;
    const size_t smem = n_stages * stage + 8 * (3 * n_stages + 1) + 16 + sizeof(float) * HP * N + 64 + 1024;
    cudaError_t err = ensure_dynamic_smem(reconstruct_tc_kernel<D, HP>, smem);
    if (err != cudaSuccess) return err;
    const dim3 grid((n_mid + kRT - 1) / kRT, s.Hkv / HP, s.B);
    reconstruct_tc_kernel<D, HP><<<grid, kThreadsR, smem, stream>>>(tmWK, tmWV, s, static_cast<const bf16*>(K), static_cast<const bf16*>(V),
                                                                   sb, st, sh, n_init, n_mid, sq, status);
    return cudaGetLastError();
}

}  // namespace

// True if the tensor-core reconstruction serves this layout, these strides and these base addresses.
bool reconstruct_tc_supported(const Dims& s, int dtype, const void* K, const void* V, int64_t sb, int64_t st, int64_t sh, int n_mid) {
    if (dtype != FA_BF16) return false;
    if (s.d != 64 && s.d != 128) return false;
    if (s.M % kRK != 0) return false;
    if ((sh % 8) || (st % 8) || (sb % 8)) return false;
    if ((reinterpret_cast<uintptr_t>(K) & 15u) || (reinterpret_cast<uintptr_t>(V) & 15u)) return false;
    if ((unsigned long long)(s.M / 2 + 1) * (unsigned long long)(n_mid + kRT) >= (1ull << 32)) return false;   // phase products stay in 32 bits
    return encode_tiled_fn() != nullptr;
}

// Bytes of the two weighted-coefficient tensors (K side, then V side; each 256-byte aligned).
size_t reconstruct_tc_scratch_bytes(const Dims& s) {
    const size_t one = ((size_t)s.B * s.M * s.Hkv * s.d * 2 + 255) / 256 * 256;
    return 2 * one;
}

// sq [B][Hkv][2][d] += sum over the middle tokens of (x~ - x)^2, from the fp32 coefficients coef_k / coef_v
// [B][Hkv][M][d] of all d dims.  scratch: reconstruct_tc_scratch_bytes(s) bytes, 256-byte aligned.
cudaError_t launch_reconstruct_tc(const Dims& s, const float* coef_k, const float* coef_v, const void* K, const void* V, int64_t sb,
                                  int64_t st, int64_t sh, int n_init, int n_mid, float* sq, int32_t* status, void* scratch,
                                  cudaStream_t stream) {
    if (n_mid <= 0) return cudaSuccess;
    bf16* wk = static_cast<bf16*>(scratch);
    bf16* wv = reinterpret_cast<bf16*>(static_cast<char*>(scratch) + reconstruct_tc_scratch_bytes(s) / 2);
    const size_t n4 = (size_t)s.B * s.M * s.Hkv * (s.d >> 2) * 2;
    const int blocks = (int)((n4 + 255) / 256 < 148 * 16 ? (n4 + 255) / 256 : 148 * 16);
    weighted_coef_kernel<<<blocks, 256, 0, stream>>>(s, coef_k, coef_v, wk, wv);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    CUtensorMap tmWK, tmWV;
    if (!make_coef_map(&tmWK, wk, s) || !make_coef_map(&tmWV, wv, s)) return cudaErrorInvalidValue;
    const bool pair = s.Hkv % 2 == 0;                        // two heads share a CTA and its basis tile
    if (s.d == 128)
        return pair ? launch_rec_t<128, 2>(tmWK, tmWV, s, K, V, sb, st, sh, n_init, n_mid, sq, status, stream)
                    : launch_rec_t<128, 1>(tmWK, tmWV, s, K, V, sb, st, sh, n_init, n_mid, sq, status, stream);
    return pair ? launch_rec_t<64, 2>(tmWK, tmWV, s, K, V, sb, st, sh, n_init, n_mid, sq, status, stream)
                : launch_rec_t<64, 1>(tmWK, tmWV, s, K, V, sb, st, sh, n_init, n_mid, sq, status, stream);
}

}  // namespace fa
