// fa_decode_attention (Eq.6), DIRECT main kernel: per token of the middle
//   s_j = q_u . K^mu_j + sum_m F[m][j] u_g[m];  online softmax;  o^u += p_j V^mu_j;
//   z[m] += p_j F[m][j];  window tokens: ordinary attention in the same softmax.
// The M basis terms of every token are summed one by one (any period, any class count):
// the reference of the GPU side and the fallback of the transform kernel.
#include "fa_common.cuh"
#include "fa_decode_ws.cuh"

namespace fa {


// ------------------------------------------------------------- direct main --
// grid (n_split, Hkv * n_pass, B), 256 threads; one thread per token of a 256-token tile.
constexpr int kTile = 256;

template <int GH>
struct RunStat {
    float m[GH];   // running max, log2 units
    float l[GH];   // running sum of p
};

// Block-wide max / sum of GH values per thread; result broadcast to every thread.
template <int GH, bool IS_MAX>
__device__ __forceinline__ void block_reduce(float (&v)[GH], float* red_s /* [8][GH] */) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int g = 0; g < GH; ++g) {
        float r = IS_MAX ? warp_max(v[g]) : warp_sum(v[g]);
        if (lane == 0) red_s[warp * GH + g] = r;
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < GH; ++g) {
        float r = red_s[g];
#pragma unroll
        for (int w = 1; w < 8; ++w) r = IS_MAX ? fmaxf(r, red_s[w * GH + g]) : r + red_s[w * GH + g];
        v[g] = r;
    }
    __syncthreads();
}

template <typename KV, int GH>
__global__ void __launch_bounds__(256) decode_direct_kernel(Dims s, CacheDev c, DecodePlan p, const KV* __restrict__ q,
                                                            char* wsp) {
    extern __shared__ float sm[];
    Ws ws = ws_view(wsp, p);
    const int split = blockIdx.x;
    const int h = blockIdx.y / p.n_pass, pass = blockIdx.y % p.n_pass;
    const int b = blockIdx.z;
    const int g_first = h * s.G + pass * GH;                 // first query head of this CTA
    const int ng = min(GH, s.G - pass * GH);
    const int tid = threadIdx.x;

    float* q_s = sm;                          // [GH][d]   scale * log2e * q, natural order
    float* qf_s = q_s + GH * s.d;             // [GH][nfk] the same gathered at D^ku
    float* u_s = qf_s + GH * s.nfk;           // [GH][M]
    float* z_s = u_s + GH * s.M;              // [GH][M]
    float* p_s = z_s + GH * s.M;              // [GH][kTile]
    float* red_s = p_s + GH * kTile;          // [8][GH]
    float* o_s = red_s + 8 * GH;              // [GH][d]  final reduce
    float* acc_s = o_s + GH * s.d;            // [256][GH] cross-thread reduce of the output accumulators

    const int n_init = c.state[kStateStride * b + 0], n_local = c.state[kStateStride * b + 1];
    const int n_mid = min(c.state[kStateStride * b + 2], s.max_mid), head = c.state[kStateStride * b + 3];
    const int32_t* idf_k = c.idx_full_k + (size_t)h * s.nfk;
    const int32_t* idf_v = c.idx_full_v + (size_t)h * s.nfv;

    for (int i = tid; i < GH * s.d; i += blockDim.x) {
        int g = i / s.d, e = i - g * s.d;
        q_s[i] = g < ng ? ld_f(q + ((size_t)b * s.Hq + g_first + g) * s.d + e) * s.scale * kLog2e : 0.f;
        o_s[i] = 0.f;
    }
    for (int i = tid; i < GH * s.M; i += blockDim.x) {
        int g = i / s.M, m = i - g * s.M;
        u_s[i] = (g < ng && s.dck > 0) ? ws.u[((size_t)b * s.Hq + g_first + g) * s.M + m] : 0.f;
        z_s[i] = 0.f;
    }
    __syncthreads();
    for (int i = tid; i < GH * s.nfk; i += blockDim.x) {
        int g = i / s.nfk, e = i - g * s.nfk;
        qf_s[i] = q_s[g * s.d + idf_k[e]];
    }
    __syncthreads();

    RunStat<GH> rs;
#pragma unroll
    for (int g = 0; g < GH; ++g) { rs.m[g] = kNegBig; rs.l[g] = 0.f; }
    float o_mid[GH], o_win[GH];
#pragma unroll
    for (int g = 0; g < GH; ++g) { o_mid[g] = 0.f; o_win[g] = 0.f; }

    // thread -> (token group, dim) maps of the two P.V products
    const int ntg_mid = s.nfv > 0 ? kTile / s.nfv : 0;
    const int tg_mid = s.nfv > 0 ? tid / s.nfv : 0, e_mid = s.nfv > 0 ? tid % s.nfv : 0;
    const bool act_mid = s.nfv > 0 && tg_mid < ntg_mid;
    const int ntg_win = kTile / s.d;
    const int tg_win = tid / s.d, e_win = tid % s.d;
    const bool act_win = tg_win < ntg_win;

    // after scores are known: update the running softmax state, leave p in p_s
    auto softmax_tile = [&](float (&sc)[GH], bool valid) {
        float mx[GH];
#pragma unroll
        for (int g = 0; g < GH; ++g) mx[g] = valid ? sc[g] : kNegBig;
        block_reduce<GH, true>(mx, red_s);
        float pv[GH], alpha[GH];
#pragma unroll
        for (int g = 0; g < GH; ++g) {
            float m_new = fmaxf(rs.m[g], mx[g]);
            alpha[g] = exp2f(rs.m[g] - m_new);
            rs.m[g] = m_new;
            pv[g] = valid ? exp2f(sc[g] - m_new) : 0.f;
            p_s[g * kTile + tid] = pv[g];
            o_mid[g] *= alpha[g];
            o_win[g] *= alpha[g];
        }
        for (int i = tid; i < GH * s.M; i += blockDim.x) z_s[i] *= alpha[i / s.M];
        block_reduce<GH, false>(pv, red_s);     // also publishes p_s and the z_s rescale
#pragma unroll
        for (int g = 0; g < GH; ++g) rs.l[g] = rs.l[g] * alpha[g] + pv[g];
    };

    // ---- middle tokens: classes [c0, c1) of this split ------------------------
    const int c0 = (int)((long long)split * s.P / p.n_split), c1 = (int)((long long)(split + 1) * s.P / p.n_split);
    for (int cls = c0; cls < c1; ++cls) {
        const int n_cls = cls < n_mid ? (n_mid - cls + s.P - 1) / s.P : 0;
        for (int a0 = 0; a0 < n_cls; a0 += kTile) {
            const int a = a0 + tid;
            const bool valid = a < n_cls;
            const int j = cls + s.P * a;
            float sc[GH];
#pragma unroll
            for (int g = 0; g < GH; ++g) sc[g] = 0.f;
            if (valid) {
                const KV* row = mid_row<KV>(c.k_mid, s, b, h, cls, a, s.nfk);
                for (int e = 0; e < s.nfk; ++e) {
                    float x = ld_f(row + e);
#pragma unroll
                    for (int g = 0; g < GH; ++g) sc[g] = fmaf(qf_s[g * s.nfk + e], x, sc[g]);
                }
                if (s.dck > 0) {
                    float cd, sd;
                    basis_cs(1, j, s.T, &cd, &sd);                  // rotation per unit of n
                    for (int n0 = 0; n0 < s.k; n0 += 32) {
                        float cr, sr;
                        basis_cs(n0, j, s.T, &cr, &sr);             // exact re-seed
                        const int n1 = min(s.k, n0 + 32);
                        for (int n = n0; n < n1; ++n) {
#pragma unroll
                            for (int g = 0; g < GH; ++g)
                                sc[g] = fmaf(u_s[g * s.M + 2 * n], cr, fmaf(u_s[g * s.M + 2 * n + 1], sr, sc[g]));
                            float t = cr * cd - sr * sd;
                            sr = fmaf(sr, cd, cr * sd);
                            cr = t;
                        }
                    }
                }
            }
            softmax_tile(sc, valid);
            const int nt = min(kTile, n_cls - a0);
            // o^u += p V^mu
            if (act_mid) {
                for (int i = tg_mid; i < nt; i += ntg_mid) {
                    float x = ld_f(mid_row<KV>(c.v_mid, s, b, h, cls, a0 + i, s.nfv) +
                                   v_mid_col(a0 + i, e_mid, s.nfv, sizeof(KV) == 2 ? FA_BF16 : FA_F32));
#pragma unroll
                    for (int g = 0; g < GH; ++g) o_mid[g] = fmaf(p_s[g * kTile + i], x, o_mid[g]);
                }
            }
            // z[m] += p F[m][j]: thread owns frequency n, walks the tile's tokens by rotation
            if (s.dcv > 0) {
                for (int n = tid; n < s.k; n += blockDim.x) {
                    float zr[GH], zi[GH];
#pragma unroll
                    for (int g = 0; g < GH; ++g) { zr[g] = 0.f; zi[g] = 0.f; }
                    float cd, sd;
                    basis_cs(n, s.P, s.T, &cd, &sd);               // step between consecutive slots
                    for (int i0 = 0; i0 < nt; i0 += 32) {
                        float cr, sr;
                        basis_cs(n, cls + s.P * (a0 + i0), s.T, &cr, &sr);
                        const int i1 = min(nt, i0 + 32);
                        for (int i = i0; i < i1; ++i) {
#pragma unroll
                            for (int g = 0; g < GH; ++g) {
                                float pv = p_s[g * kTile + i];
                                zr[g] = fmaf(pv, cr, zr[g]);
                                zi[g] = fmaf(pv, sr, zi[g]);
                            }
                            float t = cr * cd - sr * sd;
                            sr = fmaf(sr, cd, cr * sd);
                            cr = t;
                        }
                    }
#pragma unroll
                    for (int g = 0; g < GH; ++g) {
                        z_s[g * s.M + 2 * n] += zr[g];
                        z_s[g * s.M + 2 * n + 1] += zi[g];
                    }
                }
            }
            __syncthreads();
        }
    }

    // ---- window tokens [w0, w1) of this split: init rows, then the local ring --
    const int n_win = n_init + n_local;
    const int w0 = (int)((long long)split * n_win / p.n_split), w1 = (int)((long long)(split + 1) * n_win / p.n_split);
    for (int t0 = w0; t0 < w1; t0 += kTile) {
        const int t = t0 + tid;
        const bool valid = t < w1;
        auto row_of = [&](void* init, void* local, int tt) -> const KV* {
            if (tt < n_init) return win_row<KV>(init, s, b, h, s.l_init, tt);
            return win_row<KV>(local, s, b, h, s.l_local, (head + (tt - n_init)) % s.l_local);
        };
        float sc[GH];
#pragma unroll
        for (int g = 0; g < GH; ++g) sc[g] = 0.f;
        if (valid) {
            const KV* row = row_of(c.k_init, c.k_local, t);
            for (int e = 0; e < s.d; ++e) {
                float x = ld_f(row + e);
#pragma unroll
                for (int g = 0; g < GH; ++g) sc[g] = fmaf(q_s[g * s.d + e], x, sc[g]);
            }
        }
        softmax_tile(sc, valid);
        const int nt = min(kTile, w1 - t0);
        if (act_win) {
            for (int i = tg_win; i < nt; i += ntg_win) {
                float x = ld_f(row_of(c.v_init, c.v_local, t0 + i) + e_win);
#pragma unroll
                for (int g = 0; g < GH; ++g) o_win[g] = fmaf(p_s[g * kTile + i], x, o_win[g]);
            }
        }
        __syncthreads();
    }

    // ---- reduce the output accumulators over token groups, write the partials --
#pragma unroll
    for (int g = 0; g < GH; ++g) acc_s[tid * GH + g] = act_mid ? o_mid[g] : 0.f;
    __syncthreads();
    for (int i = tid; i < GH * s.nfv; i += blockDim.x) {
        int g = i / s.nfv, e = i - g * s.nfv;
        float v = 0.f;
        for (int tg = 0; tg < ntg_mid; ++tg) v += acc_s[(tg * s.nfv + e) * GH + g];
        o_s[g * s.d + idf_v[e]] = v;
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < GH; ++g) acc_s[tid * GH + g] = act_win ? o_win[g] : 0.f;
    __syncthreads();
    for (int i = tid; i < GH * s.d; i += blockDim.x) {
        int g = i / s.d, e = i - g * s.d;
        float v = o_s[i];
        for (int tg = 0; tg < ntg_win; ++tg) v += acc_s[(tg * s.d + e) * GH + g];
        if (g < ng) ws.o[(((size_t)b * s.Hq + g_first + g) * p.n_part + split) * s.d + e] = v;
    }
    for (int i = tid; i < GH * s.M; i += blockDim.x) {
        int g = i / s.M, m = i - g * s.M;
        if (g < ng) ws.z[(((size_t)b * s.Hq + g_first + g) * p.n_part + split) * s.M + m] = z_s[i];
    }
    if (tid < ng) {
        float* ml = ws.ml + (((size_t)b * s.Hq + g_first + tid) * p.n_part + split) * 2;
        float mv = kNegBig, lv = 0.f;
#pragma unroll
        for (int g = 0; g < GH; ++g) if (g == tid) { mv = rs.m[g]; lv = rs.l[g]; }
        ml[0] = mv;
        ml[1] = lv;
    }
}


template <typename KV, int GH>
static cudaError_t launch_direct_t(const Dims& s, const CacheDev& c, const DecodePlan& p, const void* q, char* ws,
                                   cudaStream_t st) {
    size_t smem = sizeof(float) * ((size_t)GH * s.d * 2 + (size_t)GH * s.nfk + 2 * (size_t)GH * s.M + (size_t)GH * kTile +
                                   8 * GH + (size_t)256 * GH);
    cudaError_t err = ensure_dynamic_smem(decode_direct_kernel<KV, GH>, smem);
    if (err != cudaSuccess) return err;
    decode_direct_kernel<KV, GH><<<dim3(p.n_split, s.Hkv * p.n_pass, s.B), 256, smem, st>>>(s, c, p, static_cast<const KV*>(q), ws);
    return cudaGetLastError();
}

cudaError_t launch_decode_direct(const Dims& s, const CacheDev& c, int dtype, const DecodePlan& p, const void* q, char* ws,
                                 cudaStream_t st) {
    if (dtype == FA_BF16) {
        if (p.gh == 4) return launch_direct_t<__nv_bfloat16, 4>(s, c, p, q, ws, st);
        if (p.gh == 2) return launch_direct_t<__nv_bfloat16, 2>(s, c, p, q, ws, st);
        return launch_direct_t<__nv_bfloat16, 1>(s, c, p, q, ws, st);
    }
    if (p.gh == 4) return launch_direct_t<float, 4>(s, c, p, q, ws, st);
    if (p.gh == 2) return launch_direct_t<float, 2>(s, c, p, q, ws, st);
    return launch_direct_t<float, 1>(s, c, p, q, ws, st);
}

}  // namespace fa
