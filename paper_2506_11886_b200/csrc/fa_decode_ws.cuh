// Views into the scratch workspace of one fa_decode_attention call, shared by
// the prologue, main and epilogue kernels.
#pragma once

#include "fa_common.cuh"

namespace fa {

struct Ws {
    int32_t* bar;  // [B][Hkv][n_pass][4]   barrier counters of the fused kernel: zero between calls
    float* u;      // [B][Hq][M]            scale * log2(e) * w_m * (C^K q)_m
    float* ml;     // [B][Hq][n_part][2]    running max (log2 units), sum of p
    float* o;      // [B][Hq][n_part][d]    un-normalised outputs, natural dim order (kept dims + windows)
    float* z;      // [B][Hq][n_part][M]    un-normalised p^T Phi
    float* oc;     // [B][Hq][max(n_slice, n_part)][dcv] partial o^c per coefficient-row slice
    float* om;     // [B][Hq][d]            merged o (fused kernel)
    int32_t* cnt;  // [B][Hkv]              epilogue tickets
};

__host__ __device__ inline Ws ws_view(char* w, const DecodePlan& p) {
    Ws v;
    v.bar = reinterpret_cast<int32_t*>(w + p.off_bar);
    v.u = reinterpret_cast<float*>(w + p.off_u);
    v.ml = reinterpret_cast<float*>(w + p.off_ml);
    v.o = reinterpret_cast<float*>(w + p.off_o);
    v.z = reinterpret_cast<float*>(w + p.off_z);
    v.oc = reinterpret_cast<float*>(w + p.off_oc);
    v.om = reinterpret_cast<float*>(w + p.off_om);
    v.cnt = reinterpret_cast<int32_t*>(w + p.off_cnt);
    return v;
}

}  // namespace fa
