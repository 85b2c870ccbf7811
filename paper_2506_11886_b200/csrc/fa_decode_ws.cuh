// Views into the scratch workspace of one fa_decode_attention call, shared by
// the prologue, main and epilogue kernels.
#pragma once

#include "fa_common.cuh"

namespace fa {

struct Ws {
    float* u;      // [B][Hq][M]            scale * log2(e) * w_m * (C^K q)_m
    float* ml;     // [B][Hq][n_split][2]   running max (log2 units), sum of p
    float* o;      // [B][Hq][n_split][d]   un-normalised outputs, natural dim order (kept dims + windows)
    float* z;      // [B][Hq][n_split][M]   un-normalised p^T Phi
    float* oc;     // [B][Hq][n_slice][dcv] partial o^c per coefficient-row slice
    int32_t* cnt;  // [B][Hkv]              epilogue tickets
};

__host__ __device__ inline Ws ws_view(char* w, const DecodePlan& p) {
    Ws v;
    v.u = reinterpret_cast<float*>(w + p.off_u);
    v.ml = reinterpret_cast<float*>(w + p.off_ml);
    v.o = reinterpret_cast<float*>(w + p.off_o);
    v.z = reinterpret_cast<float*>(w + p.off_z);
    v.oc = reinterpret_cast<float*>(w + p.off_oc);
    v.cnt = reinterpret_cast<int32_t*>(w + p.off_cnt);
    return v;
}

}  // namespace fa
