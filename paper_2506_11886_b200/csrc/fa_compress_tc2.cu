// fa_compress, tensor-core path for CTA pairs (Eq.3-4; bf16 caches, sm_100a): the kernel of fa_compress_tc.cu with
// tcgen05.mma.cta_group::2.  Two CTAs of a cluster own two neighbouring tiles of 128 coefficient rows of the same
// KV heads and token blocks; one MMA covers both (256 accumulator rows: each CTA's 128 in its own tensor memory).
// Each CTA generates the basis tile of its own rows and loads only HALF of the K / V boxes of a block — the even CTA
// the K dims, the odd CTA the V dims — and the tensor cores of the pair read both halves.  Per SM that is half the
// box traffic from L2 and, in the same shared memory, a ring of four stages instead of two, which is what hides the
// latency of the box loads that bounds the single-CTA kernel.
//
// Roles per CTA: warp 0 (one lane) TMA producer of its half of the boxes; warp 1 allocates tensor memory (one warp of
// each CTA, collectively) and, in the even CTA only, issues the MMAs of the pair; warps 2-9 generate the basis tile and
// run the epilogue; warps 10-13 write the kept-dim rows of the middle (the even CTA K^mu, the odd CTA V^mu).
// Barriers across the pair: a lane of the odd CTA waits for that CTA's basis tile and boxes of a stage and forwards
// their completion to the even CTA (mapa + remote arrive); the even CTA's tcgen05.commit
// signals the stage barriers of both CTAs (multicast of the ARRIVAL, not of a load).
// Every wait is bounded; tensor memory is freed on every path; both CTAs meet before they leave.
#include <mutex>

#include "fa_umma.cuh"

namespace fa {
namespace {

using bf16 = __nv_bfloat16;
constexpr int kBM = 128;          // coefficient rows per CTA (256 per pair)
constexpr int kBK = 64;           // tokens per pipeline stage
constexpr int kGenWarps = 8;       // basis generators (and epilogue): 16 tokens of two rows per thread and stage
constexpr int kGatherWarps = 4;    // kept-dim rows of the middle, from the B boxes
constexpr int kGatherItems = 4;    // 16-byte chunks per gather thread and stage, at most
constexpr int kThreadsTc = 64 + 32 * (kGenWarps + kGatherWarps);
using namespace umma;

// Work of a launch: the token blocks of all (batch, head group) units, laid end to end: position = unit * blocks + block.
// A TEAM is the M / 256 pairs that own the row tiles of the same blocks (they read the same boxes, in step, so the
// prefill comes from HBM once); team t takes positions start[t] .. start[t + 1], a whole number of blocks that may
// end inside a unit and go on into the next (one SEGMENT per unit touched: main loop, then an epilogue that adds the
// segment's partial sums).  The table is cut on the host so that every team has the same cost (blocks + epilogues),
// and so that teams x pairs fill the pairs that are resident at once; with per > 0 the cut is uniform instead
// (every unit in pieces of per blocks, one team each; the order-fixed mode cuts every unit in two: a coefficient is
// then zero plus two terms, and the sum of two floats does not depend on which arrives first).
constexpr int kMaxTeams = 96;
struct TeamCuts { uint32_t start[kMaxTeams + 1]; };

// D = head dim (64 or 128): N = 2 D accumulator columns per KV head (K dims, then V dims); HP heads share the pair
// and its generated basis tiles (HP * N <= 512 tensor-memory columns).  grid 2 * teams * (M / 256), clusters of two.
template <int D, int HP>
__global__ void __launch_bounds__(kThreadsTc, 1) compress_tc2_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                     const __grid_constant__ CUtensorMap tmV, Dims s,
                                                                     CacheDev c, int L, const __grid_constant__ TeamCuts cuts,
                                                                     int per, int gather) {
    constexpr int N = 2 * D;
    constexpr int kABytes = kBM * kBK * 2;                 // 16 KB basis tile
    constexpr int kBoxBytes = kBK * 64 * 2;                // 8 KB per [64 tokens x 64 dims] box
    constexpr int kBHalf1 = (D / 64) * kBoxBytes;           // this CTA's boxes of one head: all D dims of ONE side
    constexpr int kBHalf = HP * kBHalf1;
    constexpr int kStageBytesTc = kABytes + kBHalf;
    constexpr int kStagesTc = (200 * 1024) / kStageBytesTc < 6 ? (200 * 1024) / kStageBytesTc : 6;
    constexpr uint32_t kTmemCols = HP * N;
    // bf16 x bf16 -> fp32, A K-major, B MN-major, N = 2 D columns, M = 256 rows over the pair
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)((2 * kBM) >> 4) << 24);
    extern __shared__ unsigned char smem_unaligned[];
    unsigned char* smem = smem_unaligned + ((1024u - (smem_u32(smem_unaligned) & 1023u)) & 1023u);
    unsigned char* stage0 = smem;                          // kStagesTc x (A | this CTA's boxes), 1024-byte aligned
    // one barrier per stage for this CTA's basis tile (eight generator warps) and boxes (the producer's expect_tx):
    // the thread that issues the MMAs pays for every barrier it passes
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStagesTc * kStageBytesTc);
    uint64_t* peer = full + kStagesTc;                     // even CTA: the odd CTA's stage is complete
    uint64_t* empty = peer + kStagesTc;
    uint64_t* acc_ready = empty + kStagesTc;
    uint64_t* gather_done = acc_ready + 1;                 // the gather warps are past the last box of the segment
    uint64_t* epi_done = gather_done + 1;                  // the epilogue has left the stage ring (its scratch)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(epi_done + 1);
    volatile int* fail = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* idf_s = reinterpret_cast<int*>(tmem_slot + 4);    // [HP][D]: the kept dims of this CTA's side of the CTA's heads

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();               // 0: K boxes, issues the MMAs; 1: V boxes
    const int side = (int)rank;
    const int n_pairs = s.M / (2 * kBM);                   // pairs of a team
    const int cluster = (int)blockIdx.x >> 1, team = cluster / n_pairs, pair = cluster - team * n_pairs;
    const int mt = 2 * pair + (int)rank;                   // this CTA's row tile, the same in every segment
    const int n_hg = s.Hkv / HP;
    const int n_init = min(L, s.l_init);
    const int n_local = min(L - n_init, s.l_local);
    const int n_mid = L - n_init - n_local;
    const int nkb = (n_mid + kBK - 1) / kBK;
    uint32_t pos_begin, pos_end;
    if (per > 0) {                                         // uniform cut: every unit in ceil(blocks / per) pieces of per blocks
        const int pieces = (nkb + per - 1) / per, unit = team / pieces, piece = team - unit * pieces;
        pos_begin = (uint32_t)unit * (uint32_t)nkb + (uint32_t)(piece * per);
        pos_end = (uint32_t)unit * (uint32_t)nkb + (uint32_t)min(nkb, (piece + 1) * per);
    } else {
        pos_begin = cuts.start[team];
        pos_end = cuts.start[team + 1];
    }
    // the segment that starts at position pos: its unit (batch b, heads h0 ...) and blocks kb0 .. kb1
    struct Seg { int b, h0, kb0, kb1; };
    auto seg_at = [&](uint32_t pos) {
        const int unit = (int)(pos / (uint32_t)nkb), kb0 = (int)(pos - (uint32_t)unit * (uint32_t)nkb);
        const int kb1 = (int)min((uint32_t)nkb, (uint32_t)kb0 + (pos_end - pos));
        return Seg{unit / n_hg, (unit % n_hg) * HP, kb0, kb1};
    };

    // The contraction of the next layer (a call over several layers launches them one behind the other, programmatically)
    // may take the SMs that this grid's first CTAs to finish leave; it waits for this grid in front of its reductions.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        // a stage is free again when the pair's MMAs have read it and this CTA's gather warps have taken their rows
        for (int i = 0; i < kStagesTc; ++i) {
            mbar_init(full + i, kGenWarps + 1);
            mbar_init(peer + i, 1);
            mbar_init(empty + i, 1 + kGatherWarps);
        }
        mbar_init(acc_ready, 1);
        mbar_init(gather_done, kGatherWarps);
        mbar_init(epi_done, kGenWarps);
        *fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int nf_side = side ? s.nfv : s.nfk;
    if (warp == 1) {                                       // tensor memory: one warp of each CTA of the pair, collectively
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                    // the peer's barriers are initialised before anyone signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (pos_end > pos_begin) {
        if (warp == 0) {
            // ---------------- TMA producer: this CTA's half of the B operand (one side, all D dims, 64 tokens) ----------------
            if (lane == 0) {
                const CUtensorMap* tm = side ? &tmV : &tmK;
                int it = 0, seg = 0;
                bool live = true;
                for (uint32_t pos = pos_begin; live && pos < pos_end; ++seg) {
                    const Seg g = seg_at(pos);
                    // the epilogue of the segment before used the ring as its scratch
                    if (seg > 0 && !mbar_wait(epi_done, (seg - 1) & 1, fail, c.status)) break;
                    for (int kb = g.kb0; kb < g.kb1; ++kb, ++it) {
                        const int st = it % kStagesTc;
                        if (it >= kStagesTc && !mbar_wait(empty + st, ((it / kStagesTc) - 1) & 1, fail, c.status)) { live = false; break; }
                        unsigned char* bdst = stage0 + (size_t)st * kStageBytesTc + kABytes;
                        mbar_expect_tx(full + st, (uint32_t)kBHalf);
                        const int tok = n_init + kb * kBK;
#pragma unroll
                        for (int hh = 0; hh < HP; ++hh)
#pragma unroll
                            for (int bx = 0; bx < D / 64; ++bx)
                                tma_load_4d(bdst + hh * kBHalf1 + bx * kBoxBytes, tm, bx * 64, g.h0 + hh, tok, g.b, full + st);
                    }
                    pos += (uint32_t)(g.kb1 - g.kb0);
                }
            }
        } else if (warp == 1) {
            // ---------------- MMA issuer: the even CTA, for the pair ----------------
            if (lane == 0 && rank == 0) {
                int it = 0;
                bool live = true;
                for (uint32_t pos = pos_begin; live && pos < pos_end;) {
                    const Seg g = seg_at(pos);
                    // The accumulators of the segment before have been read: the stage barriers below complete only
                    // after the generator warps of both CTAs, which are the epilogue warps, are past that epilogue.
                    for (int kb = g.kb0; kb < g.kb1; ++kb, ++it) {
                        const int st = it % kStagesTc;
                        const uint32_t par = (it / kStagesTc) & 1;
                        if (!mbar_wait(full + st, par, fail, c.status) || !mbar_wait(peer + st, par, fail, c.status)) { live = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t a_addr = smem_u32(stage0 + (size_t)st * kStageBytesTc);
                        const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                        for (int ks = 0; ks < kBK / 16; ++ks) {
                            // A: K-major, rows of 128 bytes, 8-row groups 1024 bytes apart; 16 tokens = 32 bytes along the row
                            // (the same offsets in both CTAs: each supplies its own 128 rows)
                            const uint64_t adesc = umma_desc(a_addr + ks * 32, 1, 1024 >> 4);
                            // B: MN-major, 64 dims per 128-byte row, 8-token groups 1024 bytes apart, next 64 dims one box
                            // further; each CTA supplies D of the 2 D columns
#pragma unroll
                            for (int hh = 0; hh < HP; ++hh) {
                                const uint64_t bdesc = umma_desc(b_addr + hh * kBHalf1 + ks * 2048, kBoxBytes >> 4, 1024 >> 4);
                                umma_bf16_pair(tmem_base + hh * N, adesc, bdesc, kIdesc, (kb > g.kb0 || ks > 0) ? 1u : 0u);
                            }
                        }
                        umma_commit_pair(empty + st);      // frees the stage in both CTAs when these MMAs have read it
                    }
                    if (live) umma_commit_pair(acc_ready);
                    pos += (uint32_t)(g.kb1 - g.kb0);
                }
            } else if (lane == 0) {
                // the odd CTA's otherwise idle lane: when this CTA's basis tile and boxes of a stage are complete it tells
                // the even CTA, which issues the MMAs (one remote arrival per stage, kept off the generators' path)
                const int n_it = (int)(pos_end - pos_begin);
                for (int it = 0; it < n_it; ++it) {
                    const int st = it % kStagesTc;
                    const uint32_t par = (it / kStagesTc) & 1;
                    if (!mbar_wait(full + st, par, fail, c.status)) break;
                    mbar_arrive_cluster(peer + st, 0);
                }
            }
        } else if (warp >= 2 + kGenWarps) {
            // ---------------- kept dims of the middle tokens: this CTA's boxes -> K^mu (even CTA) or V^mu (odd CTA) ----------------
            const int gt = tid - 32 * (2 + kGenWarps);           // 0 .. 32 kGatherWarps - 1
            const int cph = nf_side >> 3;                                      // 16-byte chunks per kept-dim row of this side
            // the pairs of the team load the same boxes and share the tokens: this pair takes rows pair, pair + n_pairs, ...
            const int n_tok = pair < kBK ? (kBK - pair + n_pairs - 1) / n_pairs : 0;
            const int n_items = gather ? n_tok * HP * cph : 0;                // <= kGatherItems per thread (checked on the host)
            const bool p2 = (s.P & (s.P - 1)) == 0;
            const int lgP = 31 - __clz(s.P);
            int it = 0;
            bool live = true;
            // (after a wait that ran out the warp still walks the segments, without work: its partners count on it
            // at the barrier below)
            for (uint32_t pos = pos_begin; pos < pos_end;) {
                const Seg g = seg_at(pos);
                // the kept dims of this side of the segment's heads (the four gather warps, on their own barrier)
                asm volatile("bar.sync 3, %0;" ::"n"(32 * kGatherWarps) : "memory");
                if (gather)
                    for (int i = gt; i < HP * nf_side; i += 32 * kGatherWarps) {
                        const int hh = i / nf_side, r = i - hh * nf_side;
                        idf_s[hh * D + r] = (side ? c.idx_full_v : c.idx_full_k)[(size_t)(g.h0 + hh) * nf_side + r];
                    }
                asm volatile("bar.sync 3, %0;" ::"n"(32 * kGatherWarps) : "memory");
                // An item = one 16-byte chunk (8 kept dims) of one kept-dim row.  A thread keeps the same items in every
                // block: token row r of the boxes, head, side and LOGICAL chunk, so the eight source offsets inside a stage
                // are constants (two 16-bit offsets per register); only the destination row moves with the token.
                uint32_t src[kGatherItems][4];
                int meta[kGatherItems];                    // r | hh << 8 | lch << 16, or -1
#pragma unroll
                for (int u = 0; u < kGatherItems; ++u) {
                    const int idx = gt + u * 32 * kGatherWarps;
                    meta[u] = -1;
#pragma unroll
                    for (int i2 = 0; i2 < 4; ++i2) src[u][i2] = 0;
                    if (idx < n_items) {
                        const int ti = idx / (HP * cph), rem = idx - ti * (HP * cph);
                        const int hh = rem / cph, lch = rem - hh * cph;
                        const int r = pair + n_pairs * ti;
                        const int* idf = idf_s + hh * D + lch * 8;
                        const uint32_t row0 = (uint32_t)(hh * kBHalf1 + r * 128);
#pragma unroll
                        for (int i2 = 0; i2 < 4; ++i2) {
                            const int e0 = idf[2 * i2], e1 = idf[2 * i2 + 1];
                            const uint32_t o0 = row0 + (uint32_t)((e0 >> 6) * kBoxBytes + ((((e0 & 63) >> 3) ^ (r & 7)) << 4) + (e0 & 7) * 2);
                            const uint32_t o1 = row0 + (uint32_t)((e1 >> 6) * kBoxBytes + ((((e1 & 63) >> 3) ^ (r & 7)) << 4) + (e1 & 7) * 2);
                            src[u][i2] = o0 | (o1 << 16);   // a stage is at most 64 KB
                        }
                        meta[u] = r | (hh << 8) | (lch << 16);
                    }
                }
                for (int kb = g.kb0; live && kb < g.kb1; ++kb, ++it) {
                    const int st = it % kStagesTc;
                    if (!mbar_wait(full + st, (it / kStagesTc) & 1, fail, c.status)) { live = false; break; }
                    const unsigned char* bsrc = stage0 + (size_t)st * kStageBytesTc + kABytes;
                    const int jb = kb * kBK;               // first middle token of the block
                    uint4 val[kGatherItems];
#pragma unroll
                    for (int u = 0; u < kGatherItems; ++u) {
                        uint32_t w[4] = {0u, 0u, 0u, 0u};
                        if (meta[u] >= 0) {
#pragma unroll
                            for (int i2 = 0; i2 < 4; ++i2) {
                                const uint32_t lo = *reinterpret_cast<const uint16_t*>(bsrc + (src[u][i2] & 0xffffu));
                                const uint32_t hi = *reinterpret_cast<const uint16_t*>(bsrc + (src[u][i2] >> 16));
                                w[i2] = lo | (hi << 16);
                            }
                        }
                        val[u] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    __syncwarp();                          // the values are in registers: the stage goes back before the stores
                    if (lane == 0) mbar_arrive(empty + st);
#pragma unroll
                    for (int u = 0; u < kGatherItems; ++u) {
                        const int j = jb + (meta[u] & 0xff);
                        if (meta[u] >= 0 && j < n_mid) {
                            const int hh = (meta[u] >> 8) & 0xf, lch = meta[u] >> 16;
                            const int cls = p2 ? (j & (s.P - 1)) : j % s.P, slot = p2 ? (j >> lgP) : j / s.P;
                            const int nfull = nf_side;
                            // logical chunk lch of a V^mu row is stored at chunk lch ^ swizzle
                            const int ch = side ? (lch ^ v_swz(slot, nfull >> 3)) : lch;
                            bf16* dst = mid_row<bf16>(side ? c.v_mid : c.k_mid, s, g.b, g.h0 + hh, cls, slot, nfull);
                            reinterpret_cast<uint4*>(dst)[ch] = val[u];
                        }
                    }
                }
                __syncwarp();
                if (live && lane == 0) mbar_arrive(gather_done);
                pos += (uint32_t)(g.kb1 - g.kb0);
            }
        } else {
            // ---------------- basis generators: A operand ----------------
            const int t = tid - 64;                        // 0 .. 32 kGenWarps - 1
            const int fi = t >> 2, tqr = t & 3;            // frequency pair of the tile, quarter of the 64 tokens
            const unsigned n = (unsigned)(mt * (kBM / 2) + fi);         // frequency of rows 2 fi (cos), 2 fi + 1 (sin)
            const bool row_on = (int)(2 * n) < s.M;
            const float inv_T = 1.0f / (float)s.T;
            auto splat_rot = [&](unsigned long long tokens, unsigned long long& CS, unsigned long long& SN, unsigned long long& NSN) {
                const unsigned ph = (unsigned)((tokens * n) % (unsigned)s.T);
                const float a = 6.283185307179586f * ((float)ph * inv_T - ((float)ph * inv_T >= 0.5f ? 1.0f : 0.0f));
                const float cs = __cosf(a), sn = __sinf(a);
                asm("mov.b64 %0, {%1,%1};" : "=l"(CS) : "f"(cs));
                asm("mov.b64 %0, {%1,%1};" : "=l"(SN) : "f"(sn));
                asm("mov.b64 %0, {%1,%1};" : "=l"(NSN) : "f"(-sn));
            };
            // rotations by two tokens, and by the 48 tokens between the end of this thread's run and its run in the next block
            unsigned long long CS2, SN2, NSN2, CS48, SN48, NSN48;
            splat_rot(2ull, CS2, SN2, NSN2);
            splat_rot(48ull, CS48, SN48, NSN48);
            const int r0 = 2 * fi, r1 = 2 * fi + 1;
            const uint32_t row_off0 = (uint32_t)((r0 >> 3) * 1024 + (r0 & 7) * 128);
            const uint32_t row_off1 = (uint32_t)((r1 >> 3) * 1024 + (r1 & 7) * 128);
            // packed phasors of two neighbouring tokens: C = (cos, cos), S = (sin, sin).  Seeded from exact integer
            // phases every kReseed blocks and carried by rotations in between (9 per block: the drift stays far
            // below the bf16 rounding of the tile).
            constexpr int kReseed = 8;
            unsigned long long C = 0, S = 0;
            int it = 0, seg = 0;
            bool live = true;
            for (uint32_t pos = pos_begin; live && pos < pos_end; ++seg) {
                const Seg g = seg_at(pos);
                for (int kb = g.kb0; kb < g.kb1; ++kb, ++it) {
                    const int st = it % kStagesTc;
                    if (it >= kStagesTc && !mbar_wait(empty + st, ((it / kStagesTc) - 1) & 1, fail, c.status)) { live = false; break; }
                    unsigned char* a_dst = stage0 + (size_t)st * kStageBytesTc;
                    const int j0 = kb * kBK + 16 * tqr;
                    if ((kb - g.kb0) % kReseed == 0) {
                        const unsigned pa = (n * (unsigned)j0) % (unsigned)s.T, pb = (n * (unsigned)(j0 + 1)) % (unsigned)s.T;
                        const float fa = (float)pa * inv_T, fb = (float)pb * inv_T;
                        const float aa = 6.283185307179586f * (fa - (fa >= 0.5f ? 1.0f : 0.0f));
                        const float ab = 6.283185307179586f * (fb - (fb >= 0.5f ? 1.0f : 0.0f));
                        asm("mov.b64 %0, {%1,%2};" : "=l"(C) : "f"(__cosf(aa)), "f"(__cosf(ab)));
                        asm("mov.b64 %0, {%1,%2};" : "=l"(S) : "f"(__sinf(aa)), "f"(__sinf(ab)));
                    }
                    const bool whole = row_on && j0 + 16 <= n_mid;      // no masking needed in the common case
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {       // 8 tokens = one 16-byte chunk of each row
                        uint32_t wc[4], wsn[4];
#pragma unroll
                        for (int i2 = 0; i2 < 4; ++i2) {
                            float c0, c1, s0, s1;
                            asm("mov.b64 {%0,%1}, %2;" : "=f"(c0), "=f"(c1) : "l"(C));
                            asm("mov.b64 {%0,%1}, %2;" : "=f"(s0), "=f"(s1) : "l"(S));
                            if (!whole) {
                                const int j = j0 + ch * 8 + i2 * 2;
                                const bool v0 = row_on && j < n_mid, v1 = row_on && j + 1 < n_mid;
                                c0 = v0 ? c0 : 0.f; s0 = v0 ? s0 : 0.f; c1 = v1 ? c1 : 0.f; s1 = v1 ? s1 : 0.f;
                            }
                            const __nv_bfloat162 pc = __floats2bfloat162_rn(c0, c1);
                            const __nv_bfloat162 ps = __floats2bfloat162_rn(s0, s1);
                            wc[i2] = *reinterpret_cast<const uint32_t*>(&pc);
                            wsn[i2] = *reinterpret_cast<const uint32_t*>(&ps);
                            // advance both phasors by two tokens: C' = C cs2 - S sn2, S' = S cs2 + C sn2
                            unsigned long long tC, tS, nC, nS;
                            asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(tC) : "l"(C), "l"(CS2));
                            asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(tS) : "l"(S), "l"(CS2));
                            asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(nC) : "l"(S), "l"(NSN2), "l"(tC));
                            asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(nS) : "l"(C), "l"(SN2), "l"(tS));
                            C = nC;
                            S = nS;
                        }
                        const int chunk = 2 * tqr + ch;
                        *reinterpret_cast<uint4*>(a_dst + row_off0 + ((chunk ^ (r0 & 7)) << 4)) = make_uint4(wc[0], wc[1], wc[2], wc[3]);
                        *reinterpret_cast<uint4*>(a_dst + row_off1 + ((chunk ^ (r1 & 7)) << 4)) = make_uint4(wsn[0], wsn[1], wsn[2], wsn[3]);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic stores -> visible to the tensor core
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full + st);
                    {                                      // on to the same run of the next block
                        unsigned long long tC, tS, nC, nS;
                        asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(tC) : "l"(C), "l"(CS48));
                        asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(tS) : "l"(S), "l"(CS48));
                        asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(nC) : "l"(S), "l"(NSN48), "l"(tC));
                        asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(nS) : "l"(C), "l"(SN48), "l"(tS));
                        C = nC;
                        S = nS;
                    }
                }
                if (!live) break;
                // ---------------- epilogue of the segment: accumulators -> compressed columns ----------------
                // the stage ring is reused below: every MMA has read it, and the gather warps have left it
                const bool ok = mbar_wait(acc_ready, seg & 1, fail, c.status) && mbar_wait(gather_done, seg & 1, fail, c.status);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // the coefficients are cleared by the partition kernel, which this launch may overlap: wait for it here
                asm volatile("griddepcontrol.wait;" ::: "memory");
                if (!ok) break;
                {
                    const int lane_grp = warp & 3;         // a warp reads tensor-memory lanes 32 (warp % 4) ...
                    const int col_part = (warp - 2) >> 2;  // the two warps that share a lane group take half of the columns each
                    constexpr int kPart = (int)kTmemCols / (kGenWarps / 4);      // a whole number of sides (D columns each)
                    const int m_base = mt * kBM + lane_grp * 32;
                    // A thread holds 32 columns of ONE row of the accumulator.  The warp lays its 32 rows x D columns of one side
                    // (K or V of one head) out in the idle stage ring; then lane q owns the four compressed dims 4 q .. 4 q + 3
                    // (slots of D^c, ascending) and adds them row by row with one 16-byte vector reduction: a warp instruction
                    // covers a whole coefficient row of the side (d_c contiguous floats).
                    float* tile = reinterpret_cast<float*>(stage0) + (warp - 2) * (32 * (D + 1));
#pragma unroll 1
                    for (int t0 = col_part * kPart; t0 < (col_part + 1) * kPart; t0 += D) {
                        const int hh = t0 / N;
                        const bool is_k = t0 - hh * N < D;
                        const int ncomp = is_k ? s.dck : s.dcv, nq = ncomp >> 2;
                        int col[4] = {0, 0, 0, 0};
                        if (lane < nq) {
                            const int32_t* idc = (is_k ? c.idx_comp_k : c.idx_comp_v) + (size_t)(g.h0 + hh) * ncomp + 4 * lane;
#pragma unroll
                            for (int i = 0; i < 4; ++i) col[i] = idc[i];
                        }
#pragma unroll 1
                        for (int cb = 0; cb < D; cb += 32) {
                            float v[32];
                            tmem_ld32(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(t0 + cb), v);
#pragma unroll
                            for (int i = 0; i < 32; ++i) tile[lane * (D + 1) + cb + i] = v[i];
                        }
                        __syncwarp();
                        float* base = coef_rows(is_k ? c.coef_k : c.coef_v, s, g.b, g.h0 + hh, ncomp) + (size_t)m_base * ncomp + 4 * lane;
                        if (lane < nq) {
#pragma unroll 4
                            for (int rr = 0; rr < 32; ++rr) {
                                const float* trow = tile + rr * (D + 1);
                                if (m_base + rr < s.M)
                                    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(base + (size_t)rr * ncomp), "f"(trow[col[0]]),
                                                 "f"(trow[col[1]]), "f"(trow[col[2]]), "f"(trow[col[3]])
                                                 : "memory");
                            }
                        }
                        __syncwarp();
                    }
                }
                pos += (uint32_t)(g.kb1 - g.kb0);
                if (pos < pos_end) {
                    // another segment follows: the accumulators are read and the ring is free for its boxes and tiles
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(epi_done);
                    // the other generator warps' scratch lies in the stages that this warp writes next
                    if (!mbar_wait(epi_done, seg & 1, fail, c.status)) break;
                }
            }
        }
    }
    // both CTAs are done with each other's barriers and with the accumulators before tensor memory goes back
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// 4-D view (dim, head, token, batch) of a prefilled K or V with element strides (1, sh, st, sb); box = 64 dims x 64 tokens.
bool make_map2(CUtensorMap* tm, const void* base, const Dims& s, int64_t sb, int64_t st, int64_t sh, int L) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)s.d, (cuuint64_t)s.Hkv, (cuuint64_t)L, (cuuint64_t)s.B};
    cuuint64_t strides[3] = {(cuuint64_t)sh * 2, (cuuint64_t)st * 2, (cuuint64_t)(s.B > 1 ? sb : st * (int64_t)L) * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)kBK, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int HP>
cudaError_t launch_tc2_t(const CUtensorMap& tmK, const CUtensorMap& tmV, const Dims& s, const CacheDev& c, int L, int n_mid,
                         bool ordered, bool gather, cudaStream_t stream) {
    constexpr size_t stage = (size_t)kBM * kBK * 2 + (size_t)HP * (D / 64) * kBK * 64 * 2;
    constexpr size_t n_stages = (200 * 1024) / stage < 6 ? (200 * 1024) / stage : 6;
    const size_t smem = n_stages * stage + 8 * (3 * n_stages + 3) + 16 + sizeof(int) * HP * D + 64 + 1024;
    cudaError_t err = ensure_dynamic_smem(compress_tc2_kernel<D, HP>, smem);
    if (err != cudaSuccess) return err;
    const int n_pairs = s.M / (2 * kBM);
    const int nkb = (n_mid + kBK - 1) / kBK;
    const long long n_units = (long long)(s.Hkv / HP) * s.B;
    const long long total = n_units * nkb;                      // positions: the blocks of all units, end to end
    if (total <= 0 || total >= (1ll << 31)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kThreadsTc);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start under the partition kernel in front of it
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    TeamCuts cuts = {};
    int n_teams, per = 0;
    if (ordered) {
        // Two teams per unit, half of its blocks each: every coefficient is zero + a + b, and fl(a + b) = fl(b + a), so the
        // result has the same bits whichever half arrives first (three terms would not).  Pairs beyond the resident
        // ones run in later waves.
        per = (nkb + 1) / 2;
        n_teams = (int)n_units * ((nkb + per - 1) / per);
    } else {
        // pairs resident at once (cached per device): the teams fill them, no second wave
        static int resident[16] = {};
        static std::mutex mu;
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 16) return cudaErrorInvalidValue;
        std::lock_guard<std::mutex> lock(mu);
        if (resident[dev] == 0) {
            cfg.gridDim = dim3(2 * sm_count());
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, compress_tc2_kernel<D, HP>, &cfg) != cudaSuccess || n < 1) {
                cudaGetLastError();
                n = sm_count() / 2 - 2;
            }
            cfg.numAttrs = 2;
            resident[dev] = n;
        }
        n_teams = resident[dev] / n_pairs;
        if (n_teams < 1) n_teams = 1;
        if (n_teams > kMaxTeams) n_teams = kMaxTeams;
        if (n_teams > total) n_teams = (int)total;
        // Equal cost per team: a segment costs its blocks plus kEpi (epilogue, pipeline refill, in blocks).  The smallest
        // budget with which the walk below covers all positions in n_teams teams, by bisection.
        constexpr long long kEpi = 12, kMinSeg = 8;
        auto walk = [&](long long budget, uint32_t* start) {
            long long pos = 0;
            int t = 0;
            for (; t < n_teams && pos < total; ++t) {
                if (start) start[t] = (uint32_t)pos;
                long long left = budget;
                while (pos < total && left >= kEpi + kMinSeg) {
                    const long long unit_end = (pos / nkb + 1) * nkb;
                    long long take = unit_end - pos < left - kEpi ? unit_end - pos : left - kEpi;
                    if (unit_end - pos - take > 0 && unit_end - pos - take < kMinSeg) take = unit_end - pos - kMinSeg;   // no crumbs for the next team
                    if (take <= 0) break;
                    pos += take;
                    left -= take + kEpi;
                }
            }
            if (start)
                for (int u = t; u <= n_teams; ++u) start[u] = (uint32_t)(u == n_teams ? total : pos);
            return pos >= total;
        };
        long long lo = kEpi + kMinSeg, hi = total + kEpi * (n_units + 1) + kMinSeg;
        while (lo < hi) {
            const long long mid = (lo + hi) / 2;
            if (walk(mid, nullptr)) hi = mid; else lo = mid + 1;
        }
        while (!walk(lo, cuts.start)) ++lo;
        cuts.start[n_teams] = (uint32_t)total;
    }
    cfg.gridDim = dim3(2 * n_teams * n_pairs);
    return cudaLaunchKernelEx(&cfg, compress_tc2_kernel<D, HP>, tmK, tmV, s, c, L, cuts, per, gather ? 1 : 0);
}

}  // namespace

// True if the pair kernel serves this layout: what the single-CTA kernel needs, and an even number of row tiles.
bool compress_tc2_supported(const Dims& s) { return s.M % (2 * kBM) == 0; }

// True if the pair kernel can also write the kept-dim rows of the middle (its gather warps hold at most
// kGatherItems chunks per thread and stage); otherwise the partition kernel writes them.
bool compress_tc2_gathers(const Dims& s) {
    const int n_pairs = s.M / (2 * kBM);
    const int hp = s.Hkv % 2 == 0 ? 2 : 1;
    const int n_tok = (kBK + n_pairs - 1) / n_pairs;
    const int nf = s.nfk > s.nfv ? s.nfk : s.nfv;
    return n_tok * hp * (nf >> 3) <= kGatherItems * 32 * kGatherWarps;
}

// Coefficients (the caller has zeroed them) and, with gather, the kept-dim rows of the middle tokens; the windows
// and the counters are the caller's (the partition kernel).
cudaError_t launch_compress_tc2(const Dims& s, const CacheDev& c, const void* K, const void* V, int64_t sb, int64_t st,
                                int64_t sh, int L, bool ordered, bool gather, cudaStream_t stream) {
    const int n_init = L < s.l_init ? L : s.l_init;
    const int n_local = (L - n_init) < s.l_local ? (L - n_init) : s.l_local;
    const int n_mid = L - n_init - n_local;
    if (n_mid <= 0) return cudaSuccess;
    if (gather && !compress_tc2_gathers(s)) return cudaErrorInvalidValue;
    CUtensorMap tmK, tmV;
    if (!make_map2(&tmK, K, s, sb, st, sh, L) || !make_map2(&tmV, V, s, sb, st, sh, L)) return cudaErrorInvalidValue;
    const bool pair = s.Hkv % 2 == 0;                        // two heads share a CTA pair and its basis tiles
    if (s.d == 128) return pair ? launch_tc2_t<128, 2>(tmK, tmV, s, c, L, n_mid, ordered, gather, stream) : launch_tc2_t<128, 1>(tmK, tmV, s, c, L, n_mid, ordered, gather, stream);
    return pair ? launch_tc2_t<64, 2>(tmK, tmV, s, c, L, n_mid, ordered, gather, stream) : launch_tc2_t<64, 1>(tmK, tmV, s, c, L, n_mid, ordered, gather, stream);
}

}  // namespace fa
