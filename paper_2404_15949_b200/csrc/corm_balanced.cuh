// Decode kernel for bf16 caches with head_dim 128 and grouped query heads (group size 1, 2 or 4): one launch per
// step, every block the same share of the work.
//
// The step's work is the list of 32-key tiles of all units (a unit of l live keys has ceil(l / 32)). Every block
// computes that list's prefix sums from the live lengths itself and takes the tiles [T b / n, T (b + 1) / n) of it, so
// blocks differ by at most one tile whatever the units' lengths are; a block's range is cut into segments at unit
// boundaries. The four warps of a block stream the tiles of a segment in turn, each through its own ring of
// shared-memory stages: K tiles by bulk copies (a tile is one contiguous run of 256-byte rows), V tiles by 2-D
// tensor-map copies with the 128-byte swizzle, both completing on mbarriers with bounded waits.
//   Q.K   fp64 on the CUDA cores, as in corm_fast.cuh (qk_tile_pairs below): verdicts are compared with an fp64 oracle.
//   P.V   on the tensor cores: mma.m16n8k16 with A = V^T (ldmatrix.trans from the swizzled tile) and B = the
//         tile's probabilities, each split into two bf16 (p = hi + lo to ~2^-17 relative), the 2 G columns of B
//         being (head, hi / lo); fp32 accumulation. A group of four heads fills the 8 columns of one instruction.
//   softmax  per head against a fixed reference (the maximum of the warp's first tile of the segment) that moves only
//         when a logit exceeds it by more than 16; Z in fp64.
// Per segment every warp stores one record {m, Z, acc[128]} per head and the scaled logits of its tiles; warps never
// meet inside the streaming loop. Who applies Algorithm 1 afterwards depends on the kernel's form (template
// parameter MODE of decode_balanced_kernel): the verdict launch of corm_verdict.cuh, which reads the records through
// a per-unit record list (the default from per-step calls); the blocks that streamed a unit, once its records are
// all in, with the unit's last block compacting it (bal_finish_block); or, with a block per split instead of the
// balanced partition, the unit's last-arriving split alone, which is the form whose launches can be chained.
// Launched with programmatic stream serialization: a step's blocks set up their barriers while the previous
// step drains and wait for it (or, chained, for their own unit's previous step) before they read anything.
#pragma once

#include <cuda.h>

#include "corm_common.cuh"
#include "corm_fast.cuh"

namespace corm {

constexpr int kBalWarps = 4;
constexpr int kBalThreads = kBalWarps * 32;
constexpr int kBalKStages = 2;
constexpr int kBalStages = 3;                                   // 2 K + 1 V per warp
constexpr int kBalWarpBytes = kBalStages * kTileBytes;         // 24 KiB
constexpr int kBalRingBytes = kBalWarps * kBalWarpBytes;       // 96 KiB, reused by the finish phase
constexpr int kBalBlocksPerSm = 2;
constexpr int kBalSegCap = 32;                                  // segments listed per window of a block's range
constexpr int kBalRec = 16 + 4 * 128;                           // {double m, double Z, float acc[128]}
constexpr int kBalCacheUnits = 16384;                            // units whose lengths the prologue parks in shared memory
constexpr int kBalMaxTokens = 1 << 17;                          // the finish phase keeps 3 bits-per-32 arrays on chip

struct BalSeg {
    int32_t u;          // unit
    int32_t l;          // its live length including the token appended by this step
    int32_t tile0;      // first tile of the segment, counted inside the unit
    int32_t n_tiles;    // tiles of the segment
    int32_t gtile0;     // index of the unit's first tile in the step's tile list
    int32_t t;          // tokens the unit's sequence has seen, this one included
    int32_t n_unit;     // tiles of the whole unit
    int32_t pad;
};

// Small block-wide variables. The kernel declares no static shared memory at all: its dynamic shared memory then
// starts at the block's first usable byte, which is 1024-byte aligned, as the swizzled V tiles need (checked at entry).
struct BalMisc {
    unsigned long long stamp;     // kBalUnits, chained launch: the unit's stamp as tid 0 read it
    double thr[4], Zg[4];            // finish phase: thresholds and normalisers per head
    int scan[kBalThreads];           // finish phase: scratch of the block-wide prefix sums
    int wsum[kBalWarps];
    int first_u, first_P, nseg, more, next_u, next_P, last, failed;
};

// shared-memory carve-up behind the 1024-byte aligned ring
struct BalSmem {
    int psm, segq, segnew, bars, segs, misc, total, n_pre;
};
__host__ __device__ constexpr int bal_align128(int x) { return (x + 127) / 128 * 128; }
__host__ __device__ constexpr BalSmem bal_smem_layout(int G) {
    BalSmem s{};
    int off = kBalRingBytes;
    s.psm = off; off = bal_align128(off + kBalWarps * kTileKeys * 16);
    s.bars = off; off = bal_align128(off + kBalWarps * kBalStages * 8);
    s.segs = off; off = bal_align128(off + kBalSegCap * (int)sizeof(BalSeg));
    s.misc = off; off = bal_align128(off + (int)sizeof(BalMisc));
    // queries and appended rows of the first n_pre segments are fetched ahead; whatever shared memory is left
    const int budget = (228 * 1024) / kBalBlocksPerSm - 1024 /* system */;
    const int per = G * kRowBytes + 2 * kRowBytes;
    int n_pre = (budget - off) / per;
    if (n_pre > 8) n_pre = 8;
    if (n_pre < 1) n_pre = 1;
    s.n_pre = n_pre;
    s.segq = off; off = bal_align128(off + n_pre * G * kRowBytes);
    s.segnew = off; off = bal_align128(off + n_pre * 2 * kRowBytes);
    s.total = off;
    return s;
}

// ---- PTX wrappers of this kernel ----
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_m16n8k16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two floats -> one word of two bf16 (round to nearest even): `hi` in the upper half, `lo` in the lower
__device__ __forceinline__ uint32_t pack_bf16x2(float hi, float lo) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// qk_tile of corm_fast.cuh with the key slots taken in pairs (s, s + 4): the two slots' FMA chains run together
// (eight independent chains instead of four: a dependent fp64 FMA issues only every ~23 cycles) and the pair's first
// butterfly exchange follows at once, overlapping the next pair's arithmetic. Same lane -> key map, same sums up to
// the order of the additions. 2 % faster than qk_tile here (same GPU, long units).
template <int G>
__device__ __forceinline__ void qk_tile_pairs(const unsigned char* ktile, const double (&qd)[G][8], int lane,
                                              double (&sown)[G]) {
    const int h = lane >> 4, i = lane & 15, m = i >> 1, b0 = i & 1;
    double r[2][G];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        double b[G][4];
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            const int key0 = 16 * h + 8 * (it ^ b0) + (s ^ m), key1 = 16 * h + 8 * (it ^ b0) + ((s + 4) ^ m);
            const uint4 raw0 = *reinterpret_cast<const uint4*>(ktile + key0 * kRowBytes + i * 16);
            const uint4 raw1 = *reinterpret_cast<const uint4*>(ktile + key1 * kRowBytes + i * 16);
            double k0[8], k1[8];
            unpack8_to_double(raw0, k0);
            unpack8_to_double(raw1, k1);
            double a0[G], a1[G];
#pragma unroll
            for (int g = 0; g < G; ++g) { a0[g] = qd[g][0] * k0[0]; a1[g] = qd[g][0] * k1[0]; }
#pragma unroll
            for (int e = 1; e < 8; ++e)
#pragma unroll
                for (int g = 0; g < G; ++g) { a0[g] = fma(qd[g][e], k0[e], a0[g]); a1[g] = fma(qd[g][e], k1[e], a1[g]); }
#pragma unroll
            for (int g = 0; g < G; ++g) b[g][s] = a0[g] + __shfl_xor_sync(0xffffffffu, a1[g], 8);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int s = 0; s < 2; ++s) b[g][s] += __shfl_xor_sync(0xffffffffu, b[g][s + 2], 4);
            b[g][0] += __shfl_xor_sync(0xffffffffu, b[g][1], 2);
            r[it][g] = b[g][0];
        }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) sown[g] = r[0][g] + __shfl_xor_sync(0xffffffffu, r[1][g], 1);
}

// byte offset of 16-byte chunk c (0..15) of row r inside a V tile as the swizzled tensor copies lay it out: two
// halves of 64 channels, rows of 128 bytes, chunk index XOR (row mod 8)
__device__ __forceinline__ int vtile_offset(int r, int c) {
    return (c >> 3) * (kTileBytes / 2) + r * 128 + ((((c & 7) ^ r) & 7) << 4);
}

// records the balanced kernel may write in one step: one per warp of every (block, unit) pair on the tile list
__host__ __device__ inline size_t bal_record_count(int n_blocks, int U) { return ((size_t)n_blocks + (size_t)U) * kBalWarps; }

// A block per split (kBalUnits): unit u keeps its records (one per warp and split) at a place that does not depend on
// the launch, because chained launches overlap: another unit's previous step may still be reading its own. A quarter
// of the splits the arena provides records for, times four warps.
__host__ __device__ inline int bal_unit_splits(int max_splits) { return max_splits >= 4 ? max_splits / 4 : 1; }

// block of the balanced partition that owns tile x of the step's list (T tiles, n blocks)
__device__ __forceinline__ int bal_block_of(long long x, long long T, int n) { return (int)(((x + 1) * n - 1) / T); }

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Per-segment bookkeeping of the finish phase (shared memory).
struct BalFin {
    int32_t rec0, n_blocks, tile_prefix, evict_on, last, sc_off, first;
    int32_t pad;
};

// Finish phase of a block, by all its NT threads, after its streaming: Algorithm 1 for the slots of ALL the block's
// segments in one pass, so that a block with several segments pays the chain of dependent memory round trips once.
//   A. registers, positions and logits of the block's slots (its own stores and older data) are requested; then the
//      block waits (bounded) until the arrival counter of each of its units says all records are stored. Every block
//      of the launch is resident or becomes resident without anybody's help (the grid is no larger than the resident
//      slots, and a launch only starts once every block of the previous one has started), and every warp stores all
//      its records before the block waits for anything, so the waits end.
//   B. thresholds of Definition 3.1 per (segment, head) from the unit's records: one warp per pair, a record per
//      lane, fixed reduction trees, so every block of a unit gets the same bits.
//   C. verdicts of the slots (OR over the group), register update, keep bits to the unit's global bit mask
//      (segments are whole tiles, so no two blocks share a mask word).
//   D. the unit's first block reduces the accumulators to the output of Eq. 1; after a second arrival counter the
//      unit's last block scans the mask, fills the holes and publishes the new length.
// scratch: the block's ring area, free by now.
// UNIT: the block is the last-arriving split of the one unit in segs[0] (a block per split, kBalUnits) and finishes
// the whole unit alone: all the unit's records are stored, nothing is waited for, and the unit's stamp is left.
template <int G, bool PAGED, int NT, bool UNIT>
__device__ void bal_finish_block(const DecodeParams& p, const BalSeg* segs, int nseg, int blk, long long T, int nblk,
                                 unsigned char* scratch, BalMisc* misc) {
    constexpr int NW = kBalWarps;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    BalFin* fin = reinterpret_cast<BalFin*>(scratch);                         // [kBalSegCap]
    double* thr = reinterpret_cast<double*>(scratch + kBalSegCap * sizeof(BalFin));   // [kBalSegCap][4]
    double* Zg = thr + kBalSegCap * 4;                                         // [kBalSegCap][4]
    float* sc_sm = reinterpret_cast<float*>(Zg + kBalSegCap * 4);              // scale factors of the records this block reduces
    unsigned char* comp = scratch + 32 * 1024;                                 // compaction arrays (behind at most 21 KB of factors)
    const size_t pstride = partial_stride(128);
    if (tid == 0) {
        int tp = 0, off = 0;
        for (int si = 0; si < nseg; ++si) {
            const BalSeg& sg = segs[si];
            const long long P0 = sg.gtile0;
            const int fb = UNIT ? 0 : bal_block_of(P0, T, nblk);
            BalFin f;
            f.n_blocks = UNIT ? sg.pad : bal_block_of(P0 + sg.n_unit - 1, T, nblk) - fb + 1;
            f.rec0 = UNIT ? sg.u * bal_unit_splits(p.max_splits) * NW : (fb + sg.u) * NW;
            f.tile_prefix = tp;
            f.evict_on = min(p.w, __ldcg(p.base_obs + sg.u / p.Hkv) + p.step + 1) >= p.w;
            f.last = UNIT ? 1 : 0;
            f.first = UNIT || fb == blk;
            f.sc_off = off;
            f.pad = 0;
            if (f.first) off += G * f.n_blocks * NW;
            tp += sg.n_tiles;
            fin[si] = f;
        }
        misc->last = tp;                                                       // tiles of the block in this window
    }
    __syncthreads();
    const int n_slots = misc->last * kTileKeys;

    // ---- A. the block's slots, batch by batch (one batch unless units are long) ----
    constexpr int kB = (G == 4 ? 6 : 8);                                       // slots per thread and batch
    double sv[kB][G];
    uint32_t wv[kB];
    int32_t pv[kB], jv[kB], siv[kB];
    auto load_batch = [&](int base0) {
#pragma unroll
        for (int k = 0; k < kB; ++k) {
            const int x = base0 + k * NT + tid;
            wv[k] = 0u; pv[k] = 0; jv[k] = -1; siv[k] = 0;
#pragma unroll
            for (int g = 0; g < G; ++g) sv[k][g] = -INFINITY;
            if (x < n_slots) {
                const int tile = x >> 5;
                int si = 0;
                while (si + 1 < nseg && fin[si + 1].tile_prefix <= tile) ++si;
                const BalSeg& sg = segs[si];
                const int j = (sg.tile0 + tile - fin[si].tile_prefix) * kTileKeys + (x & 31);
                siv[k] = si;
                if (j < sg.l) {
                    jv[k] = j;
                    const double* st = p.stash + ((size_t)sg.u * p.C + j) * G;
                    if (G == 4) {
                        const double2 a = __ldcg(reinterpret_cast<const double2*>(st));
                        const double2 c = __ldcg(reinterpret_cast<const double2*>(st + 2));
                        sv[k][0] = a.x; sv[k][1] = a.y; sv[k][2 % G] = c.x; sv[k][3 % G] = c.y;
                    } else if (G == 2) {
                        const double2 a = __ldcg(reinterpret_cast<const double2*>(st));
                        sv[k][0] = a.x; sv[k][1 % G] = a.y;
                    } else {
                        sv[k][0] = __ldcg(st);
                    }
                    wv[k] = __ldcg(p.word + (size_t)sg.u * p.C + j);
                    pv[k] = __ldcg(p.pos + (size_t)sg.u * p.C + j);
                }
            }
        }
    };
    load_batch(0);
    if (!UNIT && tid == 0) {
        const long long start = clock64();
        for (int si = 0; si < nseg && !misc->failed; ++si) {
            if (fin[si].n_blocks == 1) continue;                               // a block's own warps arrived before its last barrier
            const uint32_t want = (uint32_t)(fin[si].n_blocks * NW);
            while (ld_acquire_u32(p.ticket + segs[si].u) < want) {
                if (clock64() - start > kWaitLimitCycles) { misc->failed = 1; break; }
                __nanosleep(64);
            }
        }
    }
    __syncthreads();
    if (misc->failed) { if (tid == 0) report_status(p.status, CORM_ERR_TIMEOUT); return; }

    // ---- B. thresholds: warp w takes the (segment, head) pairs w, w + NW, ... ----
    for (int task = warp; task < nseg * G; task += NW) {
        const int si = task / G, g = task - si * G;
        const BalFin f = fin[si];
        const int n_rec = f.n_blocks * NW;
        const unsigned char* rec_u = p.partials + ((size_t)f.rec0 * G + g) * pstride;
        double m = -INFINITY;
        for (int s0 = 0; s0 < n_rec; s0 += 128) {                              // four records per lane in flight
            double mm[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int s_ = s0 + k * 32 + lane;
                mm[k] = s_ < n_rec ? __ldcg(reinterpret_cast<const double*>(rec_u + (size_t)s_ * G * pstride)) : -INFINITY;
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) m = fmax(m, mm[k]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
        double Z = 0.0;
        for (int s0 = 0; s0 < n_rec; s0 += 128) {
            double2 mz[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int s_ = s0 + k * 32 + lane;
                mz[k] = s_ < n_rec ? __ldcg(reinterpret_cast<const double2*>(rec_u + (size_t)s_ * G * pstride)) : make_double2(-INFINITY, 0.0);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int s_ = s0 + k * 32 + lane;
                const double sc = exp_nonpos(mz[k].x - m);
                Z += mz[k].y * sc;
                if (f.first && s_ < n_rec) sc_sm[f.sc_off + g * n_rec + s_] = (float)sc;
            }
        }
        Z = warp_sum(Z);
        if (lane == 0) {
            Zg[si * 4 + g] = Z;
            thr[si * 4 + g] = m + log(Z) + p.log_alpha - log((double)segs[si].t);   // Definition 3.1: s >= lse + ln(alpha) - ln(t)
        }
    }
    __syncthreads();

    // ---- C. verdicts, register update, keep flags ----
    int n_imp = 0;
    for (int base0 = 0; base0 < n_slots; base0 += kB * NT) {
        if (base0) load_batch(base0);
#pragma unroll
        for (int k = 0; k < kB; ++k) {
            const int base = base0 + k * NT;
            if (base >= n_slots) break;                                         // uniform
            const int si = siv[k], j = jv[k];
            const BalSeg& sg = segs[si];
            bool keep = false;
            if (j >= 0) {
                bool imp = false;
#pragma unroll
                for (int g = 0; g < G; ++g) imp |= (sv[k][g] >= thr[si * 4 + g]);
                const uint32_t wd = update_register(wv[k], imp, p.w, sg.t);
                if (CORM_IN_RANGE(j < p.C, p.status)) p.word[(size_t)sg.u * p.C + j] = wd;
                keep = !fin[si].evict_on || register_needed(wd, p.w, sg.t) || pv[k] > sg.t - p.r;
                n_imp += imp ? 1 : 0;
            }
            const uint32_t ballot = __ballot_sync(0xffffffffu, keep);           // a warp's 32 slots are one tile of one segment
            const int x0 = base + warp * 32;
            if (lane == 0 && x0 < n_slots) {
                const int tile = x0 >> 5;
                int s2 = 0;
                while (s2 + 1 < nseg && fin[s2 + 1].tile_prefix <= tile) ++s2;
                const int kw = segs[s2].tile0 + tile - fin[s2].tile_prefix;
                if (CORM_IN_RANGE(kw >= 0 && kw < keepmask_words(p.C), p.status))
                    p.keepmask[(size_t)segs[s2].u * keepmask_words(p.C) + kw] = ballot;
            }
        }
    }
    warp_count(p.counters + CNT_IMPORTANT, n_imp);                             // Section 3.1's sparsity
    __threadfence();
    __syncthreads();
    if (!UNIT && tid < nseg) {
        const int si = tid, u = segs[si].u;
        const unsigned prev = atomicAdd(p.ticket2 + u, 1u);
        if (prev == (unsigned)(fin[si].n_blocks - 1)) {
            fin[si].last = 1;
            p.ticket2[u] = 0u; p.ticket[u] = 0u;                                // every block of the unit is past its wait
        }
        __threadfence();
    }
    // ---- D. Eq. 1 for the units that start in this block (thread = channel), while the arrivals above are in flight ----
    for (int si = 0; si < nseg; ++si) {
        const BalFin f = fin[si];
        if (!f.first) continue;                                                 // uniform: written before the barriers above
        const int n_rec = f.n_blocks * NW, u = segs[si].u;
        const unsigned char* rec_u = p.partials + (size_t)f.rec0 * G * pstride;
        float acc[G];
#pragma unroll
        for (int g = 0; g < G; ++g) acc[g] = 0.f;
        for (int s0 = 0; s0 < n_rec; s0 += 8) {                                 // 8 G values in flight
            float a[8][G];
#pragma unroll
            for (int k = 0; k < 8; ++k)
#pragma unroll
                for (int g = 0; g < G; ++g)
                    a[k][g] = s0 + k < n_rec ? __ldcg(reinterpret_cast<const float*>(rec_u + ((size_t)(s0 + k) * G + g) * pstride + 16) + tid) : 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k)
#pragma unroll
                for (int g = 0; g < G; ++g)
                    if (s0 + k < n_rec) acc[g] += a[k][g] * sc_sm[f.sc_off + g * n_rec + s0 + k];
        }
#pragma unroll
        for (int g = 0; g < G; ++g)
            Elem<bf16_t>::store(reinterpret_cast<bf16_t*>(p.out) + ((size_t)u * G + g) * 128 + tid, (float)((double)acc[g] / Zg[si * 4 + g]));
    }
    __syncthreads();

    // ---- the units this block is the last of: compaction ----
    for (int si = 0; si < nseg; ++si) {
        if (!fin[si].last) continue;                                            // uniform
        const BalSeg& sg = segs[si];
        const int u = sg.u, l = sg.l, t = sg.t, words = (l + 31) / 32 + 2, nwords = (l + 31) / 32;
        uint32_t* keep_sm = reinterpret_cast<uint32_t*>(comp);
        int* prefix = reinterpret_cast<int*>(keep_sm + words);
        int32_t* pt_sm = prefix + words;
        const int32_t* pt_u = PAGED ? p.page_table + (size_t)u * p.pt_stride : nullptr;
        const uint32_t* keep_g = p.keepmask + (size_t)u * keepmask_words(p.C);
        uint32_t* wordu = p.word + (size_t)u * p.C;
        int32_t* posu = p.pos + (size_t)u * p.C;
        for (int i = tid; i < nwords; i += NT) {
            keep_sm[i] = __ldcg(keep_g + i);
            if (PAGED) pt_sm[i] = __ldcg(pt_u + i);
        }
        __syncthreads();
        int new_len = l, n_moved = 0;
        if (fin[si].evict_on) {
            block_popc_scan<NT>(keep_sm, prefix, nwords, misc->scan);
            new_len = prefix[nwords];
            if (new_len < l) {
                const int kept_below = kept_before(keep_sm, prefix, new_len);
                n_moved = new_len - kept_below;
                int* holes = reinterpret_cast<int*>(p.stash + (size_t)u * G * p.C);   // every block is done with the logits
                int* movers = holes + p.C;
                for (int i = tid; i < nwords; i += NT) {
                    const uint32_t m = keep_sm[i];
                    const int w0 = i * 32;
                    const uint32_t valid = l - w0 >= 32 ? 0xffffffffu : (1u << (l - w0)) - 1u;
                    const uint32_t below = new_len - w0 >= 32 ? 0xffffffffu : (new_len > w0 ? (1u << (new_len - w0)) - 1u : 0u);
                    uint32_t hm = ~m & valid & below;                       // evicted slots below the new length
                    while (hm) {
                        const int bit = __ffs(hm) - 1;
                        hm &= hm - 1u;
                        holes[w0 - prefix[i] + __popc(~m & ((1u << bit) - 1u))] = w0 + bit;
                    }
                    uint32_t km = m & valid & ~below;                       // kept slots at or above it
                    while (km) {
                        const int bit = __ffs(km) - 1;
                        km &= km - 1u;
                        movers[prefix[i] + __popc(m & ((1u << bit) - 1u)) - kept_below] = w0 + bit;
                    }
                }
                __syncthreads();
                const size_t slab_row0 = (size_t)u * p.C;
                block_move_rows<bf16_t, 128, NT>(
                    reinterpret_cast<bf16_t*>(p.K), reinterpret_cast<bf16_t*>(p.V),
                    [&](int slot) -> size_t {
                        return PAGED ? page_row(pt_sm[slot >> 5], slot, p.pool_pages, p.status) : slab_row0 + (size_t)slot;
                    },
                    wordu, posu, movers, holes, n_moved, 0, 1, l, p.status);
            }
        }
        if (PAGED) settle_pages<NT>(p.page_table, p.page_bits, p.page_room, p.pool_pages, p.pt_stride, p.U, u, l - 1, new_len);
        if (UNIT && p.unit_stamp) __syncthreads();                      // every warp's row moves come before the stamp
        if (tid == 0) {
            p.live_out[u] = new_len;
            if (UNIT) publish_unit_stamp(p, u, new_len);
            publish_live(p.maxlive, p.step + 1, new_len);
            atomicAdd(p.counters + CNT_APPENDED, 1ull);
            atomicAdd(p.counters + CNT_ATTENDED, (unsigned long long)l);
            if (new_len < l) atomicAdd(p.counters + CNT_EVICTED, (unsigned long long)(l - new_len));
            if (n_moved) atomicAdd(p.counters + CNT_MOVED, (unsigned long long)n_moved);
        }
        __syncthreads();                                                     // the arrays are reused by the next unit
        (void)t;
    }
}

// MODE kBalStream: the kernel only streams, lists each unit's records in p.unit_rec and leaves verdicts and compaction
// to the verdict launch that follows it. kBalFinish: Algorithm 1 is finished inside this launch by the blocks that
// streamed a unit (bal_finish_block). kBalUnits: no balanced partition; grid (splits, units), a block streams one split
// of one unit (p.split_len keys) and the unit's last-arriving block finishes it alone. No block of such a launch waits
// for another, a finished unit leaves its stamp, and the launch may be chained to the previous step's (see
// decode_fast_kernel): with many short units the steps then overlap unit by unit.
constexpr int kBalStream = 0, kBalFinish = 1, kBalUnits = 2;
template <int G, bool PAGED, int MODE>
__global__ void __launch_bounds__(kBalThreads, kBalBlocksPerSm)
decode_balanced_kernel(const __grid_constant__ DecodeParams p, const __grid_constant__ CUtensorMap vmap) {
    constexpr bool FINISH = MODE == kBalFinish;
    extern __shared__ __align__(1024) unsigned char smem[];   // the swizzled V tiles want 1024-byte alignment
    constexpr int NT = kBalThreads, NW = kBalWarps;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nblk = (int)gridDim.x, blk = (int)blockIdx.x;
    constexpr BalSmem lay = bal_smem_layout(G);           // compile-time offsets: no registers held for them
    unsigned char* my_tiles = smem + warp * kBalWarpBytes;
    const uint32_t my_bars = smem_addr(smem + lay.bars) + warp * kBalStages * 8;
    unsigned char* psm = smem + lay.psm + warp * kTileKeys * 16;
    BalSeg* segs = reinterpret_cast<BalSeg*>(smem + lay.segs);
    BalMisc* misc = reinterpret_cast<BalMisc*>(smem + lay.misc);
    int* s_wsum = misc->wsum;
    int &s_first_u = misc->first_u, &s_first_P = misc->first_P, &s_nseg = misc->nseg, &s_more = misc->more,
        &s_next_u = misc->next_u, &s_next_P = misc->next_P, &s_failed = misc->failed;
    unsigned char* Kl = reinterpret_cast<unsigned char*>(p.K);
    unsigned char* Vl = reinterpret_cast<unsigned char*>(p.V);

    // ---- set-up that reads nothing the previous step writes ----
    if (smem_addr(smem) & 1023u) {                          // never expected; reported instead of mis-reading tiles
        if (tid == 0) report_status(p.status, CORM_ERR_INTERNAL);
        return;
    }
    if (tid == 0) { prefetch_tensormap(&vmap); s_failed = 0; }
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kBalStages; ++s) mbar_init(my_bars + s * 8, 1);
        fence_mbar_init();
        fence_async_smem();
    }
    if (MODE == kBalUnits) {
        // ---- one split of one unit ----
        const int u = (int)blockIdx.y, split = (int)blockIdx.x;
        int l_old;
        if (p.chain_wait) {                                   // this unit's previous step, not the previous launch
            if (tid == 0) misc->stamp = wait_unit_stamp(p.unit_stamp + u, (uint32_t)p.step, p.status);
            __syncthreads();
            const unsigned long long sw = misc->stamp;
            if ((uint32_t)(sw >> 32) != (uint32_t)p.step) return;   // the wait gave up (reported), or a block without a split
            l_old = (int)(uint32_t)sw;
            asm volatile("fence.proxy.async.global;" ::: "memory");   // the tile copies read rows that ordinary stores wrote
        } else {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            l_old = __ldcg(p.live_in + u);
        }
        const int l = l_old + 1;
        const int room = PAGED ? __ldcg(p.page_room + u) : 1;
        if (l > p.C || !room) {                               // a full slab or an exhausted pool: reported, the unit is left as it is
            if (split == 0 && tid == 0) {
                report_status(p.status, CORM_ERR_CAPACITY);
                p.live_out[u] = l_old;
                publish_unit_stamp(p, u, l_old);
                publish_live(p.maxlive, p.step + 1, l_old);
            }
            return;
        }
        const int n_unit = (l + kTileKeys - 1) / kTileKeys;
        const int n_act = (n_unit + p.split_len / kTileKeys - 1) / (p.split_len / kTileKeys);
        if (split >= n_act) return;
        const int tps = (n_unit + n_act - 1) / n_act;          // the unit's tiles shared out evenly over its splits
        if (n_act > (int)gridDim.x && split == 0 && tid == 0) report_status(p.status, CORM_ERR_INTERNAL);   // the host's bound on the unit was wrong
        if (p.early_trigger) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // every block has its length by now
        if (tid == 0) {
            BalSeg sg;
            sg.u = u; sg.l = l; sg.tile0 = min(n_unit, split * tps); sg.n_tiles = max(0, min(tps, n_unit - split * tps)); sg.gtile0 = 0;
            sg.t = __ldcg(p.base_tokens + u / p.Hkv) + p.step + 1; sg.n_unit = n_unit; sg.pad = n_act;
            segs[0] = sg;
            s_nseg = 1; s_more = 0;
        }
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");   // the previous launch on the stream has completed
    }

    // ---- the step's tile list: tiles per unit, block-wide prefix sums, this block's range ----
    // One round of global loads: every unit's length (and every sequence's token count) is parked in the ring area,
    // which holds no tile yet, so that locating the block's range and listing its first segments read shared memory.
    const int U = p.U, n_seq = U / p.Hkv;
    const bool cached = U <= kBalCacheUnits;
    int32_t* s_L = reinterpret_cast<int32_t*>(smem);                 // [U] live length incl. the new token, 0 = unit skipped
    int32_t* s_bt = s_L + kBalCacheUnits;                            // [n_seq] tokens seen before this launch's steps
    const int per = (U + NT - 1) / NT, lo = min(U, tid * per), hi = min(U, lo + per);
    auto len_global = [&](int v) -> int {                            // live length incl. the new token, 0 if the unit cannot take it
        const int l = __ldcg(p.live_in + v) + 1;
        const int room = PAGED ? __ldcg(p.page_room + v) : 1;
        return (l <= p.C && room) ? l : 0;
    };
    bool use_cache = cached;
    auto len_of = [&](int v) -> int { return use_cache ? s_L[v] : len_global(v); };
    auto tokens_of = [&](int v) -> int { return (use_cache ? s_bt[v / p.Hkv] : __ldcg(p.base_tokens + v / p.Hkv)) + p.step + 1; };
    long long T = 0, S_b = 0, S_e = 0;
    int win_u = 0, win_P = 0;
    if (MODE != kBalUnits) {
    if (cached)
        for (int i = tid; i < n_seq; i += NT) s_bt[i] = __ldcg(p.base_tokens + i);
    int sum = 0;
    for (int v = lo; v < hi; ++v) {
        const int l = len_global(v);
        if (cached) s_L[v] = l;
        if (!l && blk == 0) {        // a full slab or an exhausted pool: reported, the unit is left as it is
            const int l_old = __ldcg(p.live_in + v);
            report_status(p.status, CORM_ERR_CAPACITY);
            p.live_out[v] = l_old;
            publish_live(p.maxlive, p.step + 1, l_old);
        }
        sum += (l + kTileKeys - 1) / kTileKeys;
    }
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    int excl = incl - sum;
#pragma unroll
    for (int w = 0; w < NW; ++w) { if (w < warp) excl += s_wsum[w]; T += s_wsum[w]; }
    if (T == 0) return;
    S_b = T * blk / nblk; S_e = T * (blk + 1) / nblk;
    if (S_b == S_e) return;                                    // more blocks than tiles
    if (sum > 0 && excl <= S_b && S_b < (long long)excl + sum) {
        int run = excl;
        for (int v = lo; v < hi; ++v) {
            const int tv = (len_of(v) + kTileKeys - 1) / kTileKeys;
            if (S_b < (long long)run + tv) { s_first_u = v; s_first_P = run; break; }
            run += tv;
        }
    }
    __syncthreads();
    win_u = s_first_u; win_P = s_first_P;
    }

    const int h = lane >> 4, ci = lane & 15;
    const int key_own = 16 * h + 8 * (ci & 1) + (ci >> 1);     // tile key this lane owns after the fold of qk_tile
    const double inv_root_d = 0.088388347648318440550;        // 1/sqrt(128)
    // ldmatrix row addresses of this lane inside a V tile: matrix lane/8 of a 16 x 16 block = keys (lane/16)*8 + lane%8,
    // channels + 8 for the odd matrices; the chunk index is XORed with the row (lane % 8) by the swizzle
    const int lm_row = ((lane >> 4) << 3) + (lane & 7), lm_odd = (lane >> 3) & 1, lm_x = lane & 7;
    int n_consumed = 0;                                        // tiles this warp has consumed: ring slots and parities
    bool failed = false;

    for (;;) {   // windows of at most kBalSegCap segments (one window unless units are tiny)
        if (MODE != kBalUnits && warp == 0) {
            // lanes look at units win_u + lane; a unit with tiles that starts before the end of the range is a segment
            const int v = win_u + lane;
            const int l = v < U ? len_of(v) : 0, tv = (l + kTileKeys - 1) / kTileKeys;
            int inc = tv;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += up;
            }
            const long long Pv = (long long)win_P + inc - tv;   // index of the unit's first tile in the list
            const bool is_seg = tv > 0 && Pv < S_e && Pv + tv > S_b;
            const uint32_t segmask = __ballot_sync(0xffffffffu, is_seg);
            if (is_seg) {
                BalSeg sg;
                const long long a = Pv > S_b ? Pv : S_b, e = Pv + tv < S_e ? Pv + tv : S_e;
                sg.u = v; sg.l = l; sg.tile0 = (int)(a - Pv); sg.n_tiles = (int)(e - a); sg.gtile0 = (int)Pv;
                sg.t = tokens_of(v); sg.n_unit = tv; sg.pad = 0;
                segs[__popc(segmask & ((1u << lane) - 1u))] = sg;
            }
            const long long P_end = (long long)win_P + __shfl_sync(0xffffffffu, inc, 31);
            if (lane == 0) {
                s_nseg = __popc(segmask);
                s_more = (P_end < S_e && win_u + 32 < U) ? 1 : 0;
                s_next_u = win_u + 32;
                s_next_P = (int)P_end;
            }
        }
        __syncthreads();
        use_cache = false;                                     // the ring is about to receive tiles
        const int nseg = s_nseg;

        // ---- this warp's tiles: cursor (segment, index among the warp's tiles of that segment) ----
        struct Cur { int si, it; };
        auto seg_has = [&](int si) { return segs[si].n_tiles > warp; };
        auto cur_first = [&]() { Cur c{0, 0}; while (c.si < nseg && !seg_has(c.si)) ++c.si; return c; };
        auto cur_next = [&](Cur c) {
            if (c.si >= nseg) return c;
            ++c.it;
            if (warp + c.it * NW >= segs[c.si].n_tiles) { c.it = 0; do { ++c.si; } while (c.si < nseg && !seg_has(c.si)); }
            return c;
        };
        // first row of a tile in the layer's K / V storage; a page entry outside the pool (a broken table) is
        // reported and page 0 is read instead, so that no address is ever formed from it
        auto tile_row0 = [&](const BalSeg& sg, int ti) -> long long {
            if (!PAGED) return (long long)sg.u * p.C + (long long)ti * kTileKeys;
            const int pg = __ldcg(p.page_table + (size_t)sg.u * p.pt_stride + ti);
            if (pg <= 0 || pg > p.pool_pages) { report_status(p.status, CORM_ERR_INTERNAL); return -1; }
            return (long long)(pg - 1) * kPageKeys;
        };
        auto issue_k = [&](Cur c, int n) {                     // lane 0 only
            const BalSeg& sg = segs[c.si];
            const int ti = sg.tile0 + warp + c.it * NW, slot = n % kBalKStages;
            const uint32_t bytes = (uint32_t)min(kTileKeys, sg.l - ti * kTileKeys) * kRowBytes;
            long long row0 = tile_row0(sg, ti);
            if (row0 < 0) row0 = 0;
            mbar_expect_tx(my_bars + slot * 8, bytes);
            bulk_load(smem_addr(my_tiles + slot * kTileBytes), Kl + row0 * kRowBytes, bytes, my_bars + slot * 8);
        };
        auto issue_v = [&](Cur c) {                            // lane 0 only; the box is always 32 rows
            const BalSeg& sg = segs[c.si];
            const int ti = sg.tile0 + warp + c.it * NW;
            long long row0 = tile_row0(sg, ti);
            if (row0 < 0) row0 = 0;
            const uint32_t bar = my_bars + kBalKStages * 8, dst = smem_addr(my_tiles + kBalKStages * kTileBytes);
            mbar_expect_tx(bar, kTileBytes);
            tma_load_2d(dst, &vmap, 0, (int)row0, bar);
            tma_load_2d(dst + kTileBytes / 2, &vmap, 64, (int)row0, bar);
        };
        Cur cc = cur_first(), ck = cc, cv = cc;
        int nk = n_consumed;
        if (lane == 0) {
            fence_async_smem();
            for (int s = 0; s < kBalKStages && ck.si < nseg; ++s) { issue_k(ck, nk); ++nk; ck = cur_next(ck); }
            if (cv.si < nseg) { issue_v(cv); cv = cur_next(cv); }
        } else {
            for (int s = 0; s < kBalKStages && ck.si < nseg; ++s) { ++nk; ck = cur_next(ck); }
            if (cv.si < nseg) cv = cur_next(cv);
        }
        // queries and appended rows of the first segments, fetched while the first tiles are on their way
        {
            const int n_pre = min(nseg, lay.n_pre);
            const int per_seg = G * 16 + 32;
            for (int x = tid; x < n_pre * per_seg; x += NT) {
                const int si = x / per_seg, c = x - si * per_seg;
                const BalSeg& sg = segs[si];
                if (c < G * 16) {
                    cp_async16(smem_addr(smem + lay.segq + (si * G * 16 + c) * 16),
                               reinterpret_cast<const unsigned char*>(p.q) + ((size_t)sg.u * G * 16 + c) * 16);
                } else if (sg.tile0 + sg.n_tiles == sg.n_unit) {          // the segment holds the unit's last tile
                    const int cc2 = c - G * 16;
                    const unsigned char* src = cc2 < 16 ? reinterpret_cast<const unsigned char*>(p.k_new) + ((size_t)sg.u * 16 + cc2) * 16
                                                        : reinterpret_cast<const unsigned char*>(p.v_new) + ((size_t)sg.u * 16 + cc2 - 16) * 16;
                    cp_async16(smem_addr(smem + lay.segnew + (si * 32 + cc2) * 16), src);
                }
            }
            cp_async_wait_all();
        }
        __syncthreads();

        for (int si = 0; si < nseg; ++si) {
            const BalSeg sg = segs[si];
            const int u = sg.u, l = sg.l, l_old = l - 1, t = sg.t;
            double M[G], Zl[G];
            float Mref[G];
            float accd[8][4];
#pragma unroll
            for (int g = 0; g < G; ++g) { M[g] = -INFINITY; Zl[g] = 0.0; Mref[g] = -INFINITY; }
#pragma unroll
            for (int cb = 0; cb < 8; ++cb)
#pragma unroll
                for (int e = 0; e < 4; ++e) accd[cb][e] = 0.f;
            if (cc.si == si) {
                // the lane's 8 channels of every query head, widened to fp64
                double qd[G][8];
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const uint4 raw = si < lay.n_pre ? *reinterpret_cast<const uint4*>(smem + lay.segq + ((si * G + g) * 16 + ci) * 16)
                                                     : __ldcg(reinterpret_cast<const uint4*>(p.q) + ((size_t)u * G + g) * 16 + ci);
                    unpack8_to_double(raw, qd[g]);
                }
                uint32_t* wordu = p.word + (size_t)u * p.C;
                int32_t* posu = p.pos + (size_t)u * p.C;
                bool first = true;
                while (cc.si == si) {
                    const int ti = sg.tile0 + warp + cc.it * NW;
                    const int k0 = ti * kTileKeys;
                    const int n_valid = min(kTileKeys, l - k0);
                    const bool has_new = (l_old >= k0 && l_old < k0 + kTileKeys);   // this tile holds the appended token
                    const int kslot = n_consumed % kBalKStages;
                    unsigned char* ktile = my_tiles + kslot * kTileBytes;
                    unsigned char* vtile = my_tiles + kBalKStages * kTileBytes;
                    // the appended token's row (K or V, `which` 0 / 1) as fetched ahead, or from global memory
                    auto new_row = [&](int which) -> uint4 {
                        if (si < lay.n_pre) return *reinterpret_cast<const uint4*>(smem + lay.segnew + (si * 32 + which * 16 + (lane & 15)) * 16);
                        return __ldcg(reinterpret_cast<const uint4*>(which ? p.v_new : p.k_new) + (size_t)u * 16 + (lane & 15));
                    };
                    if (!failed && !mbar_wait(my_bars + kslot * 8, (n_consumed / kBalKStages) & 1)) failed = true;   // once one wait has expired the rest are skipped
                    if (has_new) {   // append: the new row goes to the cache and into the arriving tile
                        const long long row0 = tile_row0(sg, ti);
                        if (row0 >= 0 && lane < 16) {
                            const uint4 newk = new_row(0);
                            *reinterpret_cast<uint4*>(ktile + (l_old - k0) * kRowBytes + lane * 16) = newk;
                            reinterpret_cast<uint4*>(Kl + (row0 + (l_old - k0)) * kRowBytes)[lane] = newk;
                        }
                        if (row0 >= 0 && lane == 0) { wordu[l_old] = 0u; posu[l_old] = t; }
                        __syncwarp();
                    }
                    double sown[G];
                    qk_tile_pairs<G>(ktile, qd, lane, sown);
                    __syncwarp();
                    if (ck.si < nseg) {
                        if (lane == 0) { fence_async_smem(); issue_k(ck, nk); }
                        ++nk; ck = cur_next(ck);
                    }

                    const bool valid = key_own < n_valid;
                    const int j_own = k0 + key_own;
                    double sv[G], ex[G];
#pragma unroll
                    for (int g = 0; g < G; ++g) sv[g] = valid ? sown[g] * inv_root_d : -INFINITY;   // Eq. 2's exponent
                    bool over = first;
#pragma unroll
                    for (int g = 0; g < G; ++g) over |= ((float)sv[g] > Mref[g] + 16.f);
                    if (__any_sync(0xffffffffu, over)) {      // the reference moves: first tile, or a logit far above it (rare)
                        float mt[G];
#pragma unroll
                        for (int g = 0; g < G; ++g) mt[g] = (float)sv[g];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                            for (int g = 0; g < G; ++g) mt[g] = fmaxf(mt[g], __shfl_xor_sync(0xffffffffu, mt[g], o));
                        float scf[G];
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            const float mn = fmaxf(Mref[g], mt[g]);
                            const double sc = first ? 0.0 : exp_nonpos((double)Mref[g] - (double)mn);
                            Zl[g] *= sc;
                            scf[g] = (float)sc;
                            Mref[g] = mn;
                        }
                        // accumulators of this thread belong to head lane % 4
                        float mine = scf[0];
#pragma unroll
                        for (int g = 1; g < G; ++g) mine = (lane & 3) == g ? scf[g] : mine;
#pragma unroll
                        for (int cb = 0; cb < 8; ++cb)
#pragma unroll
                            for (int e = 0; e < 4; ++e) accd[cb][e] *= mine;
                        first = false;
                    }
                    uint32_t pw[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        ex[g] = valid ? exp_nonpos(sv[g] - (double)Mref[g]) : 0.0;
                        Zl[g] += ex[g];
                        const float pf = (float)ex[g];
                        const float hi_f = __uint_as_float(pack_bf16x2(0.f, pf) << 16);
                        pw[g] = pack_bf16x2(pf - hi_f, pf);                 // column 2g = hi, column 2g + 1 = lo
                    }
                    *reinterpret_cast<uint4*>(psm + key_own * 16) = make_uint4(pw[0], pw[1], pw[2], pw[3]);
                    if (valid && CORM_IN_RANGE(j_own < p.C, p.status)) {
                        double* dst = p.stash + ((size_t)u * p.C + j_own) * G;
                        if (G == 4) {
                            reinterpret_cast<double2*>(dst)[0] = make_double2(sv[0], sv[1]);
                            reinterpret_cast<double2*>(dst)[1] = make_double2(sv[2 % G], sv[3 % G]);
                        } else if (G == 2) {
                            reinterpret_cast<double2*>(dst)[0] = make_double2(sv[0], sv[1 % G]);
                        } else {
                            dst[0] = sv[0];
                        }
                    }
                    __syncwarp();

                    if (!failed && !mbar_wait(my_bars + kBalKStages * 8, n_consumed & 1)) failed = true;
                    if (has_new) {
                        const long long row0 = tile_row0(sg, ti);
                        if (row0 >= 0 && lane < 16) {
                            const uint4 newv = new_row(1);
                            *reinterpret_cast<uint4*>(vtile + vtile_offset(l_old - k0, lane)) = newv;
                            reinterpret_cast<uint4*>(Vl + (row0 + (l_old - k0)) * kRowBytes)[lane] = newv;
                        }
                    }
                    if (n_valid < kTileKeys)     // rows past the unit's end hold whatever the slab had: make them harmless for 0 * v
                        for (int x = lane; x < (kTileKeys - n_valid) * 16; x += 32) {
                            const int r = n_valid + (x >> 4), c = x & 15;
                            *reinterpret_cast<uint4*>(vtile + (c >> 3) * (kTileBytes / 2) + r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
                        }
                    __syncwarp();
                    {
                        uint32_t bfr[4];
                        ldmatrix_x4_trans(bfr, smem_addr(psm + lane * 16));   // keys 0-7 | 8-15 | 16-23 | 24-31 x 8 columns
                        const uint32_t vbase = smem_addr(vtile) + lm_row * 128;
#pragma unroll
                        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                            for (int cb = 0; cb < 8; ++cb) {
                                uint32_t a[4];
                                const int chunk = ((cb & 3) * 2 + lm_odd) ^ lm_x;
                                ldmatrix_x4_trans(a, vbase + (cb >> 2) * (kTileBytes / 2) + kb * 16 * 128 + chunk * 16);
                                mma_bf16_m16n8k16(accd[cb], a, bfr[2 * kb], bfr[2 * kb + 1]);          // Eq. 1
                            }
                    }
                    __syncwarp();
                    ++n_consumed;
                    cc = cur_next(cc);
                    if (cv.si < nseg) {
                        if (lane == 0) { fence_async_smem(); issue_v(cv); }
                        cv = cur_next(cv);
                    }
                }
                // fold the warp: Z over the lanes; the accumulators already hold whole-tile sums per (head, channel)
#pragma unroll
                for (int g = 0; g < G; ++g) { Zl[g] = warp_sum(Zl[g]); M[g] = (double)Mref[g]; }
            }
            // The warp's record {M, Z, acc[128]} per head goes straight to global memory (a warp without a tile in
            // this segment stores M = -inf, Z = 0, acc = 0), then the warp's arrival: no block-wide step here, the
            // other warps of the block stream on.
            const size_t pstride = partial_stride(128);
            // blk + u is unique: both grow along the tile list; a block per split numbers the records by (unit, split)
            const size_t rec_row = MODE == kBalUnits ? (size_t)u * bal_unit_splits(p.max_splits) + blockIdx.x : (size_t)(blk + u);
            unsigned char* rec_w = p.partials + (rec_row * NW + warp) * G * pstride;
            if (!CORM_IN_RANGE(MODE == kBalUnits || rec_row * NW + warp < bal_record_count(nblk, p.U), p.status)) continue;
            if (lane < G) {
                double* mz = reinterpret_cast<double*>(rec_w + (size_t)lane * pstride);
                double Mg = M[0], Zg = Zl[0];
#pragma unroll
                for (int g = 1; g < G; ++g) { Mg = lane == g ? M[g] : Mg; Zg = lane == g ? Zl[g] : Zg; }
                *reinterpret_cast<double2*>(mz) = make_double2(Mg, Zg);
            }
            if ((lane & 3) < G) {
                float* a = reinterpret_cast<float*>(rec_w + (size_t)(lane & 3) * pstride + 16);
#pragma unroll
                for (int cb = 0; cb < 8; ++cb) {
                    a[cb * 16 + (lane >> 2)] = accd[cb][0] + accd[cb][1];       // hi + lo columns of the head
                    a[cb * 16 + 8 + (lane >> 2)] = accd[cb][2] + accd[cb][3];
                }
            }
            __threadfence();
            __syncwarp();
            if (FINISH && lane == 0) atomicAdd(p.ticket + u, 1u);   // this warp's record and logits of the segment are stored
        }
        __syncthreads();
        if (failed) { report_status(p.status, CORM_ERR_TIMEOUT); s_failed = 1; }
        __syncthreads();
        if (s_failed) return;                   // a bounded wait expired: reported through the status word
        // ---- Algorithm 1 for the slots this block streamed; the ring is free now ----
        if (MODE == kBalUnits) {
            // every warp's record is stored and fenced (barriers above): the split arrives; the last one finishes the unit
            if (tid == 0) {
                const int u = segs[0].u, n_act = segs[0].pad;
                const unsigned prev = atomicAdd(p.ticket + u, 1u);
                misc->last = prev == (unsigned)(n_act - 1);
                if (misc->last) { p.ticket[u] = 0u; segs[0].tile0 = 0; segs[0].n_tiles = segs[0].n_unit; }
                __threadfence();
            }
            __syncthreads();
            if (!misc->last) return;
            bal_finish_block<G, PAGED, NT, true>(p, segs, 1, blk, T, nblk, smem, misc);
            return;
        } else if (FINISH) {
            bal_finish_block<G, PAGED, NT, false>(p, segs, nseg, blk, T, nblk, smem, misc);
            if (s_failed) return;
        } else {
            // the verdict launch may become resident now; it reads nothing of this launch before it has completed
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            for (int si = tid; si < nseg; si += NT) {          // units that start in this block: where their records are
                const BalSeg& sg = segs[si];
                const long long P0 = sg.gtile0;
                const int fb = bal_block_of(P0, T, nblk);
                if (fb == blk) p.unit_rec[sg.u] = make_int2((fb + sg.u) * NW, (bal_block_of(P0 + sg.n_unit - 1, T, nblk) - fb + 1) * NW);
            }
        }
        if (!s_more) break;
        __syncthreads();
        win_u = s_next_u; win_P = s_next_P;
        __syncthreads();
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// The V storage of one layer as a 2-D tensor [rows][128] of bf16 with boxes of 32 rows x 64 channels and the
// 128-byte swizzle; rows = every slab row or every pool row of the layer. The map only ever covers memory of the
// cache's own device.
inline corm_status_t make_v_tensor_map(CUtensorMap* out, void* v_layer, unsigned long long rows) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return CORM_ERR_UNSUPPORTED;
        }
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    const cuuint64_t dims[2] = {128, rows};
    const cuuint64_t strides[1] = {kRowBytes};
    const cuuint32_t box[2] = {64, kTileKeys};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, v_layer, dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CORM_OK : CORM_ERR_CUDA;
}


inline corm_status_t launch_decode_balanced(DecodeParams& p, const CUtensorMap& vmap, int G, int upper, int sm_count,
                                            size_t partial_capacity_records, bool verdict_launch, cudaStream_t st,
                                            int* n_launched) {
    *n_launched = 0;
    if (G != 1 && G != 2 && G != 4) return CORM_ERR_UNSUPPORTED;
    if (p.C > kBalMaxTokens) return CORM_ERR_UNSUPPORTED;
    const int sms = sm_count > 0 ? sm_count : 148;
    // one block per resident slot, fewer when the step cannot have that many tiles per warp
    const int upper_tiles = (upper + kTileKeys - 1) / kTileKeys;
    const long long tiles_upper = (long long)upper_tiles * p.U;
    long long grid = (long long)sms * kBalBlocksPerSm;
    if (tiles_upper / kBalWarps + 1 < grid) grid = tiles_upper / kBalWarps + 1;
    if (bal_record_count((int)grid, p.U) > partial_capacity_records) return CORM_ERR_UNSUPPORTED;
    constexpr int kTotal[5] = {0, bal_smem_layout(1).total, bal_smem_layout(2).total, 0, bal_smem_layout(4).total};
    const size_t smem = (size_t)kTotal[G];
    auto launch = [&](auto kern) -> corm_status_t {
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: cudaFuncSetAttribute: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kBalThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set-up overlaps the previous step's tail
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, p, vmap);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: decode launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    corm_status_t rc;
#define CORM_BAL(FIN)                                                                                                      \
    (p.page_table ? (G == 1 ? launch(decode_balanced_kernel<1, true, FIN>) : G == 2 ? launch(decode_balanced_kernel<2, true, FIN>)   \
                                                                                    : launch(decode_balanced_kernel<4, true, FIN>))  \
                  : (G == 1 ? launch(decode_balanced_kernel<1, false, FIN>) : G == 2 ? launch(decode_balanced_kernel<2, false, FIN>) \
                                                                                     : launch(decode_balanced_kernel<4, false, FIN>)))
    rc = verdict_launch ? CORM_BAL(kBalStream) : CORM_BAL(kBalFinish);
#undef CORM_BAL
    if (rc != CORM_OK) return rc;
    *n_launched = 1;
    if (!verdict_launch) return CORM_OK;
    // verdicts and compaction by the verdict launch, spread over 1024- or 2048-slot chunks of every unit
    const int n_rec_cap = kBalWarps * (int)(grid < upper_tiles ? grid : upper_tiles);   // records one unit can have
    const size_t vsmem = verdict_smem(p.C, n_rec_cap, G, p.page_table != nullptr);
    auto launch_v = [&](auto kern) -> corm_status_t {
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), vsmem);
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: cudaFuncSetAttribute: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        cudaLaunchConfig_t cfg{};
        const int batches = verdict_batches(upper, p.U, sms);
        cfg.gridDim = dim3((upper + batches * kVerdictBatch - 1) / (batches * kVerdictBatch), (unsigned)p.U);
        cfg.blockDim = dim3(kVerdictThreads);
        cfg.dynamicSmemBytes = vsmem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may become resident during the streaming tail
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, p, n_rec_cap, batches);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: verdict launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    rc = G == 1 ? launch_v(decode_verdict_kernel<bf16_t, 128, 1, true>) : G == 2 ? launch_v(decode_verdict_kernel<bf16_t, 128, 2, true>)
                                                                                 : launch_v(decode_verdict_kernel<bf16_t, 128, 4, true>);
    if (rc == CORM_OK) *n_launched = 2;
    return rc;
}

// The same streaming loop with a block per split of a unit and the unit finished by its last-arriving split
// (kBalUnits): one launch per step, no block waits for another, units leave stamps, so consecutive steps can be
// chained (want_chain / want_trigger as for launch_decode_fast). Meant for many units of a few thousand keys at most:
// the finishing block walks its whole unit alone.
inline corm_status_t launch_decode_balanced_units(DecodeParams& p, const CUtensorMap& vmap, int G, int upper, int typical,
                                                  int tune_split_len, int sm_count, size_t partial_capacity_records,
                                                  cudaStream_t st, int* n_launched, bool want_chain, bool want_trigger) {
    *n_launched = 0;
    if (G != 1 && G != 2 && G != 4) return CORM_ERR_UNSUPPORTED;
    if (p.C > kBalMaxTokens) return CORM_ERR_UNSUPPORTED;
    const int sms = sm_count > 0 ? sm_count : 148;
    const int grain = kBalWarps * kTileKeys;                       // a tile per warp at least
    int split_len = tune_split_len;
    if (!split_len) {
        // about one and a half blocks per resident slot over the whole step, from the mean unit where the host knows it
        // (128 units of 1660 keys, us per step: splits of 256 keys 47.4, 384 43.4, 512 42.5, 640 44.4, 896 47.8)
        const long long keys = (long long)(typical > 0 ? typical : upper) * p.U;
        split_len = (int)(2 * keys / (3ll * sms * kBalBlocksPerSm));
        // ... but at least 512 keys and at most 1024, or 2048 for long units: the grouped workload's first steps (units
        // of 3000-4500 keys, many evictions) take 108-112 us with splits of 512 or 1024 keys and 117-120 with 1152 or
        // 1280; 8200-key units take 132 us with splits of 2048, 142 with 1024, 162 with 512
        const int cap = (typical > 0 ? typical : upper) < 6144 ? 1024 : 2048;
        if (split_len > cap) split_len = cap;
        if (split_len < 512) split_len = 512;
    }
    const int max_unit_splits = bal_unit_splits(p.max_splits);     // records a unit has room for, in splits
    if (split_len < (upper + max_unit_splits - 1) / max_unit_splits) split_len = (upper + max_unit_splits - 1) / max_unit_splits;
    split_len = (split_len + grain - 1) / grain * grain;
    if (split_len < grain) split_len = grain;
    const int n_splits = (upper + split_len - 1) / split_len;
    if (n_splits > max_unit_splits || (size_t)p.U * max_unit_splits * kBalWarps > partial_capacity_records) return CORM_ERR_UNSUPPORTED;
    if ((size_t)G * n_splits * kBalWarps > 7000 || n_splits > 65535) return CORM_ERR_UNSUPPORTED;   // scale factors of a unit's records: shared memory
    p.split_len = split_len;
    p.chain_wait = want_chain && p.unit_stamp ? 1 : 0;
    p.early_trigger = want_trigger ? 1 : 0;
    constexpr int kTotal[5] = {0, bal_smem_layout(1).total, bal_smem_layout(2).total, 0, bal_smem_layout(4).total};
    const size_t smem = (size_t)kTotal[G];
    auto launch = [&](auto kern) -> corm_status_t {
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: cudaFuncSetAttribute: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)n_splits, (unsigned)p.U);
        cfg.blockDim = dim3(kBalThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, p, vmap);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: decode launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    const corm_status_t rc =
        p.page_table ? (G == 1 ? launch(decode_balanced_kernel<1, true, kBalUnits>) : G == 2 ? launch(decode_balanced_kernel<2, true, kBalUnits>)
                                                                                             : launch(decode_balanced_kernel<4, true, kBalUnits>))
                     : (G == 1 ? launch(decode_balanced_kernel<1, false, kBalUnits>) : G == 2 ? launch(decode_balanced_kernel<2, false, kBalUnits>)
                                                                                              : launch(decode_balanced_kernel<4, false, kBalUnits>));
    if (rc == CORM_OK) *n_launched = 1;
    return rc;
}

}  // namespace corm
