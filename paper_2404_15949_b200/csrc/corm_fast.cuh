// Decode kernel for bf16 caches with head_dim 128 (group size 1, 2 or 4): the bandwidth path.
//
// One thread block per (unit, split of its live range); every warp streams 32-key tiles of K and V through its own
// ring of shared-memory stages filled by bulk asynchronous copies (the TMA engine; a tile is one contiguous run of
// 256-byte rows in the slab) that complete on mbarriers, so warps never synchronise with each other in the main
// loop. Logits are formed in fp64: bf16 inputs widen exactly, a lane owns 8 channels of a key and 16 lanes share a
// key; the 16 partial sums of 16 keys are folded with a transposing butterfly (15 exchanges for 16 keys, no
// selects: each lane loads its keys in an order permuted by its lane bits so that every exchange step sends and
// keeps fixed registers). After the fold each lane owns one key of the tile for softmax, verdict logit and
// probability. P.V accumulates in fp32. A unit that fits one split keeps its logits in shared memory and its
// registers and positions in thread registers and finishes entirely inside the block; longer units publish split
// records and logits to global scratch, and either the last-arriving block runs the shared finalize phase (launches
// with many blocks, or short units) or the verdict launch of corm_verdict.cuh takes over (few, long units).
#pragma once

#include <cmath>

#include "corm_common.cuh"
#include "corm_verdict.cuh"

namespace corm {

#ifndef CORM_FAST_WARPS
#define CORM_FAST_WARPS 4
#endif
#ifndef CORM_FAST_BLOCKS_G1
#define CORM_FAST_BLOCKS_G1 3
#endif
constexpr int kFastWarps = CORM_FAST_WARPS;
constexpr int kFastThreads = kFastWarps * 32;
constexpr int kTileKeys = 32;
constexpr int kRowBytes = 256;                    // 128 bf16
constexpr int kTileBytes = kTileKeys * kRowBytes; // 8 KiB
constexpr int kVStages = 1;
// K stages per warp, resident blocks per SM and the shared-memory budget that allows them, by group size:
// one query head per KV head leaves registers and shared memory for three blocks per SM; larger groups keep two.
__host__ __device__ constexpr int fast_k_stages(int G) { return G == 1 ? 1 : 2; }
__host__ __device__ constexpr int fast_stages(int G) { return fast_k_stages(G) + kVStages; }
__host__ __device__ constexpr int fast_warp_bytes(int G) { return fast_stages(G) * kTileBytes; }
__host__ __device__ constexpr int fast_blocks_per_sm(int G) { return G == 1 ? CORM_FAST_BLOCKS_G1 : 2; }
// 228 KB per SM, minus 1 KB the system reserves per block and ~1.7 KB of static shared memory
__host__ __device__ constexpr int fast_smem_budget(int G) { return (228 * 1024) / fast_blocks_per_sm(G) - 2816; }
constexpr long long kWaitLimitCycles = 4000000000ll;   // bounded mbarrier waits (about 2 s)
// longest unit that may finish inside one block (bounded by the registers that carry its verdict words)
__host__ __device__ constexpr int fast_max_single_cap(int G) { return (G == 1 ? 8 : 2) * kFastThreads; }

// ---- shared-memory carve-up (bytes), all offsets multiples of 128 ----
struct FastSmem {
    int tiles, psm, stash, bars, newrow, total;
};
__host__ __device__ inline FastSmem fast_smem_layout(int G, int single_cap) {
    FastSmem s;
    int off = 0;
    auto take = [&](int bytes) { int at = off; off = (off + bytes + 127) / 128 * 128; return at; };
    s.tiles = take(kFastWarps * fast_warp_bytes(G));            // later reused: merge area, finalize lists
    s.psm = take(kFastWarps * kTileKeys * G * 4);
    s.stash = take(single_cap * G * 8);
    s.bars = take(kFastWarps * fast_stages(G) * 8);
    s.newrow = take(2 * kRowBytes);                             // the appended K and V rows, fetched ahead
    s.total = off;
    return s;
}

// ---- PTX wrappers ----
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Waits for the phase with the given parity; gives up after kWaitLimitCycles and reports false.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long start = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - start > kWaitLimitCycles) return false;
    return true;
}
// Waits until the unit's stamp says that at least `steps_done` decode steps of it are complete and returns the stamp.
// Gives up (all ones) after kWaitLimitCycles, reporting a timeout, or as soon as another block has reported a
// failure that leaves the cache unusable anyway.
__device__ __forceinline__ unsigned long long wait_unit_stamp(const unsigned long long* stamp, uint32_t steps_done, int32_t* status) {
    const long long start = clock64();
    for (;;) {
        unsigned long long v;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(stamp) : "memory");
        if ((uint32_t)(v >> 32) >= steps_done) return v;
        const int32_t s = *reinterpret_cast<volatile int32_t*>(status);
        if (s == CORM_ERR_TIMEOUT || s == CORM_ERR_INTERNAL) return ~0ull;
        if (clock64() - start > kWaitLimitCycles) { report_status(status, CORM_ERR_TIMEOUT); return ~0ull; }
        __nanosleep(64);
    }
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src_gmem, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src_gmem), "r"(bytes), "r"(bar) : "memory");
}
// 16-byte asynchronous copy global -> shared by the calling thread, and the wait for all of the thread's own
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src_gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src_gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// exp(x) for x <= ~0 (small positive arguments are fine), 0 below the normal range. Argument reduction by ln 2 in
// two pieces, degree-11 Taylor polynomial on |r| <= ln2/2 (truncation ~6e-15 relative), scaling through the exponent.
// Branch-free, so that several independent calls interleave.
__device__ __forceinline__ double exp_nonpos(double x0) {
    const double x = fmax(x0, -708.0);
    const double t = fma(x, 1.4426950408889634074, 6755399441055744.0);   // round(x / ln 2) in the low word
    const int n = __double2loint(t);
    const double nf = t - 6755399441055744.0;
    double r = fma(nf, -6.93147180369123816490e-01, x);
    r = fma(nf, -1.90821492927058770002e-10, r);
    double p = 2.505210838544172e-08;            // 1/11!
    p = fma(p, r, 2.755731922398589e-07);        // 1/10!
    p = fma(p, r, 2.755731922398589e-06);        // 1/9!
    p = fma(p, r, 2.48015873015873e-05);         // 1/8!
    p = fma(p, r, 1.984126984126984e-04);        // 1/7!
    p = fma(p, r, 1.388888888888889e-03);        // 1/6!
    p = fma(p, r, 8.333333333333333e-03);        // 1/5!
    p = fma(p, r, 4.166666666666666e-02);        // 1/4!
    p = fma(p, r, 1.666666666666667e-01);        // 1/3!
    p = fma(p, r, 0.5);
    p = fma(p, r, 1.0);
    p = fma(p, r, 1.0);
    const double y = p * __hiloint2double((1023 + n) << 20, 0);
    return x0 > -708.0 ? y : 0.0;
}

__device__ __forceinline__ void unpack8_to_double(const uint4& raw, double (&kd)[8]) {
    kd[0] = (double)__uint_as_float(raw.x << 16); kd[1] = (double)__uint_as_float(raw.x & 0xffff0000u);
    kd[2] = (double)__uint_as_float(raw.y << 16); kd[3] = (double)__uint_as_float(raw.y & 0xffff0000u);
    kd[4] = (double)__uint_as_float(raw.z << 16); kd[5] = (double)__uint_as_float(raw.z & 0xffff0000u);
    kd[6] = (double)__uint_as_float(raw.w << 16); kd[7] = (double)__uint_as_float(raw.w & 0xffff0000u);
}
// Packed fp32 pairs (sm_100 has a two-wide fp32 FMA): helpers for the P.V accumulation.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma_f32x2(unsigned long long& acc, unsigned long long a, unsigned long long b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ void mul_f32x2(unsigned long long& acc, unsigned long long a) {
    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(acc) : "l"(a));
}
// one 32-bit word holding two bf16 -> the two values as a packed fp32 pair (element 0 in the low half)
__device__ __forceinline__ unsigned long long bf16x2_to_f32x2(uint32_t w) {
    return pack_f32x2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ void unpack8_to_float(const uint4& raw, float (&v)[8]) {
    v[0] = __uint_as_float(raw.x << 16); v[1] = __uint_as_float(raw.x & 0xffff0000u);
    v[2] = __uint_as_float(raw.y << 16); v[3] = __uint_as_float(raw.y & 0xffff0000u);
    v[4] = __uint_as_float(raw.z << 16); v[5] = __uint_as_float(raw.z & 0xffff0000u);
    v[6] = __uint_as_float(raw.w << 16); v[7] = __uint_as_float(raw.w & 0xffff0000u);
}

// Unscaled q.k sums of one 32-key tile. Lane (h = lane>>4, i = lane&15) reads channel chunk i of the keys of half h;
// on return the lane holds, per query head, the full sum of tile key  16h + 8(i&1) + (i>>1).
// Pass it in {0,1} and register slot s in 0..7 load key 16h + 8(it ^ (i&1)) + (s ^ (i>>1)): with that order every
// butterfly step keeps the low slots and sends the high ones, whatever the lane.
template <int G>
__device__ __forceinline__ void qk_tile(const unsigned char* ktile, const double (&qd)[G][8], int lane,
                                        double (&sown)[G]) {
    const int h = lane >> 4, i = lane & 15, m = i >> 1, b0 = i & 1;
    double r[2][G];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        double a[G][8];
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const int key = 16 * h + 8 * (it ^ b0) + (s ^ m);
            const uint4 raw = *reinterpret_cast<const uint4*>(ktile + key * kRowBytes + i * 16);
            double kd[8];
            unpack8_to_double(raw, kd);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                double acc = qd[g][0] * kd[0];
#pragma unroll
                for (int e = 1; e < 8; ++e) acc = fma(qd[g][e], kd[e], acc);
                a[g][s] = acc;
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int s = 0; s < 4; ++s) a[g][s] += __shfl_xor_sync(0xffffffffu, a[g][s + 4], 8);
#pragma unroll
            for (int s = 0; s < 2; ++s) a[g][s] += __shfl_xor_sync(0xffffffffu, a[g][s + 2], 4);
            a[g][0] += __shfl_xor_sync(0xffffffffu, a[g][1], 2);
            r[it][g] = a[g][0];
        }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) sown[g] = r[0][g] + __shfl_xor_sync(0xffffffffu, r[1][g], 1);
}

// Single-split finalize: logits, registers and positions of the whole unit are in shared memory.
// lists: scratch for the keep mask, its prefix sums and the hole / mover lists (ints).
// wv / pv: registers and positions of slots tid, tid + NT, ... (loaded by the caller at block start).
// tile_pages: paged caches, page + 1 of tile T of the unit at [T % kFastWarps][T / kFastWarps] (shared memory).
template <int G, int NT, int KPRE, bool PAGED>
__device__ void finalize_single(const DecodeParams& p, int u, int b, int l, int t, const double* thr,
                                const double* stash_sm, int stash_ld, const uint32_t (&wv)[KPRE],
                                const int32_t (&pv)[KPRE], unsigned char* lists, int* holes, int* movers,
                                const int32_t (*tile_pages)[32]) {
    __shared__ int s_scan1[NT];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cap_words = (l + 31) / 32 + 2;
    uint32_t* keepmask = reinterpret_cast<uint32_t*>(lists);
    int* prefix = reinterpret_cast<int*>(keepmask + cap_words);
    uint32_t* wordu = p.word + (size_t)u * p.C;
    int32_t* posu = p.pos + (size_t)u * p.C;
    const int n_obs = min(p.w, __ldg(p.base_obs + b) + p.step + 1);
    const bool evict_on = n_obs >= p.w;
    int n_imp = 0;                                                // keys this thread judged important
#pragma unroll
    for (int k = 0; k < KPRE; ++k) {
        const int base = k * NT, j = base + tid;
        if (base >= l) break;                                     // uniform
        bool keep = false;
        if (j < l) {
            bool imp = false;
#pragma unroll
            for (int g = 0; g < G; ++g) imp |= (stash_sm[g * stash_ld + j] >= thr[g]);
            const uint32_t wd = update_register(wv[k], imp, p.w, t);
            n_imp += imp ? 1 : 0;
            wordu[j] = wd;
            keep = !evict_on || register_needed(wd, p.w, t) || pv[k] > t - p.r;
        }
        const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
        if (lane == 0 && base + warp * 32 < l) keepmask[(base >> 5) + warp] = ballot;
    }
    warp_count(p.counters + CNT_IMPORTANT, n_imp);                // Section 3.1's sparsity
    __syncthreads();
    int new_len = l, n_moved = 0;
    if (evict_on) {
        const int nwords = (l + 31) / 32;
        block_popc_scan<NT>(keepmask, prefix, nwords, s_scan1);
        new_len = prefix[nwords];
        if (new_len < l) {
            const int kept_below = kept_before(keepmask, prefix, new_len);
            n_moved = new_len - kept_below;
            for (int j = tid; j < l; j += NT) {
                const int kb = kept_before(keepmask, prefix, j);
                const bool kept = (keepmask[j >> 5] >> (j & 31)) & 1u;
                if (j < new_len && !kept) holes[j - kb] = j;
                if (j >= new_len && kept) movers[kb - kept_below] = j;
            }
            __syncthreads();
            const size_t slab_row0 = (size_t)u * p.C;
            block_move_rows<bf16_t, 128, NT>(
                reinterpret_cast<bf16_t*>(p.K), reinterpret_cast<bf16_t*>(p.V),
                [&](int slot) -> size_t {      // the unit is one split: its pages are the ones the warps fetched for their tiles
                    const int tile = slot >> 5;
                    return PAGED ? page_row(tile_pages[tile % kFastWarps][tile / kFastWarps], slot, p.pool_pages, p.status)
                                 : slab_row0 + (size_t)slot;
                },
                wordu, posu, movers, holes, n_moved, 0, 1, l, p.status);
        }
    }
    if (PAGED) settle_pages<NT>(p.page_table, p.page_bits, p.page_room, p.pool_pages, p.pt_stride, p.U, u, l - 1, new_len);
    if (p.unit_stamp) __syncthreads();            // the row moves and register writes of every warp come before the stamp
    if (tid == 0) {
        p.live_out[u] = new_len;
        publish_unit_stamp(p, u, new_len);
        publish_live(p.maxlive, p.step + 1, new_len);
        atomicAdd(p.counters + CNT_APPENDED, 1ull);
        atomicAdd(p.counters + CNT_ATTENDED, (unsigned long long)l);
        if (new_len < l) atomicAdd(p.counters + CNT_EVICTED, (unsigned long long)(l - new_len));
        if (n_moved) atomicAdd(p.counters + CNT_MOVED, (unsigned long long)n_moved);
    }
}

// PAGED selects the cache layout at compile time (the launcher picks the instance from p.page_table), so that the
// slab instance carries none of the paging code.
template <int G, bool PAGED>
__global__ void __launch_bounds__(kFastThreads, fast_blocks_per_sm(G)) decode_fast_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_failed;
    __shared__ int s_last;
    __shared__ double s_thr1[G];
    constexpr int NT = kFastThreads, NW = kFastWarps;
    constexpr int kKStages = fast_k_stages(G), kStagesPerWarp = fast_stages(G);
    const int u = blockIdx.y, split = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = u / p.Hkv;
    // Paged caches: the pages of this warp's tiles (tile it of warp w is tile w + it * NW of the split, lane it fetches
    // its entry) and the unit's room flag are requested together with the live length, none behind another; a unit
    // without a page for the appended row (pool exhausted) is treated like a full slab.
    __shared__ int32_t s_pt[kFastWarps][32];
    const int32_t* pt_u = PAGED ? p.page_table + (size_t)u * p.pt_stride : nullptr;
    // Launched with programmatic stream serialization: the block may start while the previous launch on the stream
    // drains. Ordinarily it reads nothing before that launch has completed. A chained launch (the previous launch was
    // the previous decode step of these same units and finished every unit inside itself) waits for less: only for
    // its own unit's previous step, whose finishing block left a stamp (steps done, live length) behind all its
    // writes. Units are independent, so nothing else of the previous launch concerns this block, and the blocks of
    // consecutive steps fill one another's last waves.
    int l_old;
    if (p.chain_wait) {
        __shared__ unsigned long long s_stamp;
        if (tid == 0) s_stamp = wait_unit_stamp(p.unit_stamp + u, (uint32_t)p.step, p.status);
        __syncthreads();
        const unsigned long long sw = s_stamp;
        // not this step's stamp: the wait gave up (reported), or the unit is already past this step, which only a
        // block that has no split to work on can find
        if ((uint32_t)(sw >> 32) != (uint32_t)p.step) return;
        l_old = (int)(uint32_t)sw;
        asm volatile("fence.proxy.async.global;" ::: "memory");     // the bulk copies below read rows that ordinary stores wrote
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        l_old = __ldcg(p.live_in + u);
    }
    int32_t my_page = 0, room = 1;
    if (PAGED) {
        const int idx = split * (p.split_len >> 5) + warp + lane * kFastWarps;
        if (idx < p.pt_stride) my_page = __ldcg(pt_u + idx);
        room = __ldcg(p.page_room + u);
    }
    const int l = l_old + 1;
    if (l > p.C || !room) {
        if (split == 0 && tid == 0) {
            report_status(p.status, CORM_ERR_CAPACITY);
            p.live_out[u] = l_old;
            publish_unit_stamp(p, u, l_old);
            publish_live(p.maxlive, p.step + 1, l_old);
        }
        return;
    }
    const int n_act = (l + p.split_len - 1) / p.split_len;
    if (split >= n_act) return;
    if (n_act > (int)gridDim.x && split == 0 && tid == 0) report_status(p.status, CORM_ERR_INTERNAL);   // the host's bound on the unit was wrong
    // From here on the next launch may become resident (a chained one: its blocks wait for their units' stamps). Not
    // earlier: an unchained block takes its unit's length from the double-buffered array, whose other half the next
    // step rewrites, so every block has its length (the branch above depends on it) before a block of the next step runs.
    if (p.early_trigger) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const bool single = (n_act == 1 && l <= p.single_cap);
    const int t = __ldg(p.base_tokens + b) + p.step + 1;
    const int begin = split * p.split_len, end = min(l, begin + p.split_len);
    const int n_tiles = (end - begin + kTileKeys - 1) / kTileKeys;
    const FastSmem lay = fast_smem_layout(G, p.single_cap);
    unsigned char* my_tiles = smem + lay.tiles + warp * fast_warp_bytes(G);
    const uint32_t my_bars = smem_addr(smem + lay.bars) + warp * kStagesPerWarp * 8;
    float* psm = reinterpret_cast<float*>(smem + lay.psm) + warp * kTileKeys * G;
    double* stash_sm = reinterpret_cast<double*>(smem + lay.stash);
    static_assert(kTileKeys == kPageKeys, "a page is one tile of the streaming kernel");
    unsigned char* Kl = reinterpret_cast<unsigned char*>(p.K);       // the layer's K / V storage: slabs or page pool
    unsigned char* Vl = reinterpret_cast<unsigned char*>(p.V);
    const size_t slab_row0 = (size_t)u * p.C;
    uint32_t* wordu = p.word + (size_t)u * p.C;
    int32_t* posu = p.pos + (size_t)u * p.C;

    if (tid == 0) s_failed = 0;

    // this warp's tiles: warp, warp + NW, ... (tile index inside the split)
    const int my_n = (n_tiles > warp) ? (n_tiles - warp + NW - 1) / NW : 0;
    if (PAGED) { s_pt[warp][lane] = my_page; __syncwarp(); }
    // first row of the warp's tile `it` in the layer's K / V storage
    auto tile_row0 = [&](int it) -> size_t {
        if (!PAGED) return slab_row0 + (size_t)(begin + (warp + it * NW) * kTileKeys);
        const int pg = it < 32 ? s_pt[warp][it] : __ldcg(pt_u + (begin >> 5) + warp + it * NW);
        return page_row(pg, 0, p.pool_pages, p.status);
    };
    auto tile_keys = [&](int it) { return min(kTileKeys, end - (begin + (warp + it * NW) * kTileKeys)); };
    auto issue_k = [&](int it) {
        const int k0 = begin + (warp + it * NW) * kTileKeys, slot = it % kKStages;
        const uint32_t bytes = (uint32_t)tile_keys(it) * kRowBytes;
        mbar_expect_tx(my_bars + slot * 8, bytes);
        bulk_load(smem_addr(my_tiles + slot * kTileBytes), Kl + tile_row0(it) * kRowBytes, bytes, my_bars + slot * 8);
    };
    auto issue_v = [&](int it) {
        const int k0 = begin + (warp + it * NW) * kTileKeys, slot = it % kVStages;
        const uint32_t bytes = (uint32_t)tile_keys(it) * kRowBytes;
        mbar_expect_tx(my_bars + (kKStages + slot) * 8, bytes);
        bulk_load(smem_addr(my_tiles + (kKStages + slot) * kTileBytes), Vl + tile_row0(it) * kRowBytes, bytes,
                  my_bars + (kKStages + slot) * 8);
    };
    // a warp's barriers and stages are its own: its first copies leave before the block meets at its first barrier
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStagesPerWarp; ++s) mbar_init(my_bars + s * 8, 1);
        fence_mbar_init();
        fence_async_smem();
        for (int it = 0; it < min(my_n, kKStages); ++it) issue_k(it);
        for (int it = 0; it < min(my_n, kVStages); ++it) issue_v(it);
    }
    __syncthreads();                                              // s_failed is initialised for everybody

    // queries widened to fp64 once per block; a single-split unit also fetches the registers and positions of the
    // slots this thread will judge in the finalize phase (slots tid, tid + NT, ...) and keeps them in registers
    constexpr int kPre = fast_max_single_cap(G) / NT;
    uint32_t wv[kPre];
    int32_t pv[kPre];
#pragma unroll
    for (int k = 0; k < kPre; ++k) { wv[k] = 0u; pv[k] = 0; }
    if (single) {
#pragma unroll
        for (int k = 0; k < kPre; ++k) {
            const int j = tid + k * NT;
            if (j < l_old) { wv[k] = __ldcg(wordu + j); pv[k] = __ldcg(posu + j); }
            else if (j == l_old) { wv[k] = 0u; pv[k] = t; }          // the token appended by this step
        }
    }
    const int h = lane >> 4, ci = lane & 15;
    const int key_own = 16 * h + 8 * (ci & 1) + (ci >> 1);     // tile key this lane owns after the fold
    // the lane's 8 channels of every query head, widened to fp64: one 16-byte load per head, no staging
    double qd[G][8];
    {
        const uint4* qg = reinterpret_cast<const uint4*>(p.q) + (size_t)u * G * 16 + ci;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint4 raw = __ldg(qg + g * 16);
            unpack8_to_double(raw, qd[g]);
        }
    }
    // The appended token's rows are fetched ahead by the warp that will meet slot l_old (the unit's last tile), so that
    // their latency (a PCIe round trip when the caller's buffers are pinned host memory) is off that tile's path;
    // requested once the warp's first tile is done, i.e. after the queries, which every warp needs first and which
    // share that bus.
    unsigned char* newrow = smem + lay.newrow;
    const bool new_is_mine = l_old >= begin && l_old < end && ((l_old - begin) / kTileKeys) % NW == warp;
    auto fetch_new_rows = [&]() {
        const unsigned char* src = lane < 16 ? reinterpret_cast<const unsigned char*>(p.k_new) + ((size_t)u * 16 + lane) * 16
                                             : reinterpret_cast<const unsigned char*>(p.v_new) + ((size_t)u * 16 + lane - 16) * 16;
        cp_async16(smem_addr(newrow + lane * 16), src);
    };
    if (new_is_mine && my_n <= 1) fetch_new_rows();              // its only tile is the one with the new row
    double M[G], Zl[G];
    unsigned long long acc2[G][4];                                // P.V accumulators: channel pairs (2e, 2e+1) of this lane's 8
#pragma unroll
    for (int g = 0; g < G; ++g) {
        M[g] = -INFINITY; Zl[g] = 0.0;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc2[g][e] = 0ull;
    }
    const double inv_root_d = 0.088388347648318440550;          // 1/sqrt(128)
    bool failed = false;

    for (int it = 0; it < my_n; ++it) {
        const int k0 = begin + (warp + it * NW) * kTileKeys;
        const int n_valid = min(kTileKeys, end - k0);
        const bool has_new = (l_old >= k0 && l_old < k0 + kTileKeys);   // this tile holds the appended token
        const int kslot = it % kKStages, vslot = it % kVStages;
        unsigned char* ktile = my_tiles + kslot * kTileBytes;
        unsigned char* vtile = my_tiles + (kKStages + vslot) * kTileBytes;
        if (!failed && !mbar_wait(my_bars + kslot * 8, (it / kKStages) & 1)) failed = true;   // after one expired wait the rest are skipped
        if (has_new) {   // append: the new row goes to the slab and replaces whatever the copy fetched for that slot
            cp_async_wait_all();
            __syncwarp();
            if (lane < 16) {
                const uint4 x = *reinterpret_cast<const uint4*>(newrow + lane * 16);
                *reinterpret_cast<uint4*>(ktile + (l_old - k0) * kRowBytes + lane * 16) = x;
                reinterpret_cast<uint4*>(Kl + (tile_row0(it) + (size_t)(l_old - k0)) * kRowBytes)[lane] = x;
            }
            if (lane == 0) { wordu[l_old] = 0u; posu[l_old] = t; }
            __syncwarp();
        }
        double sown[G];
        qk_tile<G>(ktile, qd, lane, sown);
        __syncwarp();
        if (lane == 0 && it + kKStages < my_n) { fence_async_smem(); issue_k(it + kKStages); }
        if (new_is_mine && it == 0 && my_n > 1) fetch_new_rows();  // the queries are in: the bus is free for these

        const bool valid = key_own < n_valid;
        const int j_own = k0 + key_own;
        // softmax bookkeeping for all heads at once: the per-head chains (shuffles, exponentials) are independent
        double sv[G], Mn[G], sc[G], ex[G];
        float mt[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            sv[g] = valid ? sown[g] * inv_root_d : -INFINITY;             // Eq. 2's exponent
            mt[g] = (float)sv[g];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int g = 0; g < G; ++g) mt[g] = fmaxf(mt[g], __shfl_xor_sync(0xffffffffu, mt[g], o));
#pragma unroll
        for (int g = 0; g < G; ++g) Mn[g] = fmax(M[g], (double)mt[g]);   // new reference: warp-uniform, >= every logit so far (up to fp32 rounding)
        bool moved = false;
#pragma unroll
        for (int g = 0; g < G; ++g) moved |= (Mn[g] != M[g]);
        if (moved) {                                                       // warp-uniform; rare after the first tiles
#pragma unroll
            for (int g = 0; g < G; ++g) sc[g] = exp_nonpos(M[g] - Mn[g]);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                Zl[g] *= sc[g];
                const float scf = (float)sc[g];
                const unsigned long long sc2 = pack_f32x2(scf, scf);
#pragma unroll
                for (int e = 0; e < 4; ++e) mul_f32x2(acc2[g][e], sc2);
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) ex[g] = valid ? exp_nonpos(sv[g] - Mn[g]) : 0.0;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            Zl[g] += ex[g];
            M[g] = Mn[g];
            psm[key_own * G + g] = (float)ex[g];
            if (valid) {
                if (single) { if (CORM_IN_RANGE(j_own < p.single_cap, p.status)) stash_sm[g * p.single_cap + j_own] = sv[g]; }
                else if (CORM_IN_RANGE(j_own < p.C, p.status)) p.stash[((size_t)u * G + g) * p.C + j_own] = sv[g];
            }
        }
        __syncwarp();

        if (!failed && !mbar_wait(my_bars + (kKStages + vslot) * 8, (it / kVStages) & 1)) failed = true;
        if (has_new) {
            if (lane < 16) {
                const uint4 x = *reinterpret_cast<const uint4*>(newrow + kRowBytes + lane * 16);
                *reinterpret_cast<uint4*>(vtile + (l_old - k0) * kRowBytes + lane * 16) = x;
                reinterpret_cast<uint4*>(Vl + (tile_row0(it) + (size_t)(l_old - k0)) * kRowBytes)[lane] = x;
            }
        }
        if (n_valid < kTileKeys)     // rows the copy did not fetch: make them harmless for 0 * v
            for (int x = lane; x < (kTileKeys - n_valid) * 16; x += 32)
                *reinterpret_cast<uint4*>(vtile + n_valid * kRowBytes + x * 16) = make_uint4(0, 0, 0, 0);
        __syncwarp();
#pragma unroll 4
        for (int n = 0; n < 16; ++n) {
            const int key = 16 * h + n;
            const uint4 raw = *reinterpret_cast<const uint4*>(vtile + key * kRowBytes + ci * 16);
            const unsigned long long v2[4] = {bf16x2_to_f32x2(raw.x), bf16x2_to_f32x2(raw.y), bf16x2_to_f32x2(raw.z),
                                              bf16x2_to_f32x2(raw.w)};
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float pj = psm[key * G + g];
                const unsigned long long p2 = pack_f32x2(pj, pj);
#pragma unroll
                for (int e = 0; e < 4; ++e) fma_f32x2(acc2[g][e], p2, v2[e]);           // Eq. 1
            }
        }
        __syncwarp();
        if (lane == 0 && it + kVStages < my_n) { fence_async_smem(); issue_v(it + kVStages); }
    }
    if (failed) { report_status(p.status, CORM_ERR_TIMEOUT); s_failed = 1; }
    // The verdict launch that may follow is allowed to become resident once every block of this grid is past its
    // tiles (it waits for this grid to complete before it reads anything written here). Allowing it from the top of
    // the kernel costs 1.4 us per step on 128 units of 1600 keys: its waiting blocks take room next to streaming ones.
    if (!p.early_trigger) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // fold the warp: lane-private sums of Z, the two halves of acc
    float acc[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        Zl[g] = warp_sum(Zl[g]);
#pragma unroll
        for (int e = 0; e < 4; ++e) unpack_f32x2(acc2[g][e], acc[g][2 * e], acc[g][2 * e + 1]);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[g][e] += __shfl_xor_sync(0xffffffffu, acc[g][e], 16);
    }
    __syncthreads();                       // every warp is done with its tiles: the tile area becomes scratch
    if (s_failed) {                        // a bounded wait expired: reported through the status word; the unit keeps its
        if (split == 0 && tid == 0) { p.live_out[u] = l_old; publish_live(p.maxlive, p.step + 1, l_old); }   // old length
        return;                            // (its arrival counter is not taken: the cache must be reset after this status)
    }
    unsigned char* merge = smem + lay.tiles;                      // [NW][G] records {double M, double Z, float acc[128]}
    constexpr int kRec = 16 + 4 * 128;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        unsigned char* rec = merge + (warp * G + g) * kRec;
        if (lane == 0) { reinterpret_cast<double*>(rec)[0] = M[g]; reinterpret_cast<double*>(rec)[1] = Zl[g]; }
        if (lane < 16) {
            float4* a = reinterpret_cast<float4*>(rec + 16 + ci * 32);
            a[0] = make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
            a[1] = make_float4(acc[g][4], acc[g][5], acc[g][6], acc[g][7]);
        }
    }
    __syncthreads();
    // block-level merge: thread tid owns channels tid, tid + NT, ...
    const size_t pstride = partial_stride(128);
    for (int g = 0; g < G; ++g) {
        double Mb = -INFINITY;
        for (int w = 0; w < NW; ++w) Mb = fmax(Mb, reinterpret_cast<const double*>(merge + (w * G + g) * kRec)[0]);
        double Zb = 0.0;
        float scw[NW];
        for (int w = 0; w < NW; ++w) {
            const unsigned char* rec = merge + (w * G + g) * kRec;
            const double sc = exp_nonpos(reinterpret_cast<const double*>(rec)[0] - Mb);
            Zb += reinterpret_cast<const double*>(rec)[1] * sc;
            scw[w] = (float)sc;
        }
        for (int c = tid; c < 128; c += NT) {
            float a = 0.f;
            for (int w = 0; w < NW; ++w) a += reinterpret_cast<const float*>(merge + (w * G + g) * kRec + 16)[c] * scw[w];
            if (single) {
                bf16_t* outp = reinterpret_cast<bf16_t*>(p.out) + ((size_t)u * G + g) * 128;
                Elem<bf16_t>::store(outp + c, (float)((double)a / Zb));
            } else {
                unsigned char* rec = p.partials + (((size_t)u * p.max_splits + split) * G + g) * pstride;
                reinterpret_cast<float*>(rec + 16)[c] = a;
            }
        }
        if (tid == 0) {
            if (single) s_thr1[g] = Mb + log(Zb) + p.log_alpha - log((double)t);
            else {
                unsigned char* rec = p.partials + (((size_t)u * p.max_splits + split) * G + g) * pstride;
                reinterpret_cast<double*>(rec)[0] = Mb; reinterpret_cast<double*>(rec)[1] = Zb;
            }
        }
    }
    if (single) {
        __syncthreads();
        unsigned char* lists = merge + NW * G * kRec;
        int* holes = reinterpret_cast<int*>(lists + 2 * ((l + 31) / 32 + 2) * 4);
        finalize_single<G, NT, kPre, PAGED>(p, u, b, l, t, s_thr1, stash_sm, p.single_cap, wv, pv, lists, holes, holes + l, s_pt);
        return;
    }
    // A unit of several splits: its partial records and logits are complete once every split is done. With many
    // units in flight the split that arrives last finishes the unit right here (its serial walk over the unit hides
    // behind the other units' streaming); with few units that walk would be the tail of the launch, and the verdict
    // launch that follows spreads it over many blocks instead.
    if (!p.inline_finalize) return;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned prev = atomicAdd(p.ticket + u, 1u);
        s_last = (prev == (unsigned)(n_act - 1));
        if (s_last) p.ticket[u] = 0u;
        __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    finalize_unit<bf16_t, 128, G, NT>(p, u, b, l, n_act, t, smem);
}

// Host side: split length and launch. Returns CORM_ERR_UNSUPPORTED for group sizes the kernel does not cover.
// upper bounds every unit's live length; typical is the mean live length as far as the host knows it (0 = unknown).
// want_chain / want_trigger: what the caller would like for p.chain_wait / p.early_trigger; granted only when this
// launch finishes every unit inside itself (*self_finishing), which is also what lets the next launch be chained.
inline corm_status_t launch_decode_fast(DecodeParams& p, int G, int upper, int typical, int tune_split_len, int sm_count,
                                        cudaStream_t st, int* n_launched, int finish_mode, bool want_chain = false,
                                        bool want_trigger = false, bool* self_finishing = nullptr) {
    *n_launched = 0;
    if (self_finishing) *self_finishing = false;
    if (G != 1 && G != 2 && G != 4) return CORM_ERR_UNSUPPORTED;
    // longest unit that can finish inside one block: bounded by the verdict registers a thread carries and by the
    // shared memory that holds the unit's logits
    int cap = fast_max_single_cap(G);
    while (cap > 0 && fast_smem_layout(G, cap).total > fast_smem_budget(G)) cap -= kFastWarps * kTileKeys;
    const int sms = sm_count > 0 ? sm_count : 148;
    int split_len = tune_split_len;
    if (!split_len && upper <= cap && p.U >= 2 * sms) {
        // enough units to fill the machine without splitting them: one launch, every unit finished on chip
        split_len = upper;
    } else if (!split_len) {
        // Enough blocks to fill the machine about four times over, but no smaller than one tile per warp and no
        // larger than 2048 keys (long splits amortise the per-block prologue and merge) ...
        const int grain = kFastWarps * kTileKeys;
        const long long total_tiles = (long long)((upper + kTileKeys - 1) / kTileKeys) * p.U;
        const long long target_blocks = 4ll * sms;
        long long tiles_per_block = (total_tiles + target_blocks - 1) / target_blocks;
        if (tiles_per_block < kFastWarps) tiles_per_block = kFastWarps;
        split_len = (int)(tiles_per_block * kTileKeys > 2048 ? 2048 : tiles_per_block * kTileKeys);
        split_len = (split_len + grain - 1) / grain * grain;
        // ... then one split more or less if that leaves a fuller last wave: blocks run in waves of (SMs x resident
        // blocks), and a nearly empty last wave costs almost a whole one. Measured on 128 units of 1600 keys at two
        // blocks per SM, steady state: 4 splits (1.73 waves) 63.5 us per step, 5 splits (2.16 waves) 74-80 us.
        const long long slots = (long long)sms * fast_blocks_per_sm(G);
        const int s0 = (upper + split_len - 1) / split_len;
        double best_waste = 0.0;
        int best_len = split_len;
        for (int s = s0 > 1 ? s0 - 1 : 1; s <= s0 + 1; ++s) {
            const int len = ((upper + s - 1) / s + grain - 1) / grain * grain;
            const int n = (upper + len - 1) / len;
            const double waves = (double)p.U * n / (double)slots;
            const double waste = waves <= 1.0 ? 1.0 : std::ceil(waves) / waves;      // one wave or less: nothing to gain
            if (s == s0 - 1 || s == 1 || waste < best_waste - 0.02) { best_waste = waste; best_len = len; }
        }
        split_len = best_len;
        // ... or one wave of longer splits when the units nearly fill it: the mean unit cut into as many splits as fit
        // the resident slots, if that fills at least three quarters of them with splits of at most 1152 keys (the few
        // longer units take one split more). Measured on 128 units of mean 1650 and longest 2600 keys, G = 4, 296
        // slots (us per step): splits of 896 keys 55.9, 1024 58.0, 512 59.1, the rule above alone 65.6 (it follows the
        // longest unit between 4 x 512 and 6 x 384); longer splits lose again (1280: 65.4, 1536: 72.9), and 32 units of
        // 12 500 keys gained nothing from one wave of 1536.
        const int s1 = (int)(slots / p.U);
        if (s1 >= 1 && typical > 0) {
            const int len1 = ((typical + s1 - 1) / s1 + grain - 1) / grain * grain;
            if (len1 <= 1152 && len1 > split_len && 4ll * p.U * s1 >= 3ll * slots) split_len = len1;
        }
    }
    split_len = (split_len + kFastWarps * kTileKeys - 1) / (kFastWarps * kTileKeys) * (kFastWarps * kTileKeys);
    p.split_len = split_len;
    const int n_splits = (upper + split_len - 1) / split_len;
    if (n_splits > p.max_splits) return CORM_ERR_UNSUPPORTED;
    // on-chip finish for units of one split, as far as shared memory for their logits allows
    p.single_cap = split_len < cap ? split_len : cap;
    const FastSmem lay = fast_smem_layout(G, p.single_cap);
    const size_t smem = (size_t)lay.total;
    const bool all_single = n_splits == 1 && upper <= p.single_cap;      // every unit finishes inside its one block
    // who finishes the longer units: see the end of decode_fast_kernel
    const size_t fin = (size_t)(p.page_table ? 3 : 2) * ((p.C + 31) / 32 + 2) * 4;   // keep mask + prefix sums (+ page entries) of finalize_unit
    // ... or when units are so short that the serial walk (upper x G logits over 128 threads) is cheaper than a launch
    const bool many = finish_mode == 2 || (finish_mode != 3 && ((long long)p.U * n_splits >= 4ll * sms * fast_blocks_per_sm(G) ||
                                                                (long long)upper * G <= 2048));
    p.inline_finalize = !all_single && many && fin <= smem;
    const bool self = all_single || p.inline_finalize;
    if (self_finishing) *self_finishing = self;
    if (!self) p.unit_stamp = nullptr;            // the verdict launch finishes (some of) the units: no stamps, no chain
    p.chain_wait = want_chain && p.unit_stamp ? 1 : 0;
    p.early_trigger = want_trigger && self ? 1 : 0;
    const size_t fin1 = (size_t)kFastWarps * G * (16 + 512) + (size_t)2 * ((p.single_cap + 31) / 32 + 2) * 4 +
                        (size_t)2 * p.single_cap * 4;
    if (fin1 > (size_t)kFastWarps * fast_warp_bytes(G)) return CORM_ERR_UNSUPPORTED;
    if (smem > 227 * 1024) return CORM_ERR_UNSUPPORTED;
    auto launch = [&](auto kern) -> corm_status_t {
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: cudaFuncSetAttribute: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(n_splits, (unsigned)p.U);
        cfg.blockDim = dim3(kFastThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // launch latency hides behind the previous launch's tail
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, p);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: decode launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    corm_status_t rc;
    if (p.page_table) rc = G == 1 ? launch(decode_fast_kernel<1, true>) : G == 2 ? launch(decode_fast_kernel<2, true>) : launch(decode_fast_kernel<4, true>);
    else rc = G == 1 ? launch(decode_fast_kernel<1, false>) : G == 2 ? launch(decode_fast_kernel<2, false>) : launch(decode_fast_kernel<4, false>);
    if (rc != CORM_OK) return rc;
    *n_launched = 1;
    if (all_single || p.inline_finalize) return CORM_OK;
    // verdict launch for the units that do not
    const size_t vsmem = verdict_smem(p.C, n_splits, G, p.page_table != nullptr);
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
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may overlap the streaming kernel's tail
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, p, n_splits, batches);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: verdict launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    rc = G == 1 ? launch_v(decode_verdict_kernel<bf16_t, 128, 1>) : G == 2 ? launch_v(decode_verdict_kernel<bf16_t, 128, 2>)
                                                                           : launch_v(decode_verdict_kernel<bf16_t, 128, 4>);
    if (rc == CORM_OK) *n_launched = 2;
    return rc;
}

}  // namespace corm
