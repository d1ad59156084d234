// Shared device-side definitions of the CORM kernels: parameter blocks, element access, and the per-unit
// "finalize" phase (split reduction, verdict, register update, keep decision, hole-filling compaction) that the
// last-arriving thread block of a unit runs inside a decode kernel (the generic kernels always, the fast kernel when
// it does not leave the unit to the verdict launch).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/corm.h"

namespace corm {

// Raises a kernel's dynamic shared-memory limit on the current device when a launch needs more than any earlier one
// did; the driver call is skipped otherwise (it costs more than a microsecond and decode launches are that short).
inline cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes) {
    struct Entry { const void* kernel; int device; size_t bytes; };
    constexpr int kSlots = 256;                       // fixed table: nothing is allocated here, on host or device
    static std::mutex mu;
    static Entry seen[kSlots];
    static int n_seen = 0;
    if (bytes <= 48 * 1024) return cudaSuccess;
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    Entry* slot = nullptr;
    for (int i = 0; i < n_seen && !slot; ++i)
        if (seen[i].kernel == kernel && seen[i].device == device) slot = &seen[i];
    if (slot && bytes <= slot->bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return e;
    if (slot) slot->bytes = bytes;
    else if (n_seen < kSlots) seen[n_seen++] = Entry{kernel, device, bytes};   // a full table only costs the shortcut
    return e;
}

// |fp32 dot - exact dot| <= kDotErr * |q| * |k| for a 128-term dot product of bf16 values formed the way the fast
// kernels fold it (bf16 x bf16 products are exact in fp32): 7 roundings in a lane's 8-term FMA chain and 5 in the
// cross-lane fold make 12 * 2^-24 to first order; 16 * 2^-24 leaves a third of slack for the higher-order terms and
// for the rounding of the fp32 key norm itself.
constexpr double kDotErr = 16.0 / 16777216.0;
// 1 / sqrt(head_dim), the scale of Eq. 2's exponent
__host__ __device__ constexpr double inv_root_dim(int D) { return D == 128 ? 0.088388347648318440550 : 0.125; }

// Counters kept per layer in the arena (64-bit, updated with atomics by the finalize phase / the prompt pass).
enum { CNT_APPENDED = 0, CNT_EVICTED = 1, CNT_MOVED = 2, CNT_ATTENDED = 3, CNT_IMPORTANT = 4, CNT_NEAR = 5, CNT_COUNT = 6 };

struct DecodeParams {
    void* K;                  // [U][C][D] this layer's key slabs
    void* V;                  // [U][C][D]
    uint32_t* word;           // [U][C] verdict registers
    int32_t* pos;             // [U][C] absolute 1-based token positions
    const int32_t* live_in;   // [U] live length before this step
    int32_t* live_out;        // [U] live length after this step (the other half of a double buffer)
    const int32_t* base_tokens;  // [B] tokens seen when the step counter was last rebased
    const int32_t* base_obs;     // [B] verdict rows recorded at that time
    uint32_t* ticket;         // [U] arrival counters of the splits of a unit (zero between steps)
    uint32_t* ticket2;        // [U] second arrival counters (balanced kernel: blocks done with their verdicts)
    uint32_t* ticket3;        // [U] third arrival counters (balanced kernel: blocks done with their share of the row moves)
    unsigned long long* move_info;   // [U] balanced kernel: the unit's move word (zero between steps)
    unsigned long long* counters;  // [CNT_COUNT]
    int32_t* status;          // sticky device status
    unsigned long long* maxlive;  // (steps done << 32 | longest live length after that step), atomicMax; may be null
    double* stash;            // [U*G][C] scaled logits of this step (scratch)
    unsigned char* partials;  // [U][max_splits][G] records {double m, double Z, float acc[D]} (scratch)
    uint32_t* keepmask;       // [U][ceil(C/32)+2] keep bits of the verdict launch (scratch)
    int2* unit_rec;           // [U] balanced kernel -> verdict launch: a unit's first record and its record count (scratch)
    unsigned long long* unit_stamp;  // [U] (decode steps the unit has finished << 32 | its live length after the last of them),
                                     // written by the block that finishes a unit inside the streaming launch; null = not kept
    int32_t chain_wait;       // fast kernel: a block waits for its own unit's stamp of the previous step, not for the previous launch
    int32_t early_trigger;    // fast kernel: the next launch on the stream may become resident once every block of this one has started
    const void* q;            // [B][Hq][D]
    const void* k_new;        // [B][Hkv][D]
    const void* v_new;        // [B][Hkv][D]
    void* out;                // [B][Hq][D]
    int32_t U, Hkv, C, split_len, max_splits, step, w, r;
    int32_t single_cap;       // fast kernel: units up to this length finish inside one block (0 = never)
    int32_t inline_finalize;  // fast kernel: the last-arriving split of a longer unit finishes it (else the verdict launch does)
    double log_alpha;         // ln(alpha), -inf for alpha = 0
    // paged caches only (page_table == nullptr: every unit owns a slab of C rows of K and V)
    int32_t* page_table;      // [U][pt_stride] page number + 1 of each 32-key page of a unit, 0 = none
    uint32_t* page_bits;      // [pool_pages / 32] bit set = page in use
    int32_t* page_room;       // [U] 1 iff the unit owns the page its next append goes to (0: pool exhausted)
    int32_t pool_pages, pt_stride;
};

struct PromptParams {
    const void* k_prompt;     // [B][Hkv][p_max][D]
    const void* v_prompt;
    const void* q_last;       // [B][Hq][w][D]
    const int32_t* prompt_lens;  // [B] device copy
    void* K;
    void* V;
    uint32_t* word;
    int32_t* pos;
    int32_t* live_out;        // [U]
    unsigned long long* counters;
    int32_t* status;
    unsigned long long* maxlive;
    double* stash;            // scratch, reused for temporary registers
    int32_t U, Hkv, C, p_max, w, r;
    double log_alpha;
    double bound_scale;       // multiplies the proven fp32 error bound of the tiled pass (1; tests raise it)
    int32_t* page_table;      // paged caches only, as in DecodeParams
    uint32_t* page_bits;
    int32_t* page_room;
    int32_t pool_pages, pt_stride;
};

__host__ __device__ inline size_t partial_stride(int D) { return 16 + 4 * (size_t)D; }

// A unit's step is complete: every write of the block that finished it (row moves, registers, positions) comes before
// the stamp, which a block of the next step's launch may be waiting for (wait_unit_stamp). Called by one thread after
// a block barrier that follows those writes.
__device__ __forceinline__ void publish_unit_stamp(const DecodeParams& p, int u, int new_len) {
    if (!p.unit_stamp) return;
    const unsigned long long v = ((unsigned long long)(uint32_t)(p.step + 1) << 32) | (uint32_t)new_len;
    __threadfence();
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.unit_stamp + u), "l"(v) : "memory");
}

// ---- element access: the cache dtype is only a storage format; all logits are formed in fp64 ----
struct bf16_t { uint16_t bits; };

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

// round-to-nearest-even float -> bf16 bits (finite inputs; NaN stays NaN)
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
    uint32_t x = __float_as_uint(f);
    if ((x & 0x7f800000u) == 0x7f800000u) return (uint16_t)((x >> 16) | ((x & 0xffffu) ? 0x40u : 0u));
    x += 0x7fffu + ((x >> 16) & 1u);
    return (uint16_t)(x >> 16);
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kBytes = 4;
    static __device__ __forceinline__ float load(const float* p) { return *p; }
    static __device__ __forceinline__ void store(float* p, float v) { *p = v; }
};
template <> struct Elem<bf16_t> {
    static constexpr int kBytes = 2;
    static __device__ __forceinline__ float load(const bf16_t* p) { return bf16_bits_to_float(p->bits); }
    static __device__ __forceinline__ void store(bf16_t* p, float v) { p->bits = float_to_bf16_bits(v); }
};

// N contiguous elements starting at p (p aligned to N*sizeof(T)), widened to float.
template <typename T, int N> __device__ __forceinline__ void load_slice(const T* p, float (&out)[N]);
template <> __device__ __forceinline__ void load_slice<float, 4>(const float* p, float (&out)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <> __device__ __forceinline__ void load_slice<float, 2>(const float* p, float (&out)[2]) {
    float2 v = *reinterpret_cast<const float2*>(p);
    out[0] = v.x; out[1] = v.y;
}
template <> __device__ __forceinline__ void load_slice<bf16_t, 4>(const bf16_t* p, float (&out)[4]) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xffff0000u);
    out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xffff0000u);
}
template <> __device__ __forceinline__ void load_slice<bf16_t, 2>(const bf16_t* p, float (&out)[2]) {
    uint32_t v = *reinterpret_cast<const uint32_t*>(p);
    out[0] = __uint_as_float(v << 16); out[1] = __uint_as_float(v & 0xffff0000u);
}

// Device-side errors are sticky: the status word keeps the numerically largest code reported (a broken invariant
// outranks an expired wait, which outranks a full slab), so that a later, harmless code cannot hide an earlier severe
// one nor the other way round. After any non-zero status the cache must be reset before it is used again.
__device__ __forceinline__ void report_status(int32_t* status, corm_status_t code) { atomicMax(status, (int32_t)code); }

// Range checks. compute-sanitizer cannot be run where this library is developed, so the kernels can check themselves:
// a build with -DCORM_DEBUG_BOUNDS tests every slot, list entry, record and mask index before it is used; a failed
// test reports CORM_ERR_INTERNAL through the status word and SKIPS the access (the kernel goes on and returns
// normally). The release build compiles the tests away, except for page-table entries (page_row below): those come
// from memory, and a bad one would otherwise become a wild address.
#ifdef CORM_DEBUG_BOUNDS
#define CORM_IN_RANGE(cond, status) ((cond) ? true : (corm::report_status((status), CORM_ERR_INTERNAL), false))
#else
#define CORM_IN_RANGE(cond, status) true
#endif

// Adds the warp's total of n to a 64-bit counter (one atomic per warp; all lanes must call).
__device__ __forceinline__ void warp_count(unsigned long long* counter, int n) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    if ((threadIdx.x & 31) == 0 && n) atomicAdd(counter, (unsigned long long)n);
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Publishes a unit's new live length for the host's launch sizing: the word holds the latest step in its high half,
// so the maximum over all units of the most recent step wins.
__device__ __forceinline__ void publish_live(unsigned long long* maxlive, int steps_done, int live) {
    if (maxlive) atomicMax(maxlive, ((unsigned long long)(unsigned)steps_done << 32) | (unsigned)live);
}

__device__ __forceinline__ uint32_t window_mask(int w) { return w >= 32 ? 0xffffffffu : ((1u << w) - 1u); }

// The per-key 32-bit register has two encodings. Windows of up to 32 queries: a shift register, bit b = verdict of
// the query b steps ago (Algorithm 1's message column). Wider windows (the paper runs up to 256): the step t of the
// latest query that found the key important, 0 if none has; "some query among the last w found it important" is
// then t_now - stamp < w, which selects exactly the columns Algorithm 1's any() over the last w rows selects.
__device__ __forceinline__ uint32_t update_register(uint32_t old, bool imp, int w, int t) {
    return w <= 32 ? (((old << 1) | (imp ? 1u : 0u)) & window_mask(w)) : (imp ? (uint32_t)t : old);
}
__device__ __forceinline__ bool register_needed(uint32_t reg, int w, int t) {
    return w <= 32 ? reg != 0u : (reg != 0u && t - (int)reg < w);
}

// ---- paged caches --------------------------------------------------------------------------------------------
// The paper's result is memory saved; with one slab of C rows per unit the saving is only logical. A paged cache
// keeps K and V of a layer in one pool of 32-key pages (one tile of the streaming kernel) shared by all its units:
// slot j of a unit lives in row (page_table[j / 32] - 1) * 32 + j % 32 of the pool. Registers and positions stay in
// per-unit arrays of C entries (8 bytes per key against 2 * D * e). Invariant between steps: a unit of n live keys
// owns the pages of slots 0 .. n, i.e. n / 32 + 1 pages, so the next append always has a row to go to; the block
// that finishes a unit's step (or its prompt pass) claims or releases pages to restore it. A unit whose claim failed
// because the pool is exhausted has no page for its next append: its page_room flag is cleared, and the next step
// (which reads the flag next to the live length, not behind it) reports CORM_ERR_CAPACITY and leaves the unit
// untouched, like a full slab.
constexpr int kPageKeys = 32;

// Row of a slot whose page-table entry is `entry` (page + 1). An entry outside the pool means the table is broken:
// it is reported and the slot's row inside page 0 is returned, so that no address is ever formed from a bad entry
// (checked in every build). The data is wrong from then on; the status tells the caller to reset the cache.
__device__ __forceinline__ size_t page_row(int entry, int slot, int pool_pages, int32_t* status) {
    if (entry <= 0 || entry > pool_pages) { report_status(status, CORM_ERR_INTERNAL); entry = 1; }
    return (size_t)(entry - 1) * kPageKeys + (slot & 31);
}

// row of slot `slot` in the layer's K / V storage: through the unit's page table, or inside its slab
__device__ __forceinline__ size_t kv_row(const int32_t* pt_u, size_t slab_row0, int slot, int pool_pages, int32_t* status) {
    return pt_u ? page_row(__ldcg(pt_u + (slot >> 5)), slot, pool_pages, status) : slab_row0 + (size_t)slot;
}

// Claims one free page for page-table entry `index` of unit u (of n_units). Every unit has a home region of the
// pool, pool_pages / n_units pages starting at its share of the bitmap, and entry `index` first tries the page
// `index` places into that region: while units stay inside their regions their pages are contiguous and in slot
// order, as in a slab, and units do not contend for the same bitmap words. If that page is taken the bitmap is
// scanned from there on, wrapping around. A page is claimed by setting its bit with atomicOr and
// belongs to the caller iff the bit was clear before. Bounded: every word is visited once and the inner loop ends
// after at most 32 rounds (each failed round adds a bit to w). Returns the page number or -1 when the pool is
// exhausted.
__device__ inline int claim_page(uint32_t* bits, int pool_pages, int n_units, int u, int index) {
    const int n_words = pool_pages >> 5;
    const long long home = (long long)u * pool_pages / n_units + index;      // preferred page
    int i = (int)((home >> 5) % n_words);
    {
        const uint32_t bit = 1u << (home & 31);
        if (!(atomicOr(bits + i, bit) & bit)) return i * 32 + (int)(home & 31);
    }
    for (int tries = 0; tries < n_words; ++tries) {
        uint32_t w = __ldcg(bits + i);
        while (w != 0xffffffffu) {
            const uint32_t bit = 1u << (__ffs((int)~w) - 1);
            const uint32_t old = atomicOr(bits + i, bit);
            if (!(old & bit)) return i * 32 + __ffs((int)bit) - 1;
            w = old | bit;
        }
        i = (i + 1 == n_words) ? 0 : i + 1;
    }
    return -1;
}

// Restores the page invariant of unit u after a decode step that took it from l_old live keys (pages 0 .. l_old / 32
// owned) to new_len. Called by every thread of the block that finished the unit, after its row moves: the barrier
// below orders the block's reads of rows in released pages before another unit can claim them.
template <int NT>
__device__ __forceinline__ void settle_pages(int32_t* page_table, uint32_t* page_bits, int32_t* page_room, int pool_pages,
                                             int pt_stride, int n_units, int u, int l_old, int new_len) {
    if (!page_table) return;
    const int have = l_old / kPageKeys + 1, need = new_len / kPageKeys + 1;
    if (need == have) return;                                     // the usual step: nothing to claim or release (uniform)
    __syncthreads();
    int32_t* pt_u = page_table + (size_t)u * pt_stride;
    for (int i = need + (int)threadIdx.x; i < have; i += NT) {
        const int pg = __ldcg(pt_u + i) - 1;
        pt_u[i] = 0;
        if (pg >= 0) atomicAnd(page_bits + (pg >> 5), ~(1u << (pg & 31)));
    }
    if (need > have && have < pt_stride && threadIdx.x == 0) {    // the next append starts a new page
        const int pg = claim_page(page_bits, pool_pages, n_units, u, have);
        pt_u[have] = pg + 1;
        if (pg < 0) page_room[u] = 0;                             // exhausted: the unit's next step reports it
    }
}

// Prompt pass: unit u ends with `kept` live keys and owns no page yet (the pass starts from an empty pool). Claims
// kept / 32 + 1 pages, one per thread. Returns false (to every thread) if the pool ran out. pt_copy, if given, is
// a shared-memory copy of the unit's new table entries for the gather that follows.
template <int NT>
__device__ __forceinline__ bool claim_unit_pages(int32_t* page_table, uint32_t* page_bits, int32_t* page_room, int pool_pages,
                                                 int pt_stride, int n_units, int u, int kept, int32_t* pt_copy = nullptr) {
    if (!page_table) return true;
    int32_t* pt_u = page_table + (size_t)u * pt_stride;
    const int need = min(kept / kPageKeys + 1, pt_stride);
    int failed = 0;
    for (int i = (int)threadIdx.x; i < need; i += NT) {
        const int pg = claim_page(page_bits, pool_pages, n_units, u, i);
        pt_u[i] = pg + 1;
        if (pt_copy) pt_copy[i] = pg + 1;
        failed |= (pg < 0);
    }
    const bool ok = !__syncthreads_or(failed);      // also makes the table entries visible to the whole block
    if (threadIdx.x == 0) page_room[u] = ok ? 1 : 0;
    return ok;
}

// Exclusive prefix sums of popc(mask[i]) into prefix[0..nwords], block-wide. scratch holds NT ints.
// Each thread sums a contiguous run of words; warp 0 scans the NT run totals with shuffles.
template <int NT>
__device__ void block_popc_scan(const uint32_t* mask, int* prefix, int nwords, int* scratch) {
    const int tid = threadIdx.x, lane = tid & 31;
    const int per = (nwords + NT - 1) / NT;
    const int lo = min(tid * per, nwords), hi = min(lo + per, nwords);
    int sum = 0;
    for (int i = lo; i < hi; ++i) sum += __popc(mask[i]);
    scratch[tid] = sum;
    __syncthreads();
    if (tid < 32) {
        constexpr int kPer = NT / 32;
        int v[kPer], tot = 0;
#pragma unroll
        for (int k = 0; k < kPer; ++k) { v[k] = scratch[lane * kPer + k]; tot += v[k]; }
        int incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int run = incl - tot;
#pragma unroll
        for (int k = 0; k < kPer; ++k) { scratch[lane * kPer + k] = run; run += v[k]; }
        if (lane == 31) prefix[nwords] = incl;
    }
    __syncthreads();
    int run = scratch[tid];
    for (int i = lo; i < hi; ++i) { prefix[i] = run; run += __popc(mask[i]); }
    __syncthreads();
}

__device__ __forceinline__ int kept_before(const uint32_t* mask, const int* prefix, int j) {
    return prefix[j >> 5] + __popc(mask[j >> 5] & ((1u << (j & 31)) - 1u));
}

// Hole filling: row movers[i] (K row, V row, register, position) is copied to slot holes[i], i < n_moved, by the whole
// block. Sources lie at or above the new length, destinations below it, so copies never overlap. Each warp takes
// four rows at a time and issues all their loads before the first store (the copies are latency-, not
// bandwidth-limited). Rows are D*sizeof(T) bytes = a multiple of 16.
// row_of(slot) gives the slot's row in the layer's K / V storage (Kl, Vl).
// part / n_parts: this block takes the chunks of NT / 8 rows numbered part, part + n_parts, ... (several blocks
// sharing one unit's moves); the default is every chunk.
template <typename T, int D, int NT, int KROWS = 4, typename RowOf>
__device__ __forceinline__ void block_move_rows(T* Kl, T* Vl, RowOf row_of, uint32_t* wordu, int32_t* posu,
                                                const int* movers, const int* holes, int n_moved, int part = 0,
                                                int n_parts = 1, int slot_limit = 0x7fffffff, int32_t* status = nullptr) {
    constexpr int kChunks = D * Elem<T>::kBytes / 16, kIter = (2 * kChunks + 31) / 32, kRows = KROWS, NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i0 = (part * NW + warp) * kRows; i0 < n_moved; i0 += n_parts * NW * kRows) {
        int src[kRows], dst[kRows];
        size_t srow[kRows], drow[kRows];                 // rows of the layer's K / V storage (Kl, Vl)
        uint4 buf[kRows][kIter];
        uint32_t wd = 0u;
        int32_t ps = 0;
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const bool on = i0 + r < n_moved;
            src[r] = on ? movers[i0 + r] : -1;
            dst[r] = on ? holes[i0 + r] : -1;
            if (on && !CORM_IN_RANGE(src[r] >= 0 && src[r] < slot_limit && dst[r] >= 0 && dst[r] < slot_limit, status))
                src[r] = dst[r] = -1;                      // the row is left where it is
            srow[r] = on ? row_of(src[r]) : 0;
            drow[r] = on ? row_of(dst[r]) : 0;
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            if (src[r] < 0) continue;
#pragma unroll
            for (int x = 0; x < kIter; ++x) {
                const int c = lane + 32 * x;
                if (c < kChunks) buf[r][x] = __ldcg(reinterpret_cast<const uint4*>(Kl + srow[r] * D) + c);
                else if (c < 2 * kChunks) buf[r][x] = __ldcg(reinterpret_cast<const uint4*>(Vl + srow[r] * D) + (c - kChunks));
            }
            if (lane == r) { wd = __ldcg(wordu + src[r]); ps = __ldcg(posu + src[r]); }
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            if (src[r] < 0) continue;
#pragma unroll
            for (int x = 0; x < kIter; ++x) {
                const int c = lane + 32 * x;
                if (c < kChunks) reinterpret_cast<uint4*>(Kl + drow[r] * D)[c] = buf[r][x];
                else if (c < 2 * kChunks) reinterpret_cast<uint4*>(Vl + drow[r] * D)[c - kChunks] = buf[r][x];
            }
            if (lane == r) { wordu[dst[r]] = wd; posu[dst[r]] = ps; }
        }
    }
}

// Finalize phase of one unit, run by the whole block that arrived last (every split of the unit has published its
// partial record and its logits). Steps, in the order of Algorithm 1:
//   1. reduce the split partials -> out (Eq. 1) and lse_g = ln sum_j exp(s_gj) per query head (Eq. 2's denominator)
//   2. verdict of every live key: OR over the group of [s_gj >= lse_g + ln(alpha) - ln(t)]  (Definition 3.1 in log
//      form; GQA rule), shifted into the key's register
//   3. once w rows exist: keep iff register != 0 or position > t - r; holes below the new length are filled with
//      kept rows from above it (as many row copies as there are holes; sources and destinations are disjoint)
// smem: 2*(ceil(C/32)+2) 32-bit words of dynamic shared memory, 3*(ceil(C/32)+2) for a paged cache (the unit's page
// entries are staged there for the row moves).
template <typename T, int D, int G, int NT>
__device__ void finalize_unit(const DecodeParams& p, int u, int b, int l, int n_act, int t, unsigned char* smem) {
    __shared__ double s_thr[G];
    __shared__ int s_scan[NT];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cap_words = (p.C + 31) / 32 + 2;
    uint32_t* keepmask = reinterpret_cast<uint32_t*>(smem);
    int* prefix = reinterpret_cast<int*>(keepmask + cap_words);
    const int32_t* pt_u = p.page_table ? p.page_table + (size_t)u * p.pt_stride : nullptr;
    int32_t* pt_sm = prefix + cap_words;
    if (pt_u)
        for (int i = tid; i < (l + 31) / 32; i += NT) pt_sm[i] = __ldcg(pt_u + i);   // visible after the barriers below
    uint32_t* wordu = p.word + (size_t)u * p.C;
    int32_t* posu = p.pos + (size_t)u * p.C;
    const size_t pstride = partial_stride(D);

    // 1. split reduction
    for (int g = 0; g < G; ++g) {
        const unsigned char* rec0 = p.partials + ((size_t)u * p.max_splits * G + g) * pstride;
        double m = -INFINITY;
        for (int s = 0; s < n_act; ++s)
            m = fmax(m, __ldcg(reinterpret_cast<const double*>(rec0 + (size_t)s * G * pstride)));
        double Z = 0.0;
        float acc[(D + NT - 1) / NT];
#pragma unroll
        for (int i = 0; i < (D + NT - 1) / NT; ++i) acc[i] = 0.f;
        for (int s = 0; s < n_act; ++s) {
            const unsigned char* rec = rec0 + (size_t)s * G * pstride;
            const double ms = __ldcg(reinterpret_cast<const double*>(rec));
            const double sc = exp(ms - m);
            Z += __ldcg(reinterpret_cast<const double*>(rec) + 1) * sc;
            const float scf = (float)sc;
            const float* a = reinterpret_cast<const float*>(rec + 16);
#pragma unroll
            for (int i = 0; i < (D + NT - 1) / NT; ++i) {
                const int c = tid + i * NT;
                if (c < D) acc[i] += __ldcg(a + c) * scf;
            }
        }
        T* outp = reinterpret_cast<T*>(p.out) + ((size_t)u * G + g) * D;
#pragma unroll
        for (int i = 0; i < (D + NT - 1) / NT; ++i) {
            const int c = tid + i * NT;
            if (c < D) Elem<T>::store(outp + c, (float)((double)acc[i] / Z));
        }
        if (tid == 0) s_thr[g] = m + log(Z) + p.log_alpha - log((double)t);
    }
    __syncthreads();

    // 2. verdicts, register update, keep flags
    const int n_obs = min(p.w, __ldg(p.base_obs + b) + p.step + 1);
    const bool evict_on = n_obs >= p.w;
    const double* stash_u = p.stash + (size_t)u * G * p.C;
    constexpr int kBatch = (G >= 4 ? 4 : 8);                                      // slots per thread whose loads are issued together
    int n_imp = 0;                                                                // keys this thread judged important
    for (int base0 = 0; base0 < l; base0 += kBatch * NT) {
        double sv[kBatch][G];
        uint32_t wv[kBatch];
        int32_t pv[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
            const int j = base0 + k * NT + tid;
            wv[k] = 0u; pv[k] = 0;
#pragma unroll
            for (int g = 0; g < G; ++g) sv[k][g] = -INFINITY;
            if (j < l) {
#pragma unroll
                for (int g = 0; g < G; ++g) sv[k][g] = __ldcg(stash_u + (size_t)g * p.C + j);
                wv[k] = __ldcg(wordu + j);
                pv[k] = __ldcg(posu + j);
            }
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
            const int base = base0 + k * NT, j = base + tid;
            if (base >= l) break;                                  // uniform
            bool keep = false;
            if (j < l) {
                bool imp = false;
#pragma unroll
                for (int g = 0; g < G; ++g) imp |= (sv[k][g] >= s_thr[g]);
                const uint32_t wd = update_register(wv[k], imp, p.w, t);
                if (CORM_IN_RANGE(j < p.C, p.status)) wordu[j] = wd;
                keep = !evict_on || register_needed(wd, p.w, t) || pv[k] > t - p.r;
                n_imp += imp ? 1 : 0;
            }
            const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
            if (lane == 0 && base + warp * 32 < l && CORM_IN_RANGE((base >> 5) + warp < cap_words, p.status))
                keepmask[(base >> 5) + warp] = ballot;
        }
    }
    warp_count(p.counters + CNT_IMPORTANT, n_imp);         // Section 3.1's sparsity: keys judged important this step
    __syncthreads();
    int new_len = l, n_moved = 0;
    if (evict_on) {
        const int nwords = (l + 31) / 32;
        block_popc_scan<NT>(keepmask, prefix, nwords, s_scan);
        new_len = prefix[nwords];
        if (new_len < l) {
            // 3. hole filling: the k-th kept row at or above new_len moves into the k-th hole below it
            int* holes = reinterpret_cast<int*>(const_cast<double*>(stash_u));   // the logits are consumed
            int* movers = holes + p.C;
            const int kept_below = kept_before(keepmask, prefix, new_len);   // kept rows already below new_len
            n_moved = new_len - kept_below;
            for (int j = tid; j < l; j += NT) {
                const int kb = kept_before(keepmask, prefix, j);
                const bool kept = (keepmask[j >> 5] >> (j & 31)) & 1u;
                if (j < new_len && !kept) holes[j - kb] = j;
                if (j >= new_len && kept) movers[kb - kept_below] = j;
            }
            __syncthreads();
            const size_t slab_row0 = (size_t)u * p.C;
            block_move_rows<T, D, NT>(reinterpret_cast<T*>(p.K), reinterpret_cast<T*>(p.V),
                                      [&](int slot) -> size_t {
                                          return pt_u ? page_row(pt_sm[slot >> 5], slot, p.pool_pages, p.status) : slab_row0 + (size_t)slot;
                                      }, wordu, posu, movers, holes, n_moved, 0, 1, l, p.status);
        }
    }
    settle_pages<NT>(p.page_table, p.page_bits, p.page_room, p.pool_pages, p.pt_stride, p.U, u, l - 1, new_len);
    if (p.unit_stamp) __syncthreads();            // the row moves of every warp come before the stamp
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

}  // namespace corm
