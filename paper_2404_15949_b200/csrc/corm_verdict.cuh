// Second launch of a decode step for units that span several splits: the work that follows the streaming pass
// (Algorithm 1's verdict row, register update, keep decision, compaction), spread over many blocks instead of one.
//
// The streaming kernel leaves, per unit, one partial record {m, Z, acc[D]} per split and query head and the scaled
// logits of every live key. Here a block owns 1024 or 2048 consecutive slots of one unit (one or two batches):
//   a. every block reduces the (m, Z) of the unit's splits to lse_g and the threshold of Definition 3.1 in log form
//      (a few dozen values; the same arithmetic in the same order in every block, so all blocks agree bit for bit);
//      block 0 of the unit also reduces the accumulators to the attention output of Eq. 1;
//   b. verdicts of its slots (OR over the group), register update, keep flag -> one bit per slot in a global mask;
//   c. the block that finishes last (arrival counter after a fence) scans the mask, fills the holes below the new
//      length with kept rows from above it, and publishes the new length. No block waits for another.
// The launch is programmatic-dependent on the streaming kernel: its blocks may become resident while the last
// streaming blocks still run, read what the streaming kernel does not write (lengths, registers and positions of
// the older slots), and only then wait for the streaming grid to complete.
#pragma once

#include "corm_common.cuh"

namespace corm {

constexpr int kVerdictThreads = 256;
constexpr int kVerdictPer = 4;                            // slots per thread and batch
constexpr int kVerdictBatch = kVerdictThreads * kVerdictPer;
constexpr int kVerdictMaxBatches = 2;                     // a block judges its slots in one or two batches of 1024: with two, the
                                                          // block's fixed chain of round trips (records, thresholds, arrival) is
                                                          // paid once per 2048 slots, which pays when one batch per block would
                                                          // need more than one wave of blocks (long units)
// batches per block for a launch over units of up to `upper` keys
inline int verdict_batches(int upper, int n_units, int sm_count) {
    const long long blocks = (long long)((upper + kVerdictBatch - 1) / kVerdictBatch) * n_units;
    return blocks > 4ll * sm_count ? kVerdictMaxBatches : 1;
}

__host__ __device__ inline int keepmask_words(int C) { return (C + 31) / 32 + 2; }

__host__ __device__ inline size_t verdict_smem(int C, int n_splits, int G, bool paged) {
    return (size_t)G * n_splits * (8 + 8 + 4) + 16 + (size_t)(paged ? 3 : 2) * keepmask_words(C) * 4;   // + keep mask, prefix sums (, page entries)
}

// BAL: the streaming pass was the balanced kernel (corm_balanced.cuh): a unit's records are the n_rec consecutive
// ones from rec0 on that the kernel lists in p.unit_rec, and the logits are stored [slot][G].
template <typename T, int D, int G, bool BAL = false>
__global__ void __launch_bounds__(kVerdictThreads, 4) decode_verdict_kernel(const __grid_constant__ DecodeParams p,
                                                                         const int n_splits, const int batches) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ double s_thr[G], s_Z[G];
    __shared__ int s_scan[kVerdictThreads];
    __shared__ int s_last;
    constexpr int NT = kVerdictThreads, kListCap = 512;
    __shared__ int s_lists[2 * kListCap];
    const int u = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = u / p.Hkv;
    const int32_t* pt_u = p.page_table ? p.page_table + (size_t)u * p.pt_stride : nullptr;
    const int room = pt_u ? __ldcg(p.page_room + u) : 1;                   // paged caches: a page for the appended row
    const int l_old = __ldcg(p.live_in + u), l = l_old + 1;
    if (l > p.C || !room) return;                                          // reported by the streaming kernel
    if (!BAL && (l + p.split_len - 1) / p.split_len == 1 && l <= p.single_cap) return;   // finished inside the streaming kernel
    const int chunk_slots = batches * kVerdictBatch;
    const int n_chunks = (l + chunk_slots - 1) / chunk_slots;
    if (chunk >= n_chunks) return;
    const int t = __ldg(p.base_tokens + b) + p.step + 1;
    const int n_obs = min(p.w, __ldg(p.base_obs + b) + p.step + 1);
    const bool evict_on = n_obs >= p.w;
    uint32_t* wordu = p.word + (size_t)u * p.C;
    int32_t* posu = p.pos + (size_t)u * p.C;
    const int base0 = chunk * chunk_slots;
    uint32_t wv[kVerdictPer];
    int32_t pv[kVerdictPer];
    auto load_regs = [&](int bbase) {                                      // registers and positions: not written by the streaming kernel
#pragma unroll
        for (int k = 0; k < kVerdictPer; ++k) {                            // the appended slot l_old starts as (0, t)
            const int j = bbase + k * NT + tid;
            wv[k] = j < l_old ? __ldcg(wordu + j) : 0u;
            pv[k] = j < l_old ? __ldcg(posu + j) : t;
        }
    };
    load_regs(base0);
    asm volatile("griddepcontrol.wait;" ::: "memory");                     // the streaming grid has completed
    // everything this block needs from the streaming kernel is requested at once: status, split records, logits
    const int status = __ldcg(p.status);
    const int2 ur = BAL ? __ldcg(p.unit_rec + u) : make_int2(u * p.max_splits, (l + p.split_len - 1) / p.split_len);
    const int n_act = min(ur.y, n_splits);                                 // n_splits bounds the shared-memory arrays
    const double* stash_u = p.stash + (size_t)u * G * p.C;
    double sv[kVerdictPer][G];
    auto load_logits = [&](int bbase) {
#pragma unroll
        for (int k = 0; k < kVerdictPer; ++k) {
            const int j = bbase + k * NT + tid;
#pragma unroll
            for (int g = 0; g < G; ++g)
                sv[k][g] = j < l ? __ldcg(BAL ? stash_u + (size_t)j * G + g : stash_u + (size_t)g * p.C + j) : -INFINITY;
        }
    };
    load_logits(base0);

    double* sm_m = reinterpret_cast<double*>(smem);                        // [G][n_splits]
    double* sm_Z = sm_m + (size_t)G * n_splits;
    float* sm_sc = reinterpret_cast<float*>(sm_Z + (size_t)G * n_splits);
    uint32_t* keep_sm = reinterpret_cast<uint32_t*>(smem + (((size_t)G * n_splits * 20 + 15) & ~(size_t)15));
    int* prefix = reinterpret_cast<int*>(keep_sm + keepmask_words(p.C));
    int32_t* pt_sm = prefix + keepmask_words(p.C);                         // paged caches: the unit's page entries (last block)
    const size_t pstride = partial_stride(D);
    const unsigned char* rec_u = p.partials + (size_t)ur.x * G * pstride;

    // a. split reduction
    for (int x = tid; x < G * n_act; x += NT) {
        const int g = x / n_act, s = x - g * n_act;
        const double* rec = reinterpret_cast<const double*>(rec_u + ((size_t)s * G + g) * pstride);
        sm_m[g * n_splits + s] = __ldcg(rec);
        sm_Z[g * n_splits + s] = __ldcg(rec + 1);
    }
    if (status == (int)CORM_ERR_TIMEOUT) return;                           // a copy never arrived: leave the unit as is
    __syncthreads();
    if (warp < G) {                                                        // warp g reduces head g, a split per lane
        const int g = warp;
        double m = -INFINITY;
        for (int s = lane; s < n_act; s += 32) m = fmax(m, sm_m[g * n_splits + s]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
        double Z = 0.0;
        for (int s = lane; s < n_act; s += 32) {
            const double sc = exp(sm_m[g * n_splits + s] - m);
            Z += sm_Z[g * n_splits + s] * sc;
            sm_sc[g * n_splits + s] = (float)sc;
        }
        Z = warp_sum(Z);                                                   // fixed tree: every block gets the same bits
        if (lane == 0) {
            s_Z[g] = Z;
            s_thr[g] = m + log(Z) + p.log_alpha - log((double)t);         // Definition 3.1: s >= lse + ln(alpha) - ln(t)
        }
    }
    __syncthreads();
    // b. verdicts, register update, keep flags of this block's slots
    uint32_t* keep_g = p.keepmask + (size_t)u * keepmask_words(p.C);
    int n_imp = 0;                                                         // keys this thread judged important
    for (int bt = 0; bt < batches; ++bt) {
        const int bbase = base0 + bt * kVerdictBatch;
        if (bbase >= l) break;                                             // uniform
        if (bt) { load_regs(bbase); load_logits(bbase); }
#pragma unroll
        for (int k = 0; k < kVerdictPer; ++k) {
            const int base = bbase + k * NT, j = base + tid;
            if (base >= l) break;                                          // uniform
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
            if (lane == 0 && base + warp * 32 < l && CORM_IN_RANGE((base >> 5) + warp < keepmask_words(p.C), p.status))
                keep_g[(base >> 5) + warp] = ballot;
        }
    }

    warp_count(p.counters + CNT_IMPORTANT, n_imp);                         // Section 3.1's sparsity

    // c. the last block of the unit to get here compacts it
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned prev = atomicAdd(p.ticket + u, 1u);
        s_last = (prev == (unsigned)(n_chunks - 1));
        if (s_last) p.ticket[u] = 0u;
        __threadfence();
    }
    __syncthreads();
    {   // Eq. 1: the unit's G x D outputs are shared out over its blocks
        const int per = (G * D + n_chunks - 1) / n_chunks, x_end = min(G * D, (chunk + 1) * per);
        for (int x = chunk * per + tid; x < x_end; x += NT) {
            const int g = x / D, c = x - g * D;
            float acc = 0.f;
            for (int s0 = 0; s0 < n_act; s0 += 8) {                       // eight loads in flight, summed in split order
                float a[8];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    a[k] = s0 + k < n_act
                               ? __ldcg(reinterpret_cast<const float*>(rec_u + ((size_t)(s0 + k) * G + g) * pstride + 16) + c)
                               : 0.f;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (s0 + k < n_act) acc += a[k] * sm_sc[g * n_splits + s0 + k];
            }
            Elem<T>::store(reinterpret_cast<T*>(p.out) + ((size_t)u * G + g) * D + c, (float)((double)acc / s_Z[g]));
        }
    }
    if (!s_last) return;
    int new_len = l, n_moved = 0;
    if (evict_on) {
        const int nwords = (l + 31) / 32;
        for (int i = tid; i < nwords; i += NT) {
            keep_sm[i] = __ldcg(keep_g + i);
            if (pt_u) pt_sm[i] = __ldcg(pt_u + i);                         // one entry per 32 slots, like the mask
        }
        __syncthreads();
        block_popc_scan<NT>(keep_sm, prefix, nwords, s_scan);
        new_len = prefix[nwords];
        if (new_len < l) {
            // the k-th kept row at or above new_len moves into the k-th hole below it; both lists are built word by
            // word from the keep mask (few bits qualify), in shared memory when they are short
            const int kept_below = kept_before(keep_sm, prefix, new_len);
            n_moved = new_len - kept_below;
            int* holes = s_lists;
            int* movers = s_lists + kListCap;
            if (n_moved > kListCap) {
                holes = reinterpret_cast<int*>(const_cast<double*>(stash_u));    // every block is done with the logits
                movers = holes + p.C;
            }
            for (int i = tid; i < nwords; i += NT) {
                const uint32_t m = keep_sm[i];
                const int j0 = i * 32;
                const uint32_t valid = l - j0 >= 32 ? 0xffffffffu : (1u << (l - j0)) - 1u;
                const uint32_t below = new_len - j0 >= 32 ? 0xffffffffu : (new_len > j0 ? (1u << (new_len - j0)) - 1u : 0u);
                uint32_t hm = ~m & valid & below;                  // evicted slots below the new length
                while (hm) {
                    const int bit = __ffs(hm) - 1;
                    hm &= hm - 1u;
                    holes[j0 - prefix[i] + __popc(~m & ((1u << bit) - 1u))] = j0 + bit;
                }
                uint32_t km = m & ~below;                          // kept slots at or above it
                while (km) {
                    const int bit = __ffs(km) - 1;
                    km &= km - 1u;
                    movers[prefix[i] + __popc(m & ((1u << bit) - 1u)) - kept_below] = j0 + bit;
                }
            }
            __syncthreads();
            const size_t slab_row0 = (size_t)u * p.C;
            block_move_rows<T, D, NT>(reinterpret_cast<T*>(p.K), reinterpret_cast<T*>(p.V),
                                      [&](int slot) -> size_t {
                                          return pt_u ? page_row(pt_sm[slot >> 5], slot, p.pool_pages, p.status) : slab_row0 + (size_t)slot;
                                      }, wordu, posu, movers, holes, n_moved, 0, 1, l, p.status);
        }
    }
    settle_pages<NT>(p.page_table, p.page_bits, p.page_room, p.pool_pages, p.pt_stride, p.U, u, l_old, new_len);
    if (tid == 0) {
        p.live_out[u] = new_len;
        publish_live(p.maxlive, p.step + 1, new_len);
        atomicAdd(p.counters + CNT_APPENDED, 1ull);
        atomicAdd(p.counters + CNT_ATTENDED, (unsigned long long)l);
        if (new_len < l) atomicAdd(p.counters + CNT_EVICTED, (unsigned long long)(l - new_len));
        if (n_moved) atomicAdd(p.counters + CNT_MOVED, (unsigned long long)n_moved);
    }
}

// Opt-in monitor of the premise of Section 3.3 (the current query resembles recent ones): Eq. 3 between every query
// head's query and its query of the previous decode step, summed into acc[0] (fp64) with the number of pairs in
// acc[1] (as an integer in the same 8 bytes), then the queries are kept for the next step. One warp per head.
template <typename T, int D>
__global__ void __launch_bounds__(128) query_similarity_kernel(const T* q, T* q_prev, int have_prev, int n_heads,
                                                               double* sum, unsigned long long* count) {
    const int lane = threadIdx.x & 31, head = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (head >= n_heads) return;
    double dot = 0.0, n1 = 0.0, n2 = 0.0;
    for (int c = lane; c < D; c += 32) {
        const double a = (double)Elem<T>::load(q + (size_t)head * D + c);
        if (have_prev) {
            const double b = (double)Elem<T>::load(q_prev + (size_t)head * D + c);
            dot = fma(a, b, dot); n1 = fma(a, a, n1); n2 = fma(b, b, n2);
        }
        Elem<T>::store(q_prev + (size_t)head * D + c, (float)a);
    }
    if (!have_prev) return;
    dot = warp_sum(dot); n1 = warp_sum(n1); n2 = warp_sum(n2);
    if (lane == 0 && n1 > 0.0 && n2 > 0.0) {
        atomicAdd(sum, dot / (sqrt(n1) * sqrt(n2)));
        atomicAdd(count, 1ull);
    }
}

}  // namespace corm
