// Persistent ("streaming") form of the bf16 / head_dim-128 decode kernel.
//
// Same arithmetic as decode_fast_kernel (corm_fast.cuh) - the same tile routines are called - but the grid is one
// wave of resident blocks that pull work items (unit, split) from a device queue, and every warp issues the TMA
// copies of its first tiles of the NEXT item before the block merges and finalizes the current one. The prologue
// latency of an item (live-length load, first tile from HBM) is thereby hidden behind the merge / verdict /
// compaction phase of its predecessor, which is what bounds throughput when units are short (a few tiles per warp).
// Splits of a unit are balanced in whole tiles. No block ever waits for another block: the queue is an atomic
// counter, multi-split units still finish in whichever block arrives last.
#pragma once

#include "corm_fast.cuh"

namespace corm {

struct StreamSmem {
    int tiles, qs, psm, stash, bars, merge, lists, total;
};
__host__ __device__ inline StreamSmem stream_smem_layout(int G, int single_cap, int C) {
    StreamSmem s;
    int off = 0;
    auto take = [&](int bytes) { int at = off; off = (off + bytes + 127) / 128 * 128; return at; };
    s.tiles = take(kFastWarps * fast_stages(G) * kTileBytes);
    s.qs = take(G * 128 * 8);
    s.psm = take(kFastWarps * kTileKeys * G * 4);
    s.stash = take(single_cap * G * 8);
    s.bars = take(kFastWarps * fast_stages(G) * 8);
    // per-warp {M, Z, acc[128]} records, then (after the block-level merge has consumed them) the keep mask and its
    // prefix sums for a unit of any length: the two share one region
    const int merge_bytes = kFastWarps * G * (16 + 4 * 128), list_bytes = 2 * ((C + 31) / 32 + 2) * 4;
    s.merge = take(merge_bytes > list_bytes ? merge_bytes : list_bytes);
    s.lists = s.merge;
    s.total = off;
    return s;
}

// One work item: a split of a unit, in whole tiles, balanced over the splits the unit needs.
struct StreamItem {
    int u, split, b, l_old, l, n_act, t, begin, end, n_tiles;
    bool active, cap_err;
};
__device__ __forceinline__ StreamItem stream_item(const DecodeParams& p, int item) {
    StreamItem it;
    it.u = item / p.n_splits;
    it.split = item - it.u * p.n_splits;
    it.b = it.u / p.Hkv;
    it.l_old = __ldcg(p.live_in + it.u);
    it.l = it.l_old + 1;
    it.cap_err = it.l > p.C;
    const int tiles = (it.l + kTileKeys - 1) / kTileKeys;
    const int want = (it.l + p.split_len - 1) / p.split_len;     // splits by length ...
    const int per = (tiles + want - 1) / want;                   // ... evened out in whole tiles
    it.n_act = (tiles + per - 1) / per;
    it.begin = it.split * per * kTileKeys;
    it.end = min(it.l, it.begin + per * kTileKeys);
    it.active = !it.cap_err && it.split < it.n_act;
    it.n_tiles = it.active ? (it.end - it.begin + kTileKeys - 1) / kTileKeys : 0;
    it.t = __ldg(p.base_tokens + it.b) + p.step + 1;
    return it;
}

template <int G>
__global__ void __launch_bounds__(kFastThreads, fast_blocks_per_sm(G)) decode_stream_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_item[2];
    __shared__ int s_last;
    __shared__ int s_failed;
    __shared__ double s_thr1[G];
    constexpr int NT = kFastThreads, NW = kFastWarps;
    constexpr int kKStages = fast_k_stages(G), kStagesPerWarp = fast_stages(G);
    constexpr int kRec = 16 + 4 * 128;
    constexpr int kPre = fast_max_single_cap(G) / NT;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_items = p.U * p.n_splits;
    const StreamSmem lay = stream_smem_layout(G, p.single_cap, p.C);
    unsigned char* my_tiles = smem + lay.tiles + warp * kStagesPerWarp * kTileBytes;
    const uint32_t my_bars = smem_addr(smem + lay.bars) + warp * kStagesPerWarp * 8;
    double* qs = reinterpret_cast<double*>(smem + lay.qs);
    float* psm = reinterpret_cast<float*>(smem + lay.psm) + warp * kTileKeys * G;
    double* stash_sm = reinterpret_cast<double*>(smem + lay.stash);
    unsigned char* merge = smem + lay.merge;
    unsigned char* lists = smem + lay.lists;
    const int h = lane >> 4, ci = lane & 15;
    const int key_own = 16 * h + 8 * (ci & 1) + (ci >> 1);        // tile key this lane owns after the fold
    const double inv_root_d = 0.088388347648318440550;            // 1/sqrt(128)

    if (tid == 0) { s_failed = 0; s_item[0] = (int)atomicAdd(p.queue, 1u); }
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStagesPerWarp; ++s) mbar_init(my_bars + s * 8, 1);
        fence_mbar_init();
        fence_async_smem();
    }
    __syncthreads();

    // Per-warp stage bookkeeping runs across items: tiles issued / consumed so far on the K ring and the V ring.
    int k_issued = 0, k_used = 0, v_issued = 0, v_used = 0;
    auto issue_k = [&](const StreamItem& im, int it) {             // lane 0 only
        const int k0 = im.begin + (warp + it * NW) * kTileKeys, slot = k_issued % kKStages;
        const uint32_t bytes = (uint32_t)min(kTileKeys, im.end - k0) * kRowBytes;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(p.K) + ((size_t)im.u * p.C + k0) * kRowBytes;
        mbar_expect_tx(my_bars + slot * 8, bytes);
        bulk_load(smem_addr(my_tiles + slot * kTileBytes), src, bytes, my_bars + slot * 8);
    };
    auto issue_v = [&](const StreamItem& im, int it) {
        const int k0 = im.begin + (warp + it * NW) * kTileKeys, slot = v_issued % kVStages;
        const uint32_t bytes = (uint32_t)min(kTileKeys, im.end - k0) * kRowBytes;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(p.V) + ((size_t)im.u * p.C + k0) * kRowBytes;
        mbar_expect_tx(my_bars + (kKStages + slot) * 8, bytes);
        bulk_load(smem_addr(my_tiles + (kKStages + slot) * kTileBytes), src, bytes, my_bars + (kKStages + slot) * 8);
    };
    auto my_tiles_of = [&](const StreamItem& im) { return im.n_tiles > warp ? (im.n_tiles - warp + NW - 1) / NW : 0; };
    // first tiles of an item: as many as the rings hold (all lanes keep the counters, lane 0 issues)
    auto issue_first = [&](const StreamItem& im) {
        const int n = my_tiles_of(im);
        for (int it = 0; it < min(n, kKStages); ++it) { if (lane == 0) issue_k(im, it); ++k_issued; }
        for (int it = 0; it < min(n, kVStages); ++it) { if (lane == 0) issue_v(im, it); ++v_issued; }
    };

    int cur = s_item[0], par = 0;
    StreamItem ci_item = stream_item(p, cur < n_items ? cur : 0);
    if (cur < n_items) issue_first(ci_item);
    bool failed = false;

    while (cur < n_items) {
        const StreamItem im = ci_item;
        if (tid == 0) s_item[par ^ 1] = (int)atomicAdd(p.queue, 1u);   // the item after this one
        const int u = im.u, l = im.l, l_old = im.l_old, t = im.t;
        const bool single = im.active && im.n_act == 1 && l <= p.single_cap;
        uint32_t* wordu = p.word + (size_t)u * p.C;
        int32_t* posu = p.pos + (size_t)u * p.C;
        unsigned char* Ku = reinterpret_cast<unsigned char*>(p.K) + (size_t)u * p.C * kRowBytes;
        unsigned char* Vu = reinterpret_cast<unsigned char*>(p.V) + (size_t)u * p.C * kRowBytes;
        if (im.cap_err && im.split == 0 && tid == 0) {               // the slab is full: report, leave the unit untouched
            atomicCAS(p.status, 0, (int)CORM_ERR_CAPACITY);
            p.live_out[u] = l_old;
            publish_live(p.maxlive, p.step + 1, l_old);
        }
        // registers and positions of the slots this thread judges if the unit finishes inside this block
        uint32_t wv[kPre];
        int32_t pv[kPre];
#pragma unroll
        for (int k = 0; k < kPre; ++k) { wv[k] = 0u; pv[k] = 0; }
        if (single) {
#pragma unroll
            for (int k = 0; k < kPre; ++k) {
                const int j = tid + k * NT;
                if (j < l_old) { wv[k] = __ldcg(wordu + j); pv[k] = __ldcg(posu + j); }
                else if (j == l_old) { wv[k] = 0u; pv[k] = t; }       // the token appended by this step
            }
        }
        if (im.active) {
            const bf16_t* qg = reinterpret_cast<const bf16_t*>(p.q) + (size_t)u * G * 128;
            for (int x = tid; x < G * 128; x += NT) qs[x] = (double)Elem<bf16_t>::load(qg + x);
        }
        __syncthreads();                                             // qs and s_item[par ^ 1] are visible
        const int nxt = s_item[par ^ 1];
        const StreamItem ni = stream_item(p, nxt < n_items ? nxt : 0);   // its loads are consumed only after this item's tiles

        double qd[G][8];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < 8; ++e) qd[g][e] = qs[g * 128 + ci * 8 + e];
        double M[G], Zl[G];
        unsigned long long acc2[G][4];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            M[g] = -INFINITY; Zl[g] = 0.0;
#pragma unroll
            for (int e = 0; e < 4; ++e) acc2[g][e] = 0ull;
        }
        const int my_n = my_tiles_of(im);
        for (int it = 0; it < my_n; ++it) {
            const int k0 = im.begin + (warp + it * NW) * kTileKeys;
            const int n_valid = min(kTileKeys, im.end - k0);
            const bool has_new = (l_old >= k0 && l_old < k0 + kTileKeys);   // this tile holds the appended token
            const int kslot = k_used % kKStages, vslot = v_used % kVStages;
            unsigned char* ktile = my_tiles + kslot * kTileBytes;
            unsigned char* vtile = my_tiles + (kKStages + vslot) * kTileBytes;
            if (!mbar_wait(my_bars + kslot * 8, (k_used / kKStages) & 1)) failed = true;
            ++k_used;
            if (has_new) {   // append: the new row goes to the slab and replaces whatever the copy fetched for that slot
                const uint4* kn = reinterpret_cast<const uint4*>(p.k_new) + (size_t)u * 16;
                if (lane < 16) {
                    const uint4 x = kn[lane];
                    *reinterpret_cast<uint4*>(ktile + (l_old - k0) * kRowBytes + lane * 16) = x;
                    reinterpret_cast<uint4*>(Ku + (size_t)l_old * kRowBytes)[lane] = x;
                }
                if (lane == 0) { wordu[l_old] = 0u; posu[l_old] = t; }
                __syncwarp();
            }
            double sown[G];
            qk_tile<G>(ktile, qd, lane, sown);
            __syncwarp();
            if (it + kKStages < my_n) { if (lane == 0) { fence_async_smem(); issue_k(im, it + kKStages); } ++k_issued; }

            const bool valid = key_own < n_valid;
            const int j_own = k0 + key_own;
            double sv[G], Mn[G], sc[G], ex[G];
            float mt[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                sv[g] = valid ? sown[g] * inv_root_d : -INFINITY;         // Eq. 2's exponent
                mt[g] = (float)sv[g];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int g = 0; g < G; ++g) mt[g] = fmaxf(mt[g], __shfl_xor_sync(0xffffffffu, mt[g], o));
#pragma unroll
            for (int g = 0; g < G; ++g) Mn[g] = fmax(M[g], (double)mt[g]);
#pragma unroll
            for (int g = 0; g < G; ++g) sc[g] = exp_nonpos(M[g] - Mn[g]);    // exactly 1 when the reference did not move
#pragma unroll
            for (int g = 0; g < G; ++g) ex[g] = valid ? exp_nonpos(sv[g] - Mn[g]) : 0.0;
            bool moved = false;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                moved |= (Mn[g] != M[g]);
                Zl[g] = fma(Zl[g], sc[g], ex[g]);
                M[g] = Mn[g];
                psm[key_own * G + g] = (float)ex[g];
                if (valid) {
                    if (single) stash_sm[g * p.single_cap + j_own] = sv[g];
                    else p.stash[((size_t)u * G + g) * p.C + j_own] = sv[g];
                }
            }
            if (moved) {                                                   // warp-uniform
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float scf = (float)sc[g];
                    const unsigned long long sc2 = pack_f32x2(scf, scf);
#pragma unroll
                    for (int e = 0; e < 4; ++e) mul_f32x2(acc2[g][e], sc2);
                }
            }
            __syncwarp();

            if (!mbar_wait(my_bars + (kKStages + vslot) * 8, (v_used / kVStages) & 1)) failed = true;
            ++v_used;
            if (has_new) {
                const uint4* vn = reinterpret_cast<const uint4*>(p.v_new) + (size_t)u * 16;
                if (lane < 16) {
                    const uint4 x = vn[lane];
                    *reinterpret_cast<uint4*>(vtile + (l_old - k0) * kRowBytes + lane * 16) = x;
                    reinterpret_cast<uint4*>(Vu + (size_t)l_old * kRowBytes)[lane] = x;
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
                    for (int e = 0; e < 4; ++e) fma_f32x2(acc2[g][e], p2, v2[e]);       // Eq. 1
                }
            }
            __syncwarp();
            if (it + kVStages < my_n) { if (lane == 0) { fence_async_smem(); issue_v(im, it + kVStages); } ++v_issued; }
        }
        // this warp's rings are free: start fetching its first tiles of the next item, then finish this one
        if (nxt < n_items) {
            if (lane == 0) fence_async_smem();
            issue_first(ni);
        }

        if (im.active) {
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
        }
        __syncthreads();
        bool run_unit_finalize = false;
        if (im.active) {
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
                        unsigned char* rec = p.partials + (((size_t)u * p.max_splits + im.split) * G + g) * pstride;
                        reinterpret_cast<float*>(rec + 16)[c] = a;
                    }
                }
                if (tid == 0) {
                    if (single) s_thr1[g] = Mb + log(Zb) + p.log_alpha - log((double)t);
                    else {
                        unsigned char* rec = p.partials + (((size_t)u * p.max_splits + im.split) * G + g) * pstride;
                        reinterpret_cast<double*>(rec)[0] = Mb; reinterpret_cast<double*>(rec)[1] = Zb;
                    }
                }
            }
            if (single) {
                __syncthreads();
                int* holes = reinterpret_cast<int*>(p.stash + (size_t)u * G * p.C);      // global scratch of this unit: unused on this path
                finalize_single<G, NT, kPre>(p, u, im.b, l, t, s_thr1, stash_sm, p.single_cap, wv, pv, lists, holes,
                                             holes + p.C);
            } else {
                // publish, then let the last-arriving split of this unit run the finalize phase
                __threadfence();
                __syncthreads();
                if (tid == 0) {
                    const unsigned prev = atomicAdd(p.ticket + u, 1u);
                    s_last = (prev == (unsigned)(im.n_act - 1));
                    if (s_last) p.ticket[u] = 0u;
                    __threadfence();
                }
                __syncthreads();
                run_unit_finalize = s_last != 0;
            }
        }
        if (run_unit_finalize) finalize_unit<bf16_t, 128, G, NT>(p, u, im.b, l, im.n_act, t, lists);
        __syncthreads();                 // merge area, lists, qs and stash_sm are free for the next item
        cur = nxt;
        ci_item = ni;
        par ^= 1;
    }
    if (failed) atomicCAS(p.status, 0, (int)CORM_ERR_TIMEOUT);
    // the last block to leave rewinds the queue for the next launch
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned done = atomicAdd(p.queue + 1, 1u);
        if (done == gridDim.x - 1) { p.queue[0] = 0u; p.queue[1] = 0u; __threadfence(); }
    }
}

// Host side: work-item sizing and launch of the streaming kernel.
inline corm_status_t launch_decode_stream(DecodeParams& p, int G, int upper, int tune_split_len, int sm_count,
                                          cudaStream_t st) {
    if (G != 1 && G != 2 && G != 4) return CORM_ERR_UNSUPPORTED;
    const int slots = (sm_count > 0 ? sm_count : 148) * fast_blocks_per_sm(G);
    int split_len = tune_split_len;
    if (!split_len) {
        // items of at least 24 tiles where the work allows (the per-item merge and finalize are then a small part),
        // about four items per resident block for balance, never more than 2048 keys
        const long long total_tiles = (long long)((upper + kTileKeys - 1) / kTileKeys) * p.U;
        long long tiles_per_item = (total_tiles + 4ll * slots - 1) / (4ll * slots);
        if (tiles_per_item < 24) tiles_per_item = 24;
        split_len = (int)(tiles_per_item * kTileKeys > 2048 ? 2048 : tiles_per_item * kTileKeys);
    }
    split_len = (split_len + kTileKeys - 1) / kTileKeys * kTileKeys;
    p.split_len = split_len;
    p.n_splits = (upper + split_len - 1) / split_len;
    if (p.n_splits > p.max_splits) return CORM_ERR_UNSUPPORTED;
    p.single_cap = split_len < fast_max_single_cap(G) ? split_len : fast_max_single_cap(G);
    while (p.single_cap > 0 && stream_smem_layout(G, p.single_cap, p.C).total > fast_smem_budget(G)) p.single_cap -= kTileKeys;
    const size_t smem = (size_t)stream_smem_layout(G, p.single_cap, p.C).total;
    if (smem > 227 * 1024) return CORM_ERR_UNSUPPORTED;
    const long long items = (long long)p.U * p.n_splits;
    const unsigned grid = (unsigned)(items < slots ? items : slots);
    auto launch = [&](auto kern) -> corm_status_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: cudaFuncSetAttribute: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        kern<<<grid, kFastThreads, smem, st>>>(p);
        e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: decode launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    if (G == 1) return launch(decode_stream_kernel<1>);
    if (G == 2) return launch(decode_stream_kernel<2>);
    return launch(decode_stream_kernel<4>);
}

}  // namespace corm
