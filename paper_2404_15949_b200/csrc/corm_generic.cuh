// Generic kernels: any supported dtype / head_dim / group size, written for clarity. One warp per key, lanes
// split the head dimension, fp64 logits. The bf16 / head_dim 128 decode path has a faster kernel of its own;
// this one serves fp32 caches, head_dim 64 and the prompt-end pass.
#pragma once

#include "corm_common.cuh"

namespace corm {

constexpr int kGenericThreads = 128;
constexpr int kPromptThreads = 256;

__host__ __device__ inline size_t generic_decode_smem(int D, int G, int C, bool paged) {
    const size_t warps = kGenericThreads / 32;
    size_t a = (size_t)G * D * 8 + warps * G * 16 + warps * G * D * 4;
    size_t b = (size_t)(paged ? 3 : 2) * ((C + 31) / 32 + 2) * 4;
    return a > b ? a : b;
}

// Decode step, one block per (split of a unit's live range, unit).
template <typename T, int D, int G>
__global__ void __launch_bounds__(kGenericThreads) decode_generic_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_last;
    constexpr int NT = kGenericThreads, NW = NT / 32, NPL = D / 32;
    const int u = blockIdx.y, split = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = u / p.Hkv;
    const int32_t* pt_u = p.page_table ? p.page_table + (size_t)u * p.pt_stride : nullptr;
    const int room = pt_u ? __ldcg(p.page_room + u) : 1;
    const int l_old = __ldcg(p.live_in + u), l = l_old + 1;
    if (l > p.C || !room) {   // the slab is full (paged: no page for the new row): report, leave the unit untouched
        if (split == 0 && tid == 0) { report_status(p.status, CORM_ERR_CAPACITY); p.live_out[u] = l_old; publish_live(p.maxlive, p.step + 1, l_old); }
        return;
    }
    const int n_act = (l + p.split_len - 1) / p.split_len;
    if (split >= n_act) return;
    const int t = __ldg(p.base_tokens + b) + p.step + 1;
    const int begin = split * p.split_len, end = min(l, begin + p.split_len);
    T* Kl = reinterpret_cast<T*>(p.K);                 // the layer's K / V storage: slabs or page pool
    T* Vl = reinterpret_cast<T*>(p.V);
    const size_t slab_row0 = (size_t)u * p.C;

    // append the current token (Algorithm 1's keys include it; its register starts at zero)
    if (l_old >= begin && l_old < end) {
        const T* kn = reinterpret_cast<const T*>(p.k_new) + (size_t)u * D;
        const T* vn = reinterpret_cast<const T*>(p.v_new) + (size_t)u * D;
        const size_t row = kv_row(pt_u, slab_row0, l_old, p.pool_pages, p.status);
        for (int c = tid; c < D; c += NT) { Kl[row * D + c] = kn[c]; Vl[row * D + c] = vn[c]; }
        if (tid == 0) { p.word[(size_t)u * p.C + l_old] = 0u; p.pos[(size_t)u * p.C + l_old] = t; }
        __syncthreads();
    }

    double* qs = reinterpret_cast<double*>(smem);                      // [G][D]
    double* sm_mz = qs + G * D;                                        // [NW][G][2]
    float* sm_acc = reinterpret_cast<float*>(sm_mz + NW * G * 2);      // [NW][G][D]
    const T* qg = reinterpret_cast<const T*>(p.q) + (size_t)u * G * D;
    for (int i = tid; i < G * D; i += NT) qs[i] = (double)Elem<T>::load(qg + i);
    __syncthreads();

    const int c0 = lane * NPL;
    double qr[G][NPL];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int i = 0; i < NPL; ++i) qr[g][i] = qs[g * D + c0 + i];
    double m[G], Z[G];
    float acc[G][NPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY; Z[g] = 0.0;
#pragma unroll
        for (int i = 0; i < NPL; ++i) acc[g][i] = 0.f;
    }
    const double root_d = sqrt((double)D);
    for (int j = begin + warp; j < end; j += NW) {
        float kf[NPL], vf[NPL];
        const size_t row = kv_row(pt_u, slab_row0, j, p.pool_pages, p.status);
        load_slice<T, NPL>(Kl + row * D + c0, kf);
        load_slice<T, NPL>(Vl + row * D + c0, vf);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            double part = 0.0;
#pragma unroll
            for (int i = 0; i < NPL; ++i) part += qr[g][i] * (double)kf[i];
            const double s = warp_sum(part) / root_d;                  // Eq. 2's exponent
            if (lane == 0) p.stash[((size_t)u * G + g) * p.C + j] = s;
            float pj;
            if (s > m[g]) {                                            // running-max softmax
                const double sc = exp(m[g] - s);
                Z[g] = Z[g] * sc + 1.0;
                const float scf = (float)sc;
#pragma unroll
                for (int i = 0; i < NPL; ++i) acc[g][i] *= scf;
                m[g] = s;
                pj = 1.f;
            } else {
                const double e = exp(s - m[g]);
                Z[g] += e;
                pj = (float)e;
            }
#pragma unroll
            for (int i = 0; i < NPL; ++i) acc[g][i] += pj * vf[i];     // Eq. 1
        }
    }
    // merge the warps of this block into one partial record per query head
#pragma unroll
    for (int g = 0; g < G; ++g) {
        if (lane == 0) { sm_mz[(warp * G + g) * 2] = m[g]; sm_mz[(warp * G + g) * 2 + 1] = Z[g]; }
#pragma unroll
        for (int i = 0; i < NPL; ++i) sm_acc[(warp * G + g) * D + c0 + i] = acc[g][i];
    }
    __syncthreads();
    const size_t pstride = partial_stride(D);
    for (int g = 0; g < G; ++g) {
        double M = -INFINITY;
        for (int w = 0; w < NW; ++w) M = fmax(M, sm_mz[(w * G + g) * 2]);
        double Zt = 0.0;
        unsigned char* rec = p.partials + (((size_t)u * p.max_splits + split) * G + g) * pstride;
        for (int c = tid; c < D; c += NT) {
            float a = 0.f;
            for (int w = 0; w < NW; ++w) a += sm_acc[(w * G + g) * D + c] * (float)exp(sm_mz[(w * G + g) * 2] - M);
            reinterpret_cast<float*>(rec + 16)[c] = a;
        }
        if (tid == 0) {
            for (int w = 0; w < NW; ++w) Zt += sm_mz[(w * G + g) * 2 + 1] * exp(sm_mz[(w * G + g) * 2] - M);
            reinterpret_cast<double*>(rec)[0] = M;
            reinterpret_cast<double*>(rec)[1] = Zt;
        }
    }
    // publish, then let the last-arriving split of this unit run the finalize phase
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
    finalize_unit<T, D, G, NT>(p, u, b, l, n_act, t, smem);
}

// window slots handled per pass of the generic prompt kernel (at most 64 (slot, head) rows at a time)
__host__ __device__ inline int prompt_chunk_slots(int G, int w) { const int s = 64 / G; return s < w ? s : w; }

__host__ __device__ inline size_t prompt_smem(int G, int w, int C) {
    const size_t warps = kPromptThreads / 32, rows = (size_t)G * prompt_chunk_slots(G, w);
    size_t a = warps * rows * 16 + rows * 8;
    size_t b = (size_t)2 * ((C + 31) / 32 + 2) * 4;
    return a + b;
}

// Prompt-end pass, one block per unit. Pass 1: log-sum-exp of every recorded causal row; pass 2: verdict bits of
// every key for those rows -> registers; then keep flags, prefix sums and an ordered gather into the slab.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kPromptThreads) prompt_generic_kernel(const __grid_constant__ PromptParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_scan[kPromptThreads];
    constexpr int NT = kPromptThreads, NW = NT / 32, NPL = D / 32;
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = u / p.Hkv;
    const int P = __ldg(p.prompt_lens + b);
    if (P > p.C) {
        if (tid == 0) { report_status(p.status, CORM_ERR_CAPACITY); p.live_out[u] = 0; }
        return;
    }
    if (P == 0) {
        if (tid == 0) {
            p.live_out[u] = 0;
            if (p.page_table) {  // an empty unit still owns the page its first append goes to
                const int pg = claim_page(p.page_bits, p.pool_pages, p.U, u, 0);
                p.page_table[(size_t)u * p.pt_stride] = pg + 1;
                p.page_room[u] = pg >= 0;
            }
        }
        return;
    }
    const int w = p.w, wp = min(P, w);
    const int cs = prompt_chunk_slots(G, w), rows = G * cs;           // window slots per pass, rows per pass
    double* sm_mz = reinterpret_cast<double*>(smem);                   // [NW][rows][2], row = g * cs + (slot - slot0)
    double* sm_thr = sm_mz + (size_t)NW * rows * 2;                    // [rows]
    uint32_t* keepmask = reinterpret_cast<uint32_t*>(sm_thr + rows);
    int* prefix = reinterpret_cast<int*>(keepmask + (p.C + 31) / 32 + 2);
    const T* Kp = reinterpret_cast<const T*>(p.k_prompt) + (size_t)u * p.p_max * D;
    const T* Vp = reinterpret_cast<const T*>(p.v_prompt) + (size_t)u * p.p_max * D;
    const T* Q = reinterpret_cast<const T*>(p.q_last) + (size_t)u * G * w * D;   // [G][w][D]
    const int c0 = lane * NPL;
    const double root_d = sqrt((double)D);
    uint32_t* tmp_word = reinterpret_cast<uint32_t*>(p.stash + (size_t)u * G * p.C);

    // the recorded queries are taken oldest first, a few window slots per pass over the keys
    for (int slot0 = w - wp; slot0 < w; slot0 += cs) {
        const int slot1 = min(w, slot0 + cs);
        for (int i = tid; i < NW * rows; i += NT) { sm_mz[2 * i] = -INFINITY; sm_mz[2 * i + 1] = 0.0; }
        __syncthreads();
        // pass 1: running max / sum of every row, per warp (only lane 0 owns the warp's entries)
        for (int j = warp; j < P; j += NW) {
            float kf[NPL];
            load_slice<T, NPL>(Kp + (size_t)j * D + c0, kf);
            for (int row = slot0; row < slot1; ++row) {
                const int i = P - (w - 1 - row);          // position of this query; it sees keys 1..i
                if (j + 1 > i) continue;
                for (int g = 0; g < G; ++g) {
                    float qf[NPL];
                    load_slice<T, NPL>(Q + ((size_t)g * w + row) * D + c0, qf);
                    double part = 0.0;
#pragma unroll
                    for (int k = 0; k < NPL; ++k) part += (double)qf[k] * (double)kf[k];
                    const double s = warp_sum(part) / root_d;
                    if (lane == 0) {
                        double* mz = sm_mz + ((size_t)warp * rows + g * cs + (row - slot0)) * 2;
                        if (s > mz[0]) { mz[1] = mz[1] * exp(mz[0] - s) + 1.0; mz[0] = s; }
                        else mz[1] += exp(s - mz[0]);
                    }
                }
            }
        }
        __syncthreads();
        for (int rr = tid; rr < rows; rr += NT) {
            const int row = slot0 + rr % cs;
            if (row >= slot1) { sm_thr[rr] = INFINITY; continue; }
            double M = -INFINITY, Z = 0.0;
            for (int x = 0; x < NW; ++x) M = fmax(M, sm_mz[((size_t)x * rows + rr) * 2]);
            for (int x = 0; x < NW; ++x)
                Z += sm_mz[((size_t)x * rows + rr) * 2 + 1] * exp(sm_mz[((size_t)x * rows + rr) * 2] - M);
            const int i = P - (w - 1 - row);
            sm_thr[rr] = M + log(Z) + p.log_alpha - log((double)i);  // Definition 3.1 in log form, threshold alpha/i
        }
        __syncthreads();
        // pass 2: verdicts of these queries enter the registers (shift register: the query at position P ends in
        // bit 0; wide windows: the position of the newest query that found the key important)
        for (int j = warp; j < P; j += NW) {
            float kf[NPL];
            load_slice<T, NPL>(Kp + (size_t)j * D + c0, kf);
            uint32_t wd = slot0 == w - wp ? 0u : tmp_word[j];          // written by this same thread in the previous pass
            for (int row = slot0; row < slot1; ++row) {
                const int i = P - (w - 1 - row);
                bool bit = false;
                if (j + 1 <= i) {
                    for (int g = 0; g < G; ++g) {
                        float qf[NPL];
                        load_slice<T, NPL>(Q + ((size_t)g * w + row) * D + c0, qf);
                        double part = 0.0;
#pragma unroll
                        for (int k = 0; k < NPL; ++k) part += (double)qf[k] * (double)kf[k];
                        const double s = warp_sum(part) / root_d;
                        bit |= (s >= sm_thr[g * cs + (row - slot0)]);
                    }
                }
                wd = update_register(wd, bit, w, i);
            }
            if (lane == 0) tmp_word[j] = wd;
        }
        __syncthreads();
    }
    const bool evict_on = wp >= w;
    for (int base = 0; base < P; base += NT) {
        const int j = base + tid;
        bool keep = false;
        if (j < P) keep = !evict_on || register_needed(tmp_word[j], w, P) || (j + 1) > P - p.r;
        const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
        if (lane == 0 && base + warp * 32 < P) keepmask[(base >> 5) + warp] = ballot;
    }
    __syncthreads();
    const int nwords = (P + 31) / 32;
    block_popc_scan<NT>(keepmask, prefix, nwords, s_scan);
    const int kept_total = prefix[nwords];
    const int32_t* pt_u = p.page_table ? p.page_table + (size_t)u * p.pt_stride : nullptr;
    if (!claim_unit_pages<NT>(p.page_table, p.page_bits, p.page_room, p.pool_pages, p.pt_stride, p.U, u, kept_total)) {
        if (tid == 0) { report_status(p.status, CORM_ERR_CAPACITY); p.live_out[u] = 0; }   // the pool is too small
        return;
    }
    T* Kl = reinterpret_cast<T*>(p.K);
    T* Vl = reinterpret_cast<T*>(p.V);
    constexpr int kChunks = D * Elem<T>::kBytes / 16;
    for (int j = warp; j < P; j += NW) {
        if (!((keepmask[j >> 5] >> (j & 31)) & 1u)) continue;
        const int dst = kept_before(keepmask, prefix, j);
        const uint4* ks = reinterpret_cast<const uint4*>(Kp + (size_t)j * D);
        const uint4* vs = reinterpret_cast<const uint4*>(Vp + (size_t)j * D);
        const size_t drow = kv_row(pt_u, (size_t)u * p.C, dst, p.pool_pages, p.status);
        uint4* kd = reinterpret_cast<uint4*>(Kl + drow * D);
        uint4* vd = reinterpret_cast<uint4*>(Vl + drow * D);
        for (int c = lane; c < 2 * kChunks; c += 32) {
            if (c < kChunks) kd[c] = ks[c];
            else vd[c - kChunks] = vs[c - kChunks];
        }
        if (lane == 0) { p.word[(size_t)u * p.C + dst] = tmp_word[j]; p.pos[(size_t)u * p.C + dst] = j + 1; }
    }
    if (tid == 0) {
        p.live_out[u] = kept_total;
        publish_live(p.maxlive, 0, kept_total);
        atomicAdd(p.counters + CNT_APPENDED, (unsigned long long)P);
        if (kept_total < P) atomicAdd(p.counters + CNT_EVICTED, (unsigned long long)(P - kept_total));
    }
}

}  // namespace corm
