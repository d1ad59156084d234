// Prompt-end pass for bf16 caches with head_dim 128 (any supported group size and window).
//
// The w recorded prompt queries of the G query heads of a unit form w*G "rows"; every row needs the log-sum-exp of
// its causal attention row (Eq. 2) before any verdict (Definition 3.1) can be taken. Two launches, both with one
// block per (unit, split of the prompt):
//   1. prompt_lse_kernel: fp64 logits of four rows at a time against 32-key tiles (the decode kernel's transposing
//      fold), lane-private running (max, sum) per row, partial (max, sum) per split; the last-arriving split of a
//      unit combines them into one threshold per row: lse + ln(alpha) - ln(position of the query).
//   2. prompt_verdict_kernel: recomputes the logits tile by tile, packs the verdict bits of each key (OR over the
//      heads of a query, 0 for keys newer than the query) into its register; the last-arriving split applies
//      Algorithm 1's keep rule, scans the keep mask and gathers the surviving K, V rows, registers and positions
//      into the slab in token order.
// K is read (rows/4 + 1) times, mostly from L2; nothing else of the prompt is read except the surviving V rows.
#pragma once

#include "corm_fast.cuh"

namespace corm {

constexpr int kPromptFastThreads = 256;
constexpr int kPromptFastWarps = kPromptFastThreads / 32;

struct PromptFastParams {
    PromptParams p;
    unsigned char* partials;      // scratch: [U][n_splits][rows] {double m, double Z}, then [U][rows] thresholds
    uint32_t* ticket;             // [U] arrival counters (zero between launches)
    int32_t split_len, n_splits;
    int32_t slot0, slot1;         // window slots [slot0, slot1) recorded by this pair of launches (oldest slot = 0)
    int32_t rows;                 // (slot1 - slot0) * G
};

__host__ __device__ inline size_t prompt_fast_smem(int rows, int C, bool paged) {
    size_t a = (size_t)rows * 256 + (size_t)kPromptFastWarps * rows * 16 + (size_t)rows * 16;  // q rows (bf16), per-warp (m, Z), thresholds + error factors
    size_t b = (size_t)(paged ? 3 : 2) * ((C + 31) / 32 + 2) * 4;                              // keep mask + prefix (+ page entries) of the last arriver
    return a + b + 256;
}

// qk_tile for a tile that lives in global memory and may be ragged: rows >= n_valid are read from row n_valid - 1
// (their sums are ignored by the caller).
template <int G>
__device__ __forceinline__ void qk_tile_clamped(const unsigned char* ktile, int n_valid, const double (&qd)[G][8],
                                                int lane, double (&sown)[G]) {
    const int h = lane >> 4, i = lane & 15, m = i >> 1, b0 = i & 1;
    double r[2][G];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        double a[G][8];
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const int key = min(16 * h + 8 * (it ^ b0) + (s ^ m), n_valid - 1);
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(ktile + key * kRowBytes + i * 16));
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

// fp32 form of qk_tile_clamped (bf16 x bf16 products are exact in fp32), with one more folded row: the squared norm
// of the lane's key, which scales the proven bound kDotErr |q| |k| on the accumulation error of its logits.
template <int G>
__device__ __forceinline__ void qk_tile_clamped32(const unsigned char* ktile, int n_valid, const float (&qf)[G][8],
                                                  int lane, float (&sown)[G], float& n2own) {
    const int h = lane >> 4, i = lane & 15, m = i >> 1, b0 = i & 1;
    float r[2][G + 1];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        float a[G + 1][8];
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const int key = min(16 * h + 8 * (it ^ b0) + (s ^ m), n_valid - 1);
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(ktile + key * kRowBytes + i * 16));
            float kf[8];
            unpack8_to_float(raw, kf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float acc = qf[g][0] * kf[0];
#pragma unroll
                for (int e = 1; e < 8; ++e) acc = fmaf(qf[g][e], kf[e], acc);
                a[g][s] = acc;
            }
            float nn = kf[0] * kf[0];
#pragma unroll
            for (int e = 1; e < 8; ++e) nn = fmaf(kf[e], kf[e], nn);
            a[G][s] = nn;
        }
#pragma unroll
        for (int g = 0; g <= G; ++g) {
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
    n2own = r[0][G] + __shfl_xor_sync(0xffffffffu, r[1][G], 1);
}

// One logit exactly: query row q (128 bf16 in shared memory) against key row k (128 bf16 in global memory), fp64.
__device__ __noinline__ double exact_logit(const uint16_t* q, const unsigned char* k) {
    double acc = 0.0;
    for (int c = 0; c < 16; ++c) {
        const uint4 kr = __ldg(reinterpret_cast<const uint4*>(k) + c);
        const uint4 qr = *reinterpret_cast<const uint4*>(q + c * 8);
        double kd[8], qd[8];
        unpack8_to_double(kr, kd);
        unpack8_to_double(qr, qd);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fma(qd[e], kd[e], acc);
    }
    return acc;
}

// Rows of one launch are numbered r = (rho - slot0) * G + g (query slot rho of the window, head g); the query of
// slot rho sits at prompt position P - (w - 1 - rho) and exists iff rho >= w - min(P, w). Windows whose rows do not
// fit one launch (more than 64 rows) are recorded by several launch pairs, oldest slots first.
__device__ __forceinline__ void load_row_group32(const uint16_t* q_sm, int group, int ci, float (&qf)[4][8]) {
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const uint4 raw = *reinterpret_cast<const uint4*>(q_sm + (size_t)(4 * group + x) * 128 + ci * 8);
        unpack8_to_float(raw, qf[x]);
    }
}
__device__ __forceinline__ void load_row_group(const uint16_t* q_sm, int group, int ci, double (&qd)[4][8]) {
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const uint4 raw = *reinterpret_cast<const uint4*>(q_sm + (size_t)(4 * group + x) * 128 + ci * 8);
        unpack8_to_double(raw, qd[x]);
    }
}

// Shared prologue of both kernels: stage the q rows (row-major r = rho*G + g, padded to a multiple of four rows).
__device__ __forceinline__ void stage_q_rows(const PromptParams& p, int u, int G, int slot0, int rows, int rows_pad,
                                             uint16_t* q_sm) {
    const uint16_t* Q = reinterpret_cast<const uint16_t*>(p.q_last) + (size_t)u * G * p.w * 128;   // [G][w][128]
    for (int x = threadIdx.x; x < rows_pad * 16; x += blockDim.x) {          // 16-byte chunks
        const int r = x >> 4, c = x & 15, rho = slot0 + r / G, g = r % G;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < rows) v = __ldg(reinterpret_cast<const uint4*>(Q + ((size_t)g * p.w + rho) * 128) + c);
        reinterpret_cast<uint4*>(q_sm + (size_t)r * 128)[c] = v;
    }
}

template <int G>
__global__ void __launch_bounds__(kPromptFastThreads) prompt_lse_kernel(const __grid_constant__ PromptFastParams fp) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_last;
    const PromptParams& p = fp.p;
    constexpr int NW = kPromptFastWarps;
    const int u = blockIdx.y, split = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = u / p.Hkv, P = __ldg(p.prompt_lens + b), w = p.w, wp = min(P, w);
    const int rows = fp.rows, rows_pad = (rows + 3) / 4 * 4, groups = rows_pad / 4, slot0 = fp.slot0;
    const int begin = split * fp.split_len, end = min(P, begin + fp.split_len);
    const int n_act = (P + fp.split_len - 1) / fp.split_len;
    if (P == 0 || split >= n_act) return;
    uint16_t* q_sm = reinterpret_cast<uint16_t*>(smem);
    double* mz_sm = reinterpret_cast<double*>(smem + (size_t)rows_pad * 256);        // [NW][rows_pad][2]
    stage_q_rows(p, u, G, slot0, rows, rows_pad, q_sm);
    __syncthreads();
    const unsigned char* Kp = reinterpret_cast<const unsigned char*>(p.k_prompt) + (size_t)u * p.p_max * kRowBytes;
    const int h = lane >> 4, ci = lane & 15, key_own = 16 * h + 8 * (ci & 1) + (ci >> 1);
    const double inv_root_d = 0.088388347648318440550;
    const int n_tiles = (end - begin + kTileKeys - 1) / kTileKeys;
    for (int gi = 0; gi < groups; ++gi) {
        // query positions of the four rows of this group (0 = row does not exist)
        int qpos[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const int r = 4 * gi + x, rho = slot0 + r / G;
            qpos[x] = (r < rows && rho >= w - wp) ? P - (w - 1 - rho) : 0;
        }
        double m[4], Z[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) { m[x] = -1e300; Z[x] = 0.0; }
        if (qpos[0] | qpos[1] | qpos[2] | qpos[3]) {
            double qd[4][8];
            load_row_group(q_sm, gi, ci, qd);
            for (int tix = warp; tix < n_tiles; tix += NW) {
                const int k0 = begin + tix * kTileKeys, n_valid = min(kTileKeys, end - k0);
                double sown[4];
                qk_tile_clamped<4>(Kp + (size_t)k0 * kRowBytes, n_valid, qd, lane, sown);
                const int pos_own = k0 + key_own + 1;                       // 1-based position of this lane's key
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const bool on = key_own < n_valid && pos_own <= qpos[x];   // causal row: keys 1..position of the query
                    const double s = on ? sown[x] * inv_root_d : -INFINITY;
                    const double mn = fmax(m[x], s);
                    Z[x] = fma(Z[x], exp_nonpos(m[x] - mn), exp_nonpos(s - mn));
                    m[x] = mn;
                }
            }
        }
        // fold the warp: (max, sum) pairs combine as in any split softmax
#pragma unroll
        for (int x = 0; x < 4; ++x) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double mo = __shfl_xor_sync(0xffffffffu, m[x], o), Zo = __shfl_xor_sync(0xffffffffu, Z[x], o);
                const double mn = fmax(m[x], mo);
                Z[x] = Z[x] * exp_nonpos(m[x] - mn) + Zo * exp_nonpos(mo - mn);
                m[x] = mn;
            }
            if (lane == 0) { mz_sm[((size_t)warp * rows_pad + 4 * gi + x) * 2] = m[x]; mz_sm[((size_t)warp * rows_pad + 4 * gi + x) * 2 + 1] = Z[x]; }
        }
    }
    __syncthreads();
    double* part = reinterpret_cast<double*>(fp.partials) + ((size_t)u * fp.n_splits + split) * rows_pad * 2;
    for (int r = tid; r < rows_pad; r += kPromptFastThreads) {
        double mb = -1e300, Zb = 0.0;
        for (int x = 0; x < NW; ++x) mb = fmax(mb, mz_sm[((size_t)x * rows_pad + r) * 2]);
        for (int x = 0; x < NW; ++x) Zb += mz_sm[((size_t)x * rows_pad + r) * 2 + 1] * exp_nonpos(mz_sm[((size_t)x * rows_pad + r) * 2] - mb);
        part[2 * r] = mb; part[2 * r + 1] = Zb;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned prev = atomicAdd(fp.ticket + u, 1u);
        s_last = (prev == (unsigned)(n_act - 1));
        if (s_last) fp.ticket[u] = 0u;
        __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    // thresholds of Definition 3.1 in log form: s >= lse + ln(alpha) - ln(position of the query)
    double* thr = reinterpret_cast<double*>(fp.partials) + (size_t)p.U * fp.n_splits * rows_pad * 2 + (size_t)u * rows_pad;
    for (int r = tid; r < rows_pad; r += kPromptFastThreads) {
        const int rho = slot0 + r / G;
        const bool exists = r < rows && rho >= w - wp;
        double mb = -1e300, Zb = 0.0;
        const double* pu = reinterpret_cast<const double*>(fp.partials) + (size_t)u * fp.n_splits * rows_pad * 2;
        for (int s = 0; s < n_act; ++s) mb = fmax(mb, __ldcg(pu + ((size_t)s * rows_pad + r) * 2));
        for (int s = 0; s < n_act; ++s)
            Zb += __ldcg(pu + ((size_t)s * rows_pad + r) * 2 + 1) * exp(__ldcg(pu + ((size_t)s * rows_pad + r) * 2) - mb);
        thr[r] = exists ? mb + log(Zb) + p.log_alpha - log((double)(P - (w - 1 - rho))) : INFINITY;
    }
}

template <int G>
__global__ void __launch_bounds__(kPromptFastThreads) prompt_verdict_kernel(const __grid_constant__ PromptFastParams fp) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_last;
    __shared__ int s_scan[kPromptFastThreads];
    const PromptParams& p = fp.p;
    constexpr int NW = kPromptFastWarps, NT = kPromptFastThreads;
    const int u = blockIdx.y, split = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = u / p.Hkv, P = __ldg(p.prompt_lens + b), w = p.w, wp = min(P, w);
    const bool last_launch = fp.slot1 == w;
    if (P > p.C) {
        if (last_launch && split == 0 && tid == 0) { report_status(p.status, CORM_ERR_CAPACITY); p.live_out[u] = 0; }
        return;
    }
    if (P == 0) {
        if (last_launch && split == 0 && tid == 0) {
            p.live_out[u] = 0; publish_live(p.maxlive, 0, 0);
            if (p.page_table) {  // an empty unit still owns the page its first append goes to
                const int pg = claim_page(p.page_bits, p.pool_pages, p.U, u, 0);
                p.page_table[(size_t)u * p.pt_stride] = pg + 1;
                p.page_room[u] = pg >= 0;
            }
        }
        return;
    }
    const int rows = fp.rows, rows_pad = (rows + 3) / 4 * 4, groups = rows_pad / 4, slot0 = fp.slot0;
    const int begin = split * fp.split_len, end = min(P, begin + fp.split_len);
    const int n_act = (P + fp.split_len - 1) / fp.split_len;
    if (split >= n_act) return;
    uint16_t* q_sm = reinterpret_cast<uint16_t*>(smem);
    double* thr_sm = reinterpret_cast<double*>(smem + (size_t)rows_pad * 256 + (size_t)NW * rows_pad * 16);
    double* err_sm = thr_sm + rows_pad;                          // kDotErr |q_r| / sqrt(d): times |k_j| it bounds a logit's error
    uint32_t* keepmask = reinterpret_cast<uint32_t*>(err_sm + rows_pad);
    int* prefix = reinterpret_cast<int*>(keepmask + (p.C + 31) / 32 + 2);
    int32_t* pt_sm = prefix + (p.C + 31) / 32 + 2;               // paged caches: the unit's page entries for the gather
    stage_q_rows(p, u, G, slot0, rows, rows_pad, q_sm);
    const double* thr = reinterpret_cast<const double*>(fp.partials) + (size_t)p.U * fp.n_splits * rows_pad * 2 + (size_t)u * rows_pad;
    for (int r = tid; r < rows_pad; r += NT) thr_sm[r] = __ldcg(thr + r);
    __syncthreads();
    for (int r = tid; r < rows_pad; r += NT) {
        double n2 = 0.0;
        for (int c = 0; c < 128; ++c) {
            const double x = (double)__uint_as_float((uint32_t)q_sm[(size_t)r * 128 + c] << 16);
            n2 = fma(x, x, n2);
        }
        err_sm[r] = p.bound_scale * kDotErr * inv_root_dim(128) * sqrt(n2) * (1.0 + 1e-6);
    }
    __syncthreads();
    const unsigned char* Kp = reinterpret_cast<const unsigned char*>(p.k_prompt) + (size_t)u * p.p_max * kRowBytes;
    const unsigned char* Vp = reinterpret_cast<const unsigned char*>(p.v_prompt) + (size_t)u * p.p_max * kRowBytes;
    uint32_t* tmp_word = reinterpret_cast<uint32_t*>(p.stash) + (size_t)u * p.C;     // scratch registers of this unit
    const int h = lane >> 4, ci = lane & 15, key_own = 16 * h + 8 * (ci & 1) + (ci >> 1);
    const double inv_root_d = 0.088388347648318440550;
    const int n_tiles = (end - begin + kTileKeys - 1) / kTileKeys;
    for (int tix = warp; tix < n_tiles; tix += NW) {
        const int k0 = begin + tix * kTileKeys, n_valid = min(kTileKeys, end - k0);
        const int pos_own = k0 + key_own + 1;
        // verdicts of this launch's queries for the lane's key: a bit per window slot (bit w-1-rho) when the window
        // fits a shift register, else the position of the newest query that found the key important
        uint32_t reg = 0u;
        for (int gi = 0; gi < groups; ++gi) {
            if (slot0 + (4 * gi + 3) / G < w - wp) continue;                      // none of these queries exists
            // The thresholds are exact (fp64, from the first launch), so a logit only has to be placed on one side of
            // its threshold: an fp32 dot product does that whenever it is farther from it than the proven bound on
            // its own accumulation error; the rare logit inside the bound is formed again exactly.
            float qf[4][8], s32[4], kn2;
            load_row_group32(q_sm, gi, ci, qf);
            qk_tile_clamped32<4>(Kp + (size_t)k0 * kRowBytes, n_valid, qf, lane, s32, kn2);
            const double kn = sqrt((double)kn2) * (1.0 + 1e-6);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int r = 4 * gi + x, rho = slot0 + r / G;
                const bool exists = r < rows && rho >= w - wp;
                const int qpos = P - (w - 1 - rho);
                bool imp = false;
                if (exists && pos_own <= qpos) {
                    const double margin = (double)s32[x] * inv_root_d - thr_sm[r], err = err_sm[r] * kn;
                    if (margin >= err) imp = true;
                    else if (!(margin < -err)) {
                        imp = exact_logit(q_sm + (size_t)r * 128, Kp + (size_t)(k0 + key_own) * kRowBytes) * inv_root_d >= thr_sm[r];
                        atomicAdd(p.counters + CNT_NEAR, 1ull);      // rare: a few hundred per pass
                    }
                }
                // Definition 3.1 in log form; keys newer than the query keep a 0 bit (Algorithm 1's zero padding)
                if (imp) {
                    if (w <= 32) reg |= 1u << (w - 1 - rho);
                    else reg = max(reg, (uint32_t)qpos);
                }
            }
        }
        if (key_own < n_valid) {
            uint32_t* dst = tmp_word + k0 + key_own;
            if (slot0 == 0) *dst = reg;                                            // first launch of the window
            else *dst = w <= 32 ? (*dst | reg) : max(*dst, reg);                   // same lane wrote it last time
        }
    }
    if (!last_launch) return;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned prev = atomicAdd(fp.ticket + u, 1u);
        s_last = (prev == (unsigned)(n_act - 1));
        if (s_last) fp.ticket[u] = 0u;
        __threadfence();
    }
    __syncthreads();
    if (!s_last) return;

    // last arriver: Algorithm 1's keep rule over the whole prompt, then an ordered gather into the slab
    const bool evict_on = wp >= w;
    for (int base = 0; base < P; base += NT) {
        const int j = base + tid;
        bool keep = false;
        if (j < P) keep = !evict_on || register_needed(__ldcg(tmp_word + j), w, P) || (j + 1) > P - p.r;
        const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
        if (lane == 0 && base + warp * 32 < P) keepmask[(base >> 5) + warp] = ballot;
    }
    __syncthreads();
    const int nwords = (P + 31) / 32;
    block_popc_scan<NT>(keepmask, prefix, nwords, s_scan);
    const int kept_total = prefix[nwords];
    const bool paged = p.page_table != nullptr;
    if (!claim_unit_pages<NT>(p.page_table, p.page_bits, p.page_room, p.pool_pages, p.pt_stride, p.U, u, kept_total, pt_sm)) {
        if (tid == 0) { report_status(p.status, CORM_ERR_CAPACITY); p.live_out[u] = 0; publish_live(p.maxlive, 0, 0); }
        return;                                                                       // the pool is too small
    }
    unsigned char* Kl = reinterpret_cast<unsigned char*>(p.K);
    unsigned char* Vl = reinterpret_cast<unsigned char*>(p.V);
    uint32_t* wordu = p.word + (size_t)u * p.C;
    int32_t* posu = p.pos + (size_t)u * p.C;
    // a warp takes 8 consecutive prompt rows at a time; lanes 0-15 copy the K row, 16-31 the V row; loads first
    for (int j0 = warp * 8; j0 < P; j0 += NW * 8) {
        uint4 buf[8];
        int dst[8];
        size_t drow[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const int j = j0 + x;
            const bool kept = j < P && ((keepmask[j >> 5] >> (j & 31)) & 1u);
            dst[x] = kept ? kept_before(keepmask, prefix, j) : -1;
            drow[x] = !kept ? 0 : paged ? page_row(pt_sm[dst[x] >> 5], dst[x], p.pool_pages, p.status) : (size_t)u * p.C + dst[x];
            if (kept) buf[x] = __ldg(reinterpret_cast<const uint4*>((lane < 16 ? Kp : Vp) + (size_t)j * kRowBytes) + (lane & 15));
        }
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            if (dst[x] < 0) continue;
            reinterpret_cast<uint4*>((lane < 16 ? Kl : Vl) + drow[x] * kRowBytes)[lane & 15] = buf[x];
            if (lane == 0) { wordu[dst[x]] = __ldcg(tmp_word + j0 + x); posu[dst[x]] = j0 + x + 1; }
        }
    }
    if (tid == 0) {
        p.live_out[u] = kept_total;
        publish_live(p.maxlive, 0, kept_total);
        atomicAdd(p.counters + CNT_APPENDED, (unsigned long long)P);
        if (kept_total < P) atomicAdd(p.counters + CNT_EVICTED, (unsigned long long)(P - kept_total));
    }
}

// Host side. Returns CORM_ERR_UNSUPPORTED when the configuration does not fit (the caller then uses the generic pass).
inline corm_status_t launch_prompt_fast(PromptFastParams& fp, int G, int max_p, int sm_count, size_t partial_capacity,
                                        cudaStream_t st) {
    const PromptParams& p = fp.p;
    const int chunk_slots = 64 / G < p.w ? 64 / G : p.w;                 // at most 64 (slot, head) rows per launch pair
    const int rows_pad = (chunk_slots * G + 3) / 4 * 4;
    // about four blocks per SM in flight, splits of whole tiles, at least 512 keys
    long long want_blocks = 4ll * (sm_count > 0 ? sm_count : 148);
    long long per_unit = (want_blocks + p.U - 1) / p.U;
    int split_len = (int)((max_p + per_unit - 1) / per_unit);
    if (split_len < 512) split_len = 512;
    split_len = (split_len + kTileKeys - 1) / kTileKeys * kTileKeys;
    fp.split_len = split_len;
    fp.n_splits = max_p > 0 ? (max_p + split_len - 1) / split_len : 1;
    const size_t need = ((size_t)p.U * fp.n_splits * rows_pad * 2 + (size_t)p.U * rows_pad) * 8;
    const size_t smem = prompt_fast_smem(rows_pad, p.C, p.page_table != nullptr);
    if (need > partial_capacity || smem > 200 * 1024 || p.U > 65535) return CORM_ERR_UNSUPPORTED;
    auto run = [&](auto k1, auto k2) -> corm_status_t {
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(k1), smem);
        if (e == cudaSuccess) e = ensure_dynamic_smem(reinterpret_cast<const void*>(k2), smem);
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: cudaFuncSetAttribute: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        const dim3 grid(fp.n_splits, (unsigned)p.U);
        for (int s0 = 0; s0 < p.w; s0 += chunk_slots) {                  // oldest window slots first
            fp.slot0 = s0;
            fp.slot1 = s0 + chunk_slots < p.w ? s0 + chunk_slots : p.w;
            fp.rows = (fp.slot1 - fp.slot0) * G;
            k1<<<grid, kPromptFastThreads, smem, st>>>(fp);
            k2<<<grid, kPromptFastThreads, smem, st>>>(fp);
        }
        e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: prompt launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    switch (G) {
        case 1: return run(prompt_lse_kernel<1>, prompt_verdict_kernel<1>);
        case 2: return run(prompt_lse_kernel<2>, prompt_verdict_kernel<2>);
        case 4: return run(prompt_lse_kernel<4>, prompt_verdict_kernel<4>);
        case 8: return run(prompt_lse_kernel<8>, prompt_verdict_kernel<8>);
    }
    return CORM_ERR_UNSUPPORTED;
}

// number of kernel launches launch_prompt_fast issues for this window and group size
inline int prompt_fast_launches(int G, int w) {
    const int chunk_slots = 64 / G < w ? 64 / G : w;
    return 2 * ((w + chunk_slots - 1) / chunk_slots);
}

}  // namespace corm
