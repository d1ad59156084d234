// Exact redo of a decode step's verdicts for the units whose certified fp32 logits left some key undecided (third
// launch of such a step; blocks of every other unit leave at once). The outputs of the step exist already. Here the
// unit's logits are formed again in fp64, exactly as the fp64 kernels form them, each split publishes its (m, Z),
// and the split that arrives last corrects the newest verdict of every register, decides what is kept and compacts
// the unit (finalize_unit in its patch form).
#pragma once

#include "corm_fast.cuh"

namespace corm {

__host__ __device__ inline size_t redo_smem(int G, int C) {
    size_t tiles = (size_t)kFastWarps * kTileBytes, lists = (size_t)2 * ((C + 31) / 32 + 2) * 4;
    return (tiles > lists ? tiles : lists) + (size_t)G * 128 * 8 + kFastWarps * G * 16 + kFastWarps * 8 + 128;
}

template <int G>
__global__ void __launch_bounds__(kFastThreads) decode_redo_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_last;
    __shared__ int s_failed;
    constexpr int NT = kFastThreads, NW = kFastWarps;
    const int u = blockIdx.y, split = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = u / p.Hkv;
    asm volatile("griddepcontrol.wait;" ::: "memory");                     // the verdict grid has completed
    if (__ldcg(p.redo_flag + u) == 0) return;
    const int l_old = __ldcg(p.live_in + u), l = l_old + 1;
    if (l > p.C) return;
    const int n_act = (l + p.split_len - 1) / p.split_len;
    if (split >= n_act) return;
    if (__ldcg(p.status) == (int)CORM_ERR_TIMEOUT) return;
    const int t = __ldg(p.base_tokens + b) + p.step + 1;
    const int begin = split * p.split_len, end = min(l, begin + p.split_len);
    const int n_tiles = (end - begin + kTileKeys - 1) / kTileKeys;
    const size_t lists = (size_t)2 * ((p.C + 31) / 32 + 2) * 4;
    const size_t area = ((size_t)NW * kTileBytes > lists ? (size_t)NW * kTileBytes : lists);
    unsigned char* my_tile = smem + warp * kTileBytes;
    double* qs = reinterpret_cast<double*>(smem + ((area + 127) & ~(size_t)127));
    double* mz = qs + G * 128;                                             // [NW][G][2]
    const uint32_t my_bar = smem_addr(mz + NW * G * 2) + warp * 8;
    const unsigned char* Ku = reinterpret_cast<const unsigned char*>(p.K) + (size_t)u * p.C * kRowBytes;

    if (tid == 0) s_failed = 0;
    if (lane == 0) { mbar_init(my_bar, 1); fence_mbar_init(); fence_async_smem(); }
    __syncthreads();
    const int my_n = (n_tiles > warp) ? (n_tiles - warp + NW - 1) / NW : 0;
    auto issue_k = [&](int it) {
        const int k0 = begin + (warp + it * NW) * kTileKeys;
        const uint32_t bytes = (uint32_t)min(kTileKeys, end - k0) * kRowBytes;
        mbar_expect_tx(my_bar, bytes);
        bulk_load(smem_addr(my_tile), Ku + (size_t)k0 * kRowBytes, bytes, my_bar);
    };
    if (lane == 0 && my_n > 0) issue_k(0);
    {
        const bf16_t* qg = reinterpret_cast<const bf16_t*>(p.q) + (size_t)u * G * 128;
        for (int x = tid; x < G * 128; x += NT) qs[x] = (double)Elem<bf16_t>::load(qg + x);
    }
    __syncthreads();
    const int h = lane >> 4, ci = lane & 15, key_own = 16 * h + 8 * (ci & 1) + (ci >> 1);
    double qd[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < 8; ++e) qd[g][e] = qs[g * 128 + ci * 8 + e];
    double M[G], Zl[G];
#pragma unroll
    for (int g = 0; g < G; ++g) { M[g] = -INFINITY; Zl[g] = 0.0; }
    constexpr double inv_root_d = inv_root_dim(128);
    bool failed = false;
    for (int it = 0; it < my_n; ++it) {
        const int k0 = begin + (warp + it * NW) * kTileKeys, n_valid = min(kTileKeys, end - k0);
        if (!mbar_wait(my_bar, it & 1)) failed = true;
        double sown[G];
        qk_tile<G>(my_tile, qd, lane, sown);
        __syncwarp();
        if (lane == 0 && it + 1 < my_n) { fence_async_smem(); issue_k(it + 1); }
        const bool valid = key_own < n_valid;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const double sv = valid ? sown[g] * inv_root_d : -INFINITY;    // Eq. 2's exponent
            float mt = (float)sv;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, o));
            const double Mn = fmax(M[g], (double)mt);
            Zl[g] = fma(Zl[g], exp_nonpos(M[g] - Mn), valid ? exp_nonpos(sv - Mn) : 0.0);
            M[g] = Mn;
            if (valid) p.stash[((size_t)u * G + g) * p.C + k0 + key_own] = sv;
        }
    }
    if (failed) { atomicCAS(p.status, 0, (int)CORM_ERR_TIMEOUT); s_failed = 1; }
#pragma unroll
    for (int g = 0; g < G; ++g) {
        Zl[g] = warp_sum(Zl[g]);
        if (lane == 0) { mz[(warp * G + g) * 2] = M[g]; mz[(warp * G + g) * 2 + 1] = Zl[g]; }
    }
    __syncthreads();
    if (s_failed) return;                                                  // reported through the status word
    if (tid < G) {
        const int g = tid;
        double Mb = -INFINITY, Zb = 0.0;
        for (int w = 0; w < NW; ++w) Mb = fmax(Mb, mz[(w * G + g) * 2]);
        for (int w = 0; w < NW; ++w) Zb += mz[(w * G + g) * 2 + 1] * exp_nonpos(mz[(w * G + g) * 2] - Mb);
        double* rec = reinterpret_cast<double*>(p.partials + (((size_t)u * p.max_splits + split) * G + g) * partial_stride(128));
        rec[0] = Mb; rec[1] = Zb;
    }
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
    finalize_unit<bf16_t, 128, G, NT, true>(p, u, b, l, n_act, t, smem);
    if (tid == 0) { p.redo_flag[u] = 0; atomicAdd(p.counters + CNT_REDONE, 1ull); }
}

// Launched after the verdict launch of every step whose logits are fp32; programmatic-dependent on it.
inline corm_status_t launch_redo(DecodeParams& p, int G, int n_splits, cudaStream_t st, int* n_launched) {
    const size_t smem = redo_smem(G, p.C);
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
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, p);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { std::fprintf(stderr, "corm: redo launch: %s\n", cudaGetErrorString(e)); return CORM_ERR_CUDA; }
        return CORM_OK;
    };
    corm_status_t rc = G == 2 ? launch(decode_redo_kernel<2>) : G == 4 ? launch(decode_redo_kernel<4>) : CORM_ERR_UNSUPPORTED;
    if (rc == CORM_OK) *n_launched += 1;
    return rc;
}

}  // namespace corm
