// Host side of the C-ABI library: arena layout, argument checks, launch configuration. Every step of the hot
// path runs in the kernels of corm_fast.cuh / corm_balanced.cuh / corm_verdict.cuh / corm_prompt_fast.cuh /
// corm_generic.cuh; nothing
// here touches tensor data on the CPU.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cmath>
#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <type_traits>
#include <vector>

#include "../../include/corm.h"
#include "corm_common.cuh"
#include "corm_fast.cuh"
#include "corm_balanced.cuh"
#include "corm_generic.cuh"
#include "corm_prompt_fast.cuh"

using namespace corm;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMinSplit = 64;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
    size_t K, V, word, pos, live, base_tokens, base_obs, ticket, ticket2, ticket3, move_info, unit_stamp, counters, status, maxlive, sim_acc, page_table, page_bits, page_room, q_prev, stash, partials, keepmask, unit_rec;
    size_t stage_q, stage_k, stage_v, stage_out, total, bookkeeping_begin, bookkeeping_end;
};

bool config_ok(const corm_config_t* c, corm_status_t* why) {
    *why = CORM_ERR_INVALID_ARG;
    if (!c) return false;
    if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1) return false;
    if (c->n_q_heads % c->n_kv_heads) return false;
    if (c->max_tokens < 1 || c->window_w < 1 || c->recent_r < 1) return false;
    if (!(c->alpha >= 0.f) || !std::isfinite(c->alpha)) return false;
    if (c->kv_dtype != CORM_F32 && c->kv_dtype != CORM_BF16) return false;
    if (c->device < 0) return false;
    *why = CORM_ERR_UNSUPPORTED;
    const int G = c->n_q_heads / c->n_kv_heads;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (G != 1 && G != 2 && G != 4 && G != 8) return false;
    if (c->window_w > 256) return false;
    if ((long long)c->batch * c->n_kv_heads > 65535) return false;     // grid.y of the decode kernel
    if (c->max_tokens > (1 << 19)) return false;                        // the keep mask of a unit must fit shared memory
    *why = CORM_OK;
    return true;
}

int max_splits_of(const corm_config_t& c) { return (c.max_tokens + kMinSplit - 1) / kMinSplit; }

// Split partial records the arena holds: one per (unit, split) of the block-per-split kernels, and enough for the
// balanced kernel's one record per (block, unit) pair of its tile list at up to kMaxBalancedBlocks blocks.
constexpr int kMaxBalancedBlocks = 1024;
// layers whose units one launch may cover: all of a slab cache's layers if their units fit a grid dimension, else one
size_t fused_layers_of(const corm_config_t& c, int pool_pages) {
    const long long U = (long long)c.batch * c.n_kv_heads;
    return (pool_pages == 0 && c.n_layers > 1 && U * c.n_layers <= 65535) ? (size_t)c.n_layers : 1;
}
size_t partial_records_of(const corm_config_t& c, int pool_pages) {
    const size_t U = (size_t)c.batch * c.n_kv_heads * fused_layers_of(c, pool_pages);
    return std::max(U * (size_t)max_splits_of(c), bal_record_count(kMaxBalancedBlocks, (int)U));
}

int pt_stride_of(const corm_config_t& c) { return (c.max_tokens + kPageKeys - 1) / kPageKeys; }

// pool_pages = 0: one slab of max_tokens rows per unit; > 0: that many 32-key pages of K and of V per layer
bool pool_ok(const corm_config_t& c, int pool_pages) {
    if (pool_pages == 0) return true;
    const long long U = (long long)c.batch * c.n_kv_heads;
    return pool_pages > 0 && pool_pages % 32 == 0 && pool_pages >= U;     // every unit always owns at least one page
}

Layout make_layout(const corm_config_t& c, int pool_pages) {
    Layout L{};
    const size_t U = (size_t)c.batch * c.n_kv_heads, Ltot = c.n_layers, C = c.max_tokens, D = c.head_dim;
    const size_t e = c.kv_dtype == CORM_BF16 ? 2 : 4, G = c.n_q_heads / c.n_kv_heads;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes); return at; };
    const size_t kv_rows = pool_pages ? (size_t)pool_pages * kPageKeys : U * C;   // rows of K (and of V) per layer
    L.K = take(Ltot * kv_rows * D * e);
    L.V = take(Ltot * kv_rows * D * e);
    L.word = take(Ltot * U * C * 4);
    L.pos = take(Ltot * U * C * 4);
    L.bookkeeping_begin = off;
    L.live = take(Ltot * 2 * U * 4);
    L.base_tokens = take(Ltot * c.batch * 4);
    L.base_obs = take(Ltot * c.batch * 4);
    L.ticket = take(Ltot * U * 4);
    L.ticket2 = take(Ltot * U * 4);
    L.ticket3 = take(Ltot * U * 4);
    L.move_info = take(Ltot * U * 8);
    L.unit_stamp = take(Ltot * U * 8);
    L.counters = take(Ltot * CNT_COUNT * 8);
    L.status = take(4);
    L.maxlive = take(Ltot * 8);
    L.sim_acc = take(16);
    L.page_table = take(pool_pages ? Ltot * U * pt_stride_of(c) * 4 : 0);
    L.page_bits = take(pool_pages ? Ltot * (size_t)(pool_pages / 32) * 4 : 0);
    L.page_room = take(pool_pages ? Ltot * U * 4 : 0);
    L.bookkeeping_end = off;
    L.q_prev = take(Ltot * (size_t)c.batch * c.n_q_heads * D * e);
    // scratch of one launch; a launch covers one layer's units, or all layers' units when corm_decode_step_layers
    // steps them together (slab caches): 8 G bytes per slot against the 2 D e bytes of its K and V rows
    const size_t Us = U * fused_layers_of(c, pool_pages);
    L.stash = take(Us * G * C * 8);
    L.partials = take(partial_records_of(c, pool_pages) * G * partial_stride((int)D));
    L.keepmask = take(Us * (size_t)keepmask_words((int)C) * 4);
    L.unit_rec = take(Us * 8);
    L.stage_q = take((size_t)c.batch * c.n_q_heads * D * e);
    L.stage_k = take(U * D * e);
    L.stage_v = take(U * D * e);
    L.stage_out = take((size_t)c.batch * c.n_q_heads * D * e);
    L.total = off;
    return L;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Named range around a boundary call, visible to profilers that collect NVTX (a no-op without one).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

#define CORM_CUDA(expr)                                                         \
    do {                                                                        \
        cudaError_t e_ = (expr);                                                \
        if (e_ != cudaSuccess) {                                                \
            std::fprintf(stderr, "corm: %s failed: %s\n", #expr, cudaGetErrorString(e_)); \
            return CORM_ERR_CUDA;                                               \
        }                                                                       \
    } while (0)

}  // namespace

struct corm_cache {
    corm_config_t cfg;
    Layout lay;
    unsigned char* arena;
    int U, G;
    size_t e;
    std::vector<int> parity, steps, ready, live_upper;
    // sizing feedback: the kernels publish the longest live length, the host reads it back without ever waiting
    unsigned long long* maxlive_host = nullptr;   // pinned, [n_layers] words followed by [n_layers][U] live lengths
    int32_t* live_host = nullptr;                 // the second part of that buffer
    std::vector<int> live_mean;                   // mean live length at the last read-back that landed (0 = unknown)
    std::vector<cudaEvent_t> readback_ev;
    std::vector<int> readback_pending, last_readback_step;
    int tune_split_len = 0, allow_fast = 1;
    double bound_scale = 1.0;
    int monitor_similarity = 0;
    std::vector<int> have_q_prev;                 // the layer's previous decode queries are stored
    int sm_count = 148;
    long long launches = 0;
    int pool_pages = 0, pt_stride = 0;            // paged cache: pages per layer, page-table entries per unit
    std::vector<CUtensorMap> vmaps;               // per layer: the V storage as a tiled tensor (balanced kernel); empty = unavailable
    CUtensorMap vmap_all;                         // the V storage of all layers of a slab cache as one tensor (layers stepped together)
    bool have_vmap_all = false;
    // per layer: the group of layers (first layer * 65536 + count) it has been stepped with ever since its prompt pass
    // (-1: not stepped yet, -2: alone or in different groups); only then does the group's length read-back describe it
    std::vector<int> step_group;
    // per layer, meaningful for the first layer of a group: bound on the longest unit of ALL the group's layers, taken
    // from a length word that a launch over the whole group wrote (INT_MAX = none yet). The first layer's own
    // live_upper may be smaller: right after the prompt pass it describes that layer alone.
    std::vector<int> group_upper;
    // per layer: its latest decode launch finished every unit inside the streaming kernel and left the units' stamps,
    // so the next step's launch may be chained to it (corm_decode_steps)
    std::vector<int> chain_ok;
    long long chained_launches = 0;
};

namespace {

template <typename F> corm_status_t dispatch(const corm_cache* c, F&& f) {
    const bool bf = c->cfg.kv_dtype == CORM_BF16;
    const int D = c->cfg.head_dim, G = c->G;
#define CORM_CASE(TT, DD, GG) if (D == DD && G == GG) return f((TT*)nullptr, std::integral_constant<int, DD>(), std::integral_constant<int, GG>());
    if (bf) {
        CORM_CASE(bf16_t, 64, 1) CORM_CASE(bf16_t, 64, 2) CORM_CASE(bf16_t, 64, 4) CORM_CASE(bf16_t, 64, 8)
        CORM_CASE(bf16_t, 128, 1) CORM_CASE(bf16_t, 128, 2) CORM_CASE(bf16_t, 128, 4) CORM_CASE(bf16_t, 128, 8)
    } else {
        CORM_CASE(float, 64, 1) CORM_CASE(float, 64, 2) CORM_CASE(float, 64, 4) CORM_CASE(float, 64, 8)
        CORM_CASE(float, 128, 1) CORM_CASE(float, 128, 2) CORM_CASE(float, 128, 4) CORM_CASE(float, 128, 8)
    }
#undef CORM_CASE
    return CORM_ERR_UNSUPPORTED;
}

unsigned char* layer_ptr(const corm_cache* c, size_t base, size_t per_layer_bytes, int layer) {
    return c->arena + base + per_layer_bytes * (size_t)layer;
}

// bytes of K (and of V) one layer holds: its units' slabs or its page pool
size_t kv_layer_bytes(const corm_cache* c) {
    const size_t rows = c->pool_pages ? (size_t)c->pool_pages * kPageKeys : (size_t)c->U * c->cfg.max_tokens;
    return rows * c->cfg.head_dim * c->e;
}

int32_t* page_table_ptr(const corm_cache* c, int layer) {
    return reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.page_table, (size_t)c->U * c->pt_stride * 4, layer));
}
uint32_t* page_bits_ptr(const corm_cache* c, int layer) {
    return reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.page_bits, (size_t)(c->pool_pages / 32) * 4, layer));
}

int32_t* page_room_ptr(const corm_cache* c, int layer) {
    return reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.page_room, (size_t)c->U * 4, layer));
}

template <typename P> void set_paging(const corm_cache* c, int layer, P& p) {
    p.page_room = c->pool_pages ? page_room_ptr(c, layer) : nullptr;
    p.page_table = c->pool_pages ? page_table_ptr(c, layer) : nullptr;
    p.page_bits = c->pool_pages ? page_bits_ptr(c, layer) : nullptr;
    p.pool_pages = c->pool_pages;
    p.pt_stride = c->pt_stride;
}

int32_t* live_buf(const corm_cache* c, int layer, int parity) {
    // [2][L][U]: the layers' buffers of one parity are contiguous, so that layers stepped together form one array
    return reinterpret_cast<int32_t*>(c->arena + c->lay.live) + ((size_t)parity * c->cfg.n_layers + layer) * c->U;
}

bool layer_ok(const corm_cache* c, int layer) { return c && layer >= 0 && layer < c->cfg.n_layers; }

double log_alpha_of(const corm_cache* c) { return c->cfg.alpha > 0.f ? std::log((double)c->cfg.alpha) : -INFINITY; }

unsigned long long* maxlive_ptr(const corm_cache* c, int layer) {
    return reinterpret_cast<unsigned long long*>(c->arena + c->lay.maxlive) + layer;
}

// If an earlier read-back has landed, tighten the bound on this layer's longest unit: a unit grows by at most one
// key per step, so (length after step s) + (steps since s) bounds every unit now.
// A host that enqueues steps much faster than the GPU runs them would otherwise size its launches from a bound that
// is hundreds of steps stale (every step adds one key to it): once it is kMaxRunAhead steps past a read-back that
// has not landed it waits for that one, which leaves the GPU that many steps of queued work and costs it nothing.
constexpr int kMaxRunAhead = 24;
void poll_live_bound(corm_cache* c, int layer) {
    if (!c->readback_pending[layer]) return;
    if (c->steps[layer] - c->last_readback_step[layer] >= kMaxRunAhead) {
        if (cudaEventSynchronize(c->readback_ev[layer]) != cudaSuccess) return;
    } else if (cudaEventQuery(c->readback_ev[layer]) != cudaSuccess) {
        (void)cudaGetLastError();   // cudaErrorNotReady is not an error
        return;
    }
    c->readback_pending[layer] = 0;
    const unsigned long long v = c->maxlive_host[layer];
    const int steps_done = (int)(v >> 32), len = (int)(v & 0xffffffffu);
    if (steps_done > c->steps[layer]) return;   // stale word from before a reset / new prompt
    const int bound = len + (c->steps[layer] - steps_done);
    if (bound < c->live_upper[layer]) c->live_upper[layer] = bound;
    // a word written by a decode launch over the layer's group covers every layer of the group
    if (steps_done >= 1 && c->step_group[layer] >= 0 && bound < c->group_upper[layer]) c->group_upper[layer] = bound;
    long long sum = 0;                            // the lengths themselves came with the same read-back
    for (int u = 0; u < c->U; ++u) sum += c->live_host[(size_t)layer * c->U + u];
    c->live_mean[layer] = (int)(sum / c->U);
}

void schedule_live_readback(corm_cache* c, int layer, cudaStream_t st) {
    if (c->readback_pending[layer] || !c->maxlive_host) return;
    if (cudaMemcpyAsync(c->maxlive_host + layer, maxlive_ptr(c, layer), 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return;
    if (cudaMemcpyAsync(c->live_host + (size_t)layer * c->U, live_buf(c, layer, c->parity[layer]), (size_t)c->U * 4,
                        cudaMemcpyDeviceToHost, st) != cudaSuccess) return;
    if (cudaEventRecord(c->readback_ev[layer], st) != cudaSuccess) return;
    c->readback_pending[layer] = 1;
    c->last_readback_step[layer] = c->steps[layer];
}

// Eq. 3 between this step's queries and the layer's previous decode queries (opt-in; one small launch), after any
// of the decode entry points: the queries stored as "previous" are always those of the step before.
corm_status_t monitor_similarity(corm_cache* c, int layer, const void* q, cudaStream_t st) {
    if (!c->monitor_similarity) return CORM_OK;
    const corm_config_t& cf = c->cfg;
    const int n_heads = cf.batch * cf.n_q_heads;
    const size_t qb = (size_t)n_heads * cf.head_dim * c->e;
    double* sum = reinterpret_cast<double*>(c->arena + c->lay.sim_acc);
    unsigned long long* cnt = reinterpret_cast<unsigned long long*>(c->arena + c->lay.sim_acc + 8);
    corm_status_t rc = dispatch(c, [&](auto* tp, auto dd, auto) -> corm_status_t {
        using T = std::remove_pointer_t<decltype(tp)>;
        constexpr int DD = decltype(dd)::value;
        query_similarity_kernel<T, DD><<<(n_heads + 3) / 4, 128, 0, st>>>(
            reinterpret_cast<const T*>(q), reinterpret_cast<T*>(layer_ptr(c, c->lay.q_prev, qb, layer)),
            c->have_q_prev[layer], n_heads, sum, cnt);
        CORM_CUDA(cudaGetLastError());
        return CORM_OK;
    });
    if (rc != CORM_OK) return rc;
    c->have_q_prev[layer] = 1;
    c->launches += 1;
    return CORM_OK;
}

// One decode step of layers [layer, layer + n_fused) as ONE launch (pair): the layers' units are consecutive in every
// per-unit array of the arena, so n_fused layers of U units are one array of n_fused * U units to the kernels. The
// caller has checked that the layers are at the same step with the same buffer parity and that q, k_new, v_new and
// out of consecutive layers are contiguous. Counters of the step go to the first layer's slots (totals are unchanged).
// chain: the caller enqueued this layer's (these layers') previous step immediately before and nothing since, and
// this step's inputs were complete before that; more: the next step follows in the same way.
corm_status_t launch_decode(corm_cache* c, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                            cudaStream_t st, int n_fused = 1, bool chain = false, bool more = false) {
    for (int i = 0; i < n_fused; ++i) poll_live_bound(c, layer + i);
    {   // A launch publishes its longest unit in its first layer's word. That bounds every layer of the group, but only
        // while that word has only ever been written by launches over this same group of layers.
        const int now = n_fused > 1 ? layer * 65536 + n_fused : -2;           // this launch's group (solo launches: none)
        bool same_group = n_fused > 1;
        for (int i = 0; i < n_fused; ++i) {
            int& g = c->step_group[layer + i];
            g = (g == -1 || g == now) ? now : -2;
            same_group &= g == now && now != -2;
        }
        if (same_group && c->group_upper[layer] != INT_MAX)
            for (int i = 0; i < n_fused; ++i) c->live_upper[layer + i] = std::min(c->live_upper[layer + i], c->group_upper[layer]);
    }
    const corm_config_t& cf = c->cfg;
    const size_t C = cf.max_tokens, D = cf.head_dim, U = c->U;
    DecodeParams p{};
    p.K = layer_ptr(c, c->lay.K, kv_layer_bytes(c), layer);
    p.V = layer_ptr(c, c->lay.V, kv_layer_bytes(c), layer);
    set_paging(c, layer, p);
    p.word = reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.word, U * C * 4, layer));
    p.pos = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.pos, U * C * 4, layer));
    p.live_in = live_buf(c, layer, c->parity[layer]);
    p.live_out = live_buf(c, layer, c->parity[layer] ^ 1);
    p.base_tokens = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.base_tokens, (size_t)cf.batch * 4, layer));
    p.base_obs = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.base_obs, (size_t)cf.batch * 4, layer));
    p.ticket = reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.ticket, U * 4, layer));
    p.ticket2 = reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.ticket2, U * 4, layer));
    p.ticket3 = reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.ticket3, U * 4, layer));
    p.move_info = reinterpret_cast<unsigned long long*>(layer_ptr(c, c->lay.move_info, U * 8, layer));
    p.counters = reinterpret_cast<unsigned long long*>(layer_ptr(c, c->lay.counters, CNT_COUNT * 8, layer));
    p.status = reinterpret_cast<int32_t*>(c->arena + c->lay.status);
    p.maxlive = maxlive_ptr(c, layer);
    p.stash = reinterpret_cast<double*>(c->arena + c->lay.stash);
    p.partials = c->arena + c->lay.partials;
    p.keepmask = reinterpret_cast<uint32_t*>(c->arena + c->lay.keepmask);
    p.unit_rec = reinterpret_cast<int2*>(c->arena + c->lay.unit_rec);
    p.unit_stamp = reinterpret_cast<unsigned long long*>(layer_ptr(c, c->lay.unit_stamp, U * 8, layer));
    p.q = q; p.k_new = k_new; p.v_new = v_new; p.out = out;
    p.U = (int)U * n_fused; p.Hkv = cf.n_kv_heads; p.C = cf.max_tokens; p.max_splits = max_splits_of(cf);
    p.step = c->steps[layer]; p.w = cf.window_w; p.r = cf.recent_r;
    p.log_alpha = log_alpha_of(c);
    int bound = 0, mean_sum = 0, mean_known = 1;
    for (int i = 0; i < n_fused; ++i) {
        bound = std::max(bound, c->live_upper[layer + i]);
        mean_known &= c->live_mean[layer + i] > 0;
        mean_sum += c->live_mean[layer + i];
    }
    const int upper = std::min(cf.max_tokens, bound + 1);   // no unit can hold more live keys

    const bool fast = c->allow_fast && cf.kv_dtype == CORM_BF16 && cf.head_dim == 128 && c->G <= 4;
    corm_status_t rc;
    int n_launched = 1;
    // Grouped query heads take the balanced streaming kernel followed by the verdict launch (measured against the
    // block-per-split kernels on one GPU, us per step: 53 against 55 in the steady state of the grouped workload, 122
    // against 136 in its first steps, 174 against 190 on 24k-key units, 157 against 177 on 8k-key units without
    // evictions); one query head per KV head stays on the block-per-split kernel, whose loop is lighter (three
    // blocks per SM). Tuning values 4 / 5 force the balanced kernel finishing in the launch / with the verdict launch.
    // Inside a call of several steps (corm_decode_steps) grouped heads take that kernel's loop with a block per split
    // and the unit finished by its last split instead, because such launches can be chained: 43 against 51 us per step
    // on 128 units of 1660 keys, 132 against 142 on 8200-key units. Not with few long units, whose finishing block
    // walks the whole unit alone (32 units of 12-24k keys: 133 against 103 us). Tuning value 6 forces it.
    const bool units = fast && !c->vmaps.empty() &&
                       (c->allow_fast == 6 || (c->allow_fast == 1 && c->G >= 2 && (chain || more) && !c->monitor_similarity &&
                                               (long long)upper <= 96ll * (long long)p.U));
    const bool balanced = !units && fast && !c->vmaps.empty() &&
                          (c->allow_fast == 4 || c->allow_fast == 5 || (c->allow_fast == 1 && c->G >= 2));
    const bool balanced_verdict = c->allow_fast != 4;
    bool chain_ok_before = chain && !c->monitor_similarity;
    for (int i = 0; i < n_fused; ++i) chain_ok_before &= c->chain_ok[layer + i] != 0;
    bool self_finishing = false;
    if (!(fast && !balanced) && !units) p.unit_stamp = nullptr;    // only the block-per-split kernels keep stamps
    if (units) {
        const int typical = mean_known ? std::min(upper, mean_sum / n_fused + c->steps[layer] - c->last_readback_step[layer] + 1) : 0;
        rc = launch_decode_balanced_units(p, n_fused > 1 ? c->vmap_all : c->vmaps[layer], c->G, upper, typical, c->tune_split_len,
                                          c->sm_count, partial_records_of(cf, c->pool_pages), st, &n_launched,
                                          chain_ok_before, more && !c->monitor_similarity);
        self_finishing = rc == CORM_OK;
        if (rc == CORM_OK && p.chain_wait) c->chained_launches += 1;
    } else if (balanced) {
        rc = launch_decode_balanced(p, n_fused > 1 ? c->vmap_all : c->vmaps[layer], c->G, upper, c->sm_count, partial_records_of(cf, c->pool_pages), balanced_verdict, st, &n_launched);
    } else if (fast) {
        // the mean grows by at most one key per step, like the bound
        const int typical = mean_known ? std::min(upper, mean_sum / n_fused + c->steps[layer] - c->last_readback_step[layer] + 1) : 0;
        rc = launch_decode_fast(p, c->G, upper, typical, c->tune_split_len, c->sm_count, st, &n_launched, c->allow_fast,
                                chain_ok_before, more && !c->monitor_similarity, &self_finishing);
        if (rc == CORM_OK && p.chain_wait) c->chained_launches += 1;
    } else {
        p.split_len = c->tune_split_len ? c->tune_split_len : 256;
        const int n_splits = (upper + p.split_len - 1) / p.split_len;
        rc = dispatch(c, [&](auto* tp, auto dd, auto gg) -> corm_status_t {
            using T = std::remove_pointer_t<decltype(tp)>;
            constexpr int DD = decltype(dd)::value, GG = decltype(gg)::value;
            const size_t smem = generic_decode_smem(DD, GG, cf.max_tokens, c->pool_pages != 0);
            auto kern = decode_generic_kernel<T, DD, GG>;
            CORM_CUDA(ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem));
            kern<<<dim3(n_splits, (unsigned)p.U), kGenericThreads, smem, st>>>(p);
            CORM_CUDA(cudaGetLastError());
            return CORM_OK;
        });
    }
    if (rc != CORM_OK) return rc;
    c->launches += n_launched;
    for (int i = 0; i < n_fused; ++i) {
        const int l = layer + i;
        c->chain_ok[l] = self_finishing ? 1 : 0;
        c->parity[l] ^= 1;
        c->steps[l] += 1;
        c->live_upper[l] = std::min(cf.max_tokens, c->live_upper[l] + 1);
        if (c->group_upper[l] != INT_MAX) c->group_upper[l] += 1;
        if (c->steps[l] - c->last_readback_step[l] >= 8) schedule_live_readback(c, l, st);
    }
    return n_fused == 1 ? monitor_similarity(c, layer, q, st) : CORM_OK;
}

}  // namespace

extern "C" {

size_t corm_cache_arena_bytes(const corm_config_t* cfg) { return corm_cache_arena_bytes_paged(cfg, 0); }

size_t corm_cache_arena_bytes_paged(const corm_config_t* cfg, int32_t pool_pages) {
    corm_status_t why;
    if (!config_ok(cfg, &why) || !pool_ok(*cfg, pool_pages)) return 0;
    return make_layout(*cfg, pool_pages).total;
}

corm_status_t corm_cache_create(const corm_config_t* cfg, void* arena_device, size_t arena_bytes, corm_cache_t** out) {
    return corm_cache_create_paged(cfg, 0, arena_device, arena_bytes, out);
}

corm_status_t corm_cache_create_paged(const corm_config_t* cfg, int32_t pool_pages, void* arena_device, size_t arena_bytes,
                                      corm_cache_t** out) {
    corm_status_t why;
    if (!out) return CORM_ERR_INVALID_ARG;
    *out = nullptr;
    if (!config_ok(cfg, &why)) return why;
    if (!pool_ok(*cfg, pool_pages)) return CORM_ERR_INVALID_ARG;
    if (!arena_device || (reinterpret_cast<uintptr_t>(arena_device) % kAlign)) return CORM_ERR_INVALID_ARG;
    Layout lay = make_layout(*cfg, pool_pages);
    if (arena_bytes < lay.total) return CORM_ERR_ARENA_TOO_SMALL;
    DeviceGuard guard(cfg->device);
    if (!guard.ok) return CORM_ERR_CUDA;
    corm_cache* c = new (std::nothrow) corm_cache();
    if (!c) return CORM_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->lay = lay;
    c->arena = static_cast<unsigned char*>(arena_device);
    c->U = cfg->batch * cfg->n_kv_heads;
    c->G = cfg->n_q_heads / cfg->n_kv_heads;
    c->e = cfg->kv_dtype == CORM_BF16 ? 2 : 4;
    c->pool_pages = pool_pages;
    c->pt_stride = pool_pages ? pt_stride_of(*cfg) : 0;
    c->parity.assign(cfg->n_layers, 0);
    c->steps.assign(cfg->n_layers, 0);
    c->ready.assign(cfg->n_layers, 0);
    c->live_upper.assign(cfg->n_layers, 0);
    c->live_mean.assign(cfg->n_layers, 0);
    c->have_q_prev.assign(cfg->n_layers, 0);
    c->step_group.assign(cfg->n_layers, -1);
    c->group_upper.assign(cfg->n_layers, INT_MAX);
    c->chain_ok.assign(cfg->n_layers, 0);
    c->readback_pending.assign(cfg->n_layers, 0);
    c->last_readback_step.assign(cfg->n_layers, 0);
    c->readback_ev.assign(cfg->n_layers, nullptr);
    bool host_ok = cudaHostAlloc(reinterpret_cast<void**>(&c->maxlive_host),
                                 sizeof(unsigned long long) * cfg->n_layers + sizeof(int32_t) * (size_t)cfg->n_layers * c->U,
                                 cudaHostAllocDefault) == cudaSuccess;   // pinned HOST memory; device memory stays the caller's
    if (host_ok) {
        c->live_host = reinterpret_cast<int32_t*>(c->maxlive_host + cfg->n_layers);
        std::memset(c->maxlive_host, 0, sizeof(unsigned long long) * cfg->n_layers + sizeof(int32_t) * (size_t)cfg->n_layers * c->U);
    }
    for (int l = 0; host_ok && l < cfg->n_layers; ++l)
        host_ok = cudaEventCreateWithFlags(&c->readback_ev[l], cudaEventDisableTiming) == cudaSuccess;
    if (!host_ok) {
        std::fprintf(stderr, "corm: could not set up the host-side read-back buffer\n");
        for (cudaEvent_t ev : c->readback_ev) if (ev) cudaEventDestroy(ev);
        if (c->maxlive_host) cudaFreeHost(c->maxlive_host);
        delete c;
        return CORM_ERR_CUDA;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess && sms > 0) c->sm_count = sms;
    if (cfg->kv_dtype == CORM_BF16 && cfg->head_dim == 128 && c->G <= 4 && cfg->max_tokens <= kBalMaxTokens) {
        const unsigned long long rows = pool_pages ? (unsigned long long)pool_pages * kPageKeys
                                                   : (unsigned long long)c->U * cfg->max_tokens;
        c->vmaps.resize(cfg->n_layers);
        for (int l = 0; l < cfg->n_layers; ++l)
            if (make_v_tensor_map(&c->vmaps[l], layer_ptr(c, lay.V, kv_layer_bytes(c), l), rows) != CORM_OK) {
                c->vmaps.clear();                 // the block-per-split kernels serve the cache instead
                break;
            }
        if (!c->vmaps.empty() && !pool_pages && cfg->n_layers > 1)
            c->have_vmap_all = make_v_tensor_map(&c->vmap_all, layer_ptr(c, lay.V, kv_layer_bytes(c), 0), rows * cfg->n_layers) == CORM_OK;
    }
    cudaError_t e = cudaMemset(c->arena + lay.bookkeeping_begin, 0, lay.bookkeeping_end - lay.bookkeeping_begin);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        std::fprintf(stderr, "corm: clearing the arena failed: %s\n", cudaGetErrorString(e));
        for (cudaEvent_t ev : c->readback_ev) if (ev) cudaEventDestroy(ev);
        cudaFreeHost(c->maxlive_host);
        delete c;
        return CORM_ERR_CUDA;
    }
    *out = c;
    return CORM_OK;
}

corm_status_t corm_cache_destroy(corm_cache_t* cache) {
    if (!cache) return CORM_ERR_INVALID_ARG;
    {
        DeviceGuard guard(cache->cfg.device);
        for (cudaEvent_t ev : cache->readback_ev) if (ev) cudaEventDestroy(ev);
        if (cache->maxlive_host) cudaFreeHost(cache->maxlive_host);
    }
    delete cache;
    return CORM_OK;
}

corm_status_t corm_cache_reset(corm_cache_t* c, void* stream) {
    if (!c) return CORM_ERR_INVALID_ARG;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    CORM_CUDA(cudaMemsetAsync(c->arena + c->lay.bookkeeping_begin, 0, c->lay.bookkeeping_end - c->lay.bookkeeping_begin,
                              static_cast<cudaStream_t>(stream)));
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        c->parity[l] = 0; c->steps[l] = 0; c->ready[l] = 0; c->live_upper[l] = 0; c->live_mean[l] = 0; c->have_q_prev[l] = 0;
        c->readback_pending[l] = 0; c->last_readback_step[l] = 0; c->step_group[l] = -1; c->chain_ok[l] = 0; c->group_upper[l] = INT_MAX;
    }
    return CORM_OK;
}

corm_status_t corm_compress_prompt(corm_cache_t* c, int32_t layer, const void* k_prompt, const void* v_prompt,
                                   const void* q_last, const int32_t* prompt_lens_host, int32_t p_max, void* stream) {
    NvtxRange nvtx_range("corm_compress_prompt");
    if (!layer_ok(c, layer) || !prompt_lens_host || p_max < 0) return CORM_ERR_INVALID_ARG;
    const corm_config_t& cf = c->cfg;
    int max_p = 0;
    std::vector<int32_t> obs(cf.batch);
    for (int b = 0; b < cf.batch; ++b) {
        const int P = prompt_lens_host[b];
        if (P < 0 || P > p_max) return CORM_ERR_INVALID_ARG;
        if (P > cf.max_tokens) return CORM_ERR_CAPACITY;
        max_p = std::max(max_p, P);
        obs[b] = std::min(P, cf.window_w);
    }
    if (max_p > 0 && (!k_prompt || !v_prompt || !q_last)) return CORM_ERR_INVALID_ARG;
    if (max_p > 0 && ((reinterpret_cast<uintptr_t>(k_prompt) | reinterpret_cast<uintptr_t>(v_prompt) |
                       reinterpret_cast<uintptr_t>(q_last)) % 16)) return CORM_ERR_INVALID_ARG;
    DeviceGuard guard(cf.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t C = cf.max_tokens, D = cf.head_dim, U = c->U;
    int32_t* base_tokens = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.base_tokens, (size_t)cf.batch * 4, layer));
    int32_t* base_obs = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.base_obs, (size_t)cf.batch * 4, layer));
    // pageable sources are staged by the runtime before these calls return
    CORM_CUDA(cudaMemcpyAsync(base_tokens, prompt_lens_host, (size_t)cf.batch * 4, cudaMemcpyHostToDevice, st));
    CORM_CUDA(cudaMemcpyAsync(base_obs, obs.data(), (size_t)cf.batch * 4, cudaMemcpyHostToDevice, st));
    CORM_CUDA(cudaMemsetAsync(layer_ptr(c, c->lay.ticket, U * 4, layer), 0, U * 4, st));
    CORM_CUDA(cudaMemsetAsync(layer_ptr(c, c->lay.ticket2, U * 4, layer), 0, U * 4, st));
    CORM_CUDA(cudaMemsetAsync(layer_ptr(c, c->lay.ticket3, U * 4, layer), 0, U * 4, st));
    CORM_CUDA(cudaMemsetAsync(layer_ptr(c, c->lay.move_info, U * 8, layer), 0, U * 8, st));
    CORM_CUDA(cudaMemsetAsync(layer_ptr(c, c->lay.unit_stamp, U * 8, layer), 0, U * 8, st));   // step counts restart
    c->chain_ok[layer] = 0;
    CORM_CUDA(cudaMemsetAsync(maxlive_ptr(c, layer), 0, 8, st));
    CORM_CUDA(cudaMemsetAsync(layer_ptr(c, c->lay.counters, CNT_COUNT * 8, layer), 0, CNT_COUNT * 8, st));   // a new prompt restarts the layer's statistics
    c->readback_pending[layer] = 0;   // an older read-back no longer describes this layer
    PromptParams p{};
    p.k_prompt = k_prompt; p.v_prompt = v_prompt; p.q_last = q_last;
    p.prompt_lens = base_tokens;
    p.K = layer_ptr(c, c->lay.K, kv_layer_bytes(c), layer);
    p.V = layer_ptr(c, c->lay.V, kv_layer_bytes(c), layer);
    set_paging(c, layer, p);
    if (c->pool_pages) {   // whatever the layer held is replaced: all its pages return to the pool
        CORM_CUDA(cudaMemsetAsync(p.page_table, 0, U * c->pt_stride * 4, st));
        CORM_CUDA(cudaMemsetAsync(p.page_bits, 0, (size_t)(c->pool_pages / 32) * 4, st));
        CORM_CUDA(cudaMemsetAsync(p.page_room, 0, U * 4, st));
    }
    p.word = reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.word, U * C * 4, layer));
    p.pos = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.pos, U * C * 4, layer));
    p.live_out = live_buf(c, layer, 0);
    p.counters = reinterpret_cast<unsigned long long*>(layer_ptr(c, c->lay.counters, CNT_COUNT * 8, layer));
    p.status = reinterpret_cast<int32_t*>(c->arena + c->lay.status);
    p.maxlive = maxlive_ptr(c, layer);
    p.stash = reinterpret_cast<double*>(c->arena + c->lay.stash);
    p.U = (int)U; p.Hkv = cf.n_kv_heads; p.C = cf.max_tokens; p.p_max = p_max; p.w = cf.window_w; p.r = cf.recent_r;
    p.log_alpha = log_alpha_of(c);
    p.bound_scale = c->bound_scale;
    corm_status_t rc = CORM_ERR_UNSUPPORTED;
    int n_launched = 1;
    if (cf.kv_dtype == CORM_BF16 && cf.head_dim == 128 && c->allow_fast) {     // two-launch tiled pass
        PromptFastParams fp{};
        fp.p = p;
        fp.partials = c->arena + c->lay.partials;
        fp.ticket = reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.ticket, U * 4, layer));
        const size_t cap = U * (size_t)max_splits_of(cf) * c->G * partial_stride((int)D);   // one layer's share is enough here
        rc = launch_prompt_fast(fp, c->G, max_p, c->sm_count, cap, st);
        n_launched = prompt_fast_launches(c->G, cf.window_w);
    }
    if (rc == CORM_ERR_UNSUPPORTED) {
        n_launched = 1;
        rc = dispatch(c, [&](auto* tp, auto dd, auto gg) -> corm_status_t {
            using T = std::remove_pointer_t<decltype(tp)>;
            constexpr int DD = decltype(dd)::value, GG = decltype(gg)::value;
            const size_t smem = prompt_smem(GG, cf.window_w, cf.max_tokens);
            auto kern = prompt_generic_kernel<T, DD, GG>;
            CORM_CUDA(ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem));
            kern<<<(unsigned)U, kPromptThreads, smem, st>>>(p);
            CORM_CUDA(cudaGetLastError());
            return CORM_OK;
        });
    }
    if (rc != CORM_OK) return rc;
    c->launches += n_launched;
    c->parity[layer] = 0; c->steps[layer] = 0; c->ready[layer] = 1; c->live_upper[layer] = max_p; c->live_mean[layer] = 0;
    c->have_q_prev[layer] = 0;                    // the previous decode query belonged to the old text
    c->step_group[layer] = -1;
    c->group_upper[layer] = INT_MAX;
    c->last_readback_step[layer] = 0;
    schedule_live_readback(c, layer, st);
    return CORM_OK;
}

corm_status_t corm_decode_step(corm_cache_t* c, int32_t layer, const void* q, const void* k_new, const void* v_new,
                               void* out, void* stream) {
    NvtxRange nvtx_range("corm_decode_step");
    if (!layer_ok(c, layer) || !q || !k_new || !v_new || !out) return CORM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
         reinterpret_cast<uintptr_t>(out)) % 16) return CORM_ERR_INVALID_ARG;
    if (!c->ready[layer]) return CORM_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    return launch_decode(c, layer, q, k_new, v_new, out, static_cast<cudaStream_t>(stream));
}

corm_status_t corm_decode_step_layers(corm_cache_t* c, int32_t first_layer, int32_t n_layers, const void* const* q,
                                      const void* const* k_new, const void* const* v_new, void* const* out,
                                      void* stream) {
    NvtxRange nvtx_range("corm_decode_step_layers");
    if (!c || n_layers < 1 || !layer_ok(c, first_layer) || !layer_ok(c, first_layer + n_layers - 1) || !q || !k_new ||
        !v_new || !out) return CORM_ERR_INVALID_ARG;
    for (int i = 0; i < n_layers; ++i) {                 // everything is checked before anything is enqueued
        if (!q[i] || !k_new[i] || !v_new[i] || !out[i]) return CORM_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(q[i]) | reinterpret_cast<uintptr_t>(k_new[i]) | reinterpret_cast<uintptr_t>(v_new[i]) |
             reinterpret_cast<uintptr_t>(out[i])) % 16) return CORM_ERR_INVALID_ARG;
        if (!c->ready[first_layer + i]) return CORM_ERR_STATE;
    }
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    // One launch for all the layers when the kernels can see them as one array of units: a slab cache on the
    // bf16 / head_dim-128 kernels, every layer at the same step with the same buffer parity, and the layers' q,
    // k_new, v_new and out contiguous in layer order. (Grouped heads also need the tensor map over all layers, which
    // starts at layer 0.)
    const corm_config_t& cf = c->cfg;
    const size_t qb = (size_t)cf.batch * cf.n_q_heads * cf.head_dim * c->e, kb = (size_t)c->U * cf.head_dim * c->e;
    bool fuse = n_layers > 1 && fused_layers_of(cf, c->pool_pages) > 1 && c->allow_fast && cf.kv_dtype == CORM_BF16 &&
                cf.head_dim == 128 && c->G <= 4 && !c->monitor_similarity &&
                ((c->allow_fast != 6 && (c->G == 1 || c->allow_fast == 2 || c->allow_fast == 3)) || (c->have_vmap_all && first_layer == 0));
    for (int i = 1; fuse && i < n_layers; ++i) {
        const auto at = [](const void* ptr, size_t off) { return static_cast<const unsigned char*>(ptr) + off; };
        fuse = c->steps[first_layer + i] == c->steps[first_layer] && c->parity[first_layer + i] == c->parity[first_layer] &&
               q[i] == at(q[0], i * qb) && out[i] == at(out[0], i * qb) && k_new[i] == at(k_new[0], i * kb) &&
               v_new[i] == at(v_new[0], i * kb);
    }
    if (fuse) return launch_decode(c, first_layer, q[0], k_new[0], v_new[0], out[0], static_cast<cudaStream_t>(stream), n_layers);
    for (int i = 0; i < n_layers; ++i) {
        const corm_status_t rc = launch_decode(c, first_layer + i, q[i], k_new[i], v_new[i], out[i], static_cast<cudaStream_t>(stream));
        if (rc != CORM_OK) return rc;
    }
    return CORM_OK;
}

}  // extern "C"

namespace {
corm_status_t decode_steps_impl(corm_cache_t* c, int32_t first_layer, int32_t n_layers, int32_t n_steps, const void* q,
                                const void* k_new, const void* v_new, void* out, void* stream) {
    if (!c || n_layers < 1 || n_steps < 0 || !layer_ok(c, first_layer) || !layer_ok(c, first_layer + n_layers - 1))
        return CORM_ERR_INVALID_ARG;
    if (n_steps == 0) return CORM_OK;
    if (!q || !k_new || !v_new || !out) return CORM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
         reinterpret_cast<uintptr_t>(out)) % 16) return CORM_ERR_INVALID_ARG;
    for (int i = 0; i < n_layers; ++i)
        if (!c->ready[first_layer + i]) return CORM_ERR_STATE;
    const corm_config_t& cf = c->cfg;
    DeviceGuard guard(cf.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t qb = (size_t)cf.batch * cf.n_q_heads * cf.head_dim * c->e, kb = (size_t)c->U * cf.head_dim * c->e;
    // all layers of a step as one launch under the same conditions as corm_decode_step_layers (the buffers are
    // contiguous by this call's layout)
    bool fuse = n_layers > 1 && fused_layers_of(cf, c->pool_pages) > 1 && c->allow_fast && cf.kv_dtype == CORM_BF16 &&
                cf.head_dim == 128 && c->G <= 4 && !c->monitor_similarity &&
                ((c->allow_fast != 6 && (c->G == 1 || c->allow_fast == 2 || c->allow_fast == 3)) || (c->have_vmap_all && first_layer == 0));
    for (int i = 1; fuse && i < n_layers; ++i)
        fuse = c->steps[first_layer + i] == c->steps[first_layer] && c->parity[first_layer + i] == c->parity[first_layer];
    const auto at = [](const void* ptr, size_t off) { return static_cast<const unsigned char*>(ptr) + off; };
    const auto at_out = [](void* ptr, size_t off) { return static_cast<unsigned char*>(ptr) + off; };
    // A call that enqueues many steps at once would size all of them from whatever the host knew on entry. If a length
    // read-back is still in flight (typically the prompt pass's: without it the bound is the prompt length, several
    // times the survivors), wait for it here, once: the GPU is busy with what precedes it anyway.
    if (n_steps > 1)
        for (int i = 0; i < n_layers; ++i)
            if (c->readback_pending[first_layer + i]) (void)cudaEventSynchronize(c->readback_ev[first_layer + i]);
    for (int s = 0; s < n_steps; ++s) {
        // A step is chained to the one before it when that one was enqueued by this call (nothing of the caller's can
        // sit between them on the stream, and every step's inputs precede the call) and neither is the last word on
        // its units' lengths for the host: a length read-back between two launches separates them anyway.
        const bool chain = s > 0, more = s + 1 < n_steps;
        if (fuse || n_layers == 1) {
            const size_t i0 = (size_t)s * n_layers;
            const corm_status_t rc = launch_decode(c, first_layer, at(q, i0 * qb), at(k_new, i0 * kb), at(v_new, i0 * kb),
                                                   at_out(out, i0 * qb), st, n_layers, chain, more);
            if (rc != CORM_OK) return rc;
            continue;
        }
        for (int i = 0; i < n_layers; ++i) {   // separate launches per layer: another layer's launch sits between two steps of one
            const size_t ix = (size_t)s * n_layers + i;
            const corm_status_t rc = launch_decode(c, first_layer + i, at(q, ix * qb), at(k_new, ix * kb), at(v_new, ix * kb),
                                                   at_out(out, ix * qb), st);
            if (rc != CORM_OK) return rc;
        }
    }
    return CORM_OK;
}
}  // namespace

extern "C" {

corm_status_t corm_decode_steps(corm_cache_t* c, int32_t first_layer, int32_t n_layers, int32_t n_steps, const void* q,
                                const void* k_new, const void* v_new, void* out, void* stream) {
    NvtxRange nvtx_range("corm_decode_steps");
    return decode_steps_impl(c, first_layer, n_layers, n_steps, q, k_new, v_new, out, stream);
}

corm_status_t corm_decode_steps_host(corm_cache_t* c, int32_t first_layer, int32_t n_layers, int32_t n_steps,
                                     const void* q_host, const void* k_new_host, const void* v_new_host, void* out_host,
                                     void* stream) {
    NvtxRange nvtx_range("corm_decode_steps_host");
    if (!c || n_layers < 1 || n_steps < 0 || !layer_ok(c, first_layer) || !layer_ok(c, first_layer + n_layers - 1))
        return CORM_ERR_INVALID_ARG;
    if (n_steps == 0) return CORM_OK;
    if (!q_host || !k_new_host || !v_new_host || !out_host) return CORM_ERR_INVALID_ARG;
    {   // pinned, mapped buffers: the kernels read and write them in place, exactly as corm_decode_steps would
        DeviceGuard guard(c->cfg.device);
        if (!guard.ok) return CORM_ERR_CUDA;
        const void* in[4] = {q_host, k_new_host, v_new_host, out_host};
        void* dev[4] = {nullptr, nullptr, nullptr, nullptr};
        bool mapped = true;
        for (int i = 0; i < 4 && mapped; ++i) {
            cudaPointerAttributes at{};
            if (cudaPointerGetAttributes(&at, in[i]) != cudaSuccess) { (void)cudaGetLastError(); mapped = false; break; }
            mapped = at.type == cudaMemoryTypeHost && at.devicePointer && reinterpret_cast<uintptr_t>(at.devicePointer) % 16 == 0;
            dev[i] = at.devicePointer;
        }
        if (mapped) return decode_steps_impl(c, first_layer, n_layers, n_steps, dev[0], dev[1], dev[2], dev[3], stream);
    }
    // any other host memory: step by step and layer by layer through the staging buffers
    const size_t qb = (size_t)c->cfg.batch * c->cfg.n_q_heads * c->cfg.head_dim * c->e, kb = (size_t)c->U * c->cfg.head_dim * c->e;
    for (int s = 0; s < n_steps; ++s)
        for (int i = 0; i < n_layers; ++i) {
            const size_t ix = (size_t)s * n_layers + i;
            const corm_status_t rc = corm_decode_step_host(c, first_layer + i, static_cast<const unsigned char*>(q_host) + ix * qb,
                                                           static_cast<const unsigned char*>(k_new_host) + ix * kb,
                                                           static_cast<const unsigned char*>(v_new_host) + ix * kb,
                                                           static_cast<unsigned char*>(out_host) + ix * qb, stream);
            if (rc != CORM_OK) return rc;
        }
    return CORM_OK;
}

int64_t corm_cache_chained_launches(const corm_cache_t* c) { return c ? c->chained_launches : 0; }

corm_status_t corm_decode_step_host(corm_cache_t* c, int32_t layer, const void* q_host, const void* k_new_host,
                                    const void* v_new_host, void* out_host, void* stream) {
    NvtxRange nvtx_range("corm_decode_step_host");
    if (!layer_ok(c, layer) || !q_host || !k_new_host || !v_new_host || !out_host) return CORM_ERR_INVALID_ARG;
    if (!c->ready[layer]) return CORM_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t qb = (size_t)c->cfg.batch * c->cfg.n_q_heads * c->cfg.head_dim * c->e;
    const size_t kb = (size_t)c->U * c->cfg.head_dim * c->e;
    // Pinned, mapped host buffers are handed to the kernels as they are: each unit's 256-byte query, key and value
    // rows cross the bus from inside the launch and the outputs are written straight to the host, so a step needs
    // no copy engine work at all. Any other host memory goes through the staging buffers of the arena.
    {
        const void* in[3] = {q_host, k_new_host, v_new_host};
        void* dev[4] = {nullptr, nullptr, nullptr, nullptr};
        bool mapped = true;
        for (int i = 0; i < 4 && mapped; ++i) {
            const void* h = i < 3 ? in[i] : out_host;
            cudaPointerAttributes at{};
            if (cudaPointerGetAttributes(&at, h) != cudaSuccess) { (void)cudaGetLastError(); mapped = false; break; }
            mapped = at.type == cudaMemoryTypeHost && at.devicePointer && reinterpret_cast<uintptr_t>(at.devicePointer) % 16 == 0;
            dev[i] = at.devicePointer;
        }
        if (mapped) return launch_decode(c, layer, dev[0], dev[1], dev[2], dev[3], st);
    }
    unsigned char *dq = c->arena + c->lay.stage_q, *dk = c->arena + c->lay.stage_k, *dv = c->arena + c->lay.stage_v,
                  *dout = c->arena + c->lay.stage_out;
    CORM_CUDA(cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, st));
    CORM_CUDA(cudaMemcpyAsync(dk, k_new_host, kb, cudaMemcpyHostToDevice, st));
    CORM_CUDA(cudaMemcpyAsync(dv, v_new_host, kb, cudaMemcpyHostToDevice, st));
    corm_status_t rc = launch_decode(c, layer, dq, dk, dv, dout, st);
    if (rc != CORM_OK) return rc;
    CORM_CUDA(cudaMemcpyAsync(out_host, dout, qb, cudaMemcpyDeviceToHost, st));
    return CORM_OK;
}

// ---- decode step for callers that cannot allocate device memory ------------------------------------------------
// The scratch of the decode kernel (this step's logits, the split partial records and the per-unit arrival
// counters) lives in one file-scope device array instead of caller memory. Every GPU that loads this library
// holds the array until the process exits.
constexpr size_t kStaticScratchBytes = (size_t)16 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
unsigned char* g_static_scratch_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_static_scratch_mu;                           // two host threads may make a device's first call together

// The array's name is only a handle on the host; its device address must be asked for, once per device, with that
// device current. The caller holds a DeviceGuard for `device`.
corm_status_t static_scratch_address(int device, unsigned char** out) {
    if (device < 0 || device >= kMaxDevices) return CORM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_scratch_mu);
    if (!g_static_scratch_ptr[device]) {
        void* ptr = nullptr;
        CORM_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        g_static_scratch_ptr[device] = static_cast<unsigned char*>(ptr);
    }
    *out = g_static_scratch_ptr[device];
    return CORM_OK;
}
}  // namespace

corm_status_t corm_decode_step_static(corm_cache_t* c, int32_t layer, const void* q, const void* k_new,
                                      const void* v_new, void* out, void* stream) {
    NvtxRange nvtx_range("corm_decode_step_static");
    if (!layer_ok(c, layer) || !q || !k_new || !v_new || !out) return CORM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
         reinterpret_cast<uintptr_t>(out)) % 16) return CORM_ERR_INVALID_ARG;
    if (!c->ready[layer]) return CORM_ERR_STATE;
    const corm_config_t& cf = c->cfg;
    const size_t C = cf.max_tokens, D = cf.head_dim, U = c->U, G = c->G;
    const int split_len = 256;
    const int upper = std::min(cf.max_tokens, c->live_upper[layer] + 1);
    const int n_splits = (upper + split_len - 1) / split_len;
    const size_t stash_bytes = align_up(U * G * C * 8);
    const size_t partial_bytes = align_up(U * (size_t)n_splits * G * partial_stride((int)D));
    const size_t ticket_bytes = align_up(U * 4);
    if (stash_bytes + partial_bytes + ticket_bytes > kStaticScratchBytes) {
        std::fprintf(stderr, "corm_decode_step_static: this cache needs %zu bytes of scratch per step, the built-in "
                             "scratch holds %zu; use corm_decode_step with an arena instead\n",
                     stash_bytes + partial_bytes + ticket_bytes, kStaticScratchBytes);
        return CORM_ERR_CAPACITY;
    }
    DeviceGuard guard(cf.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    unsigned char* scratch = nullptr;
    corm_status_t rc = static_scratch_address(cf.device, &scratch);
    if (rc != CORM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DecodeParams p{};
    p.K = layer_ptr(c, c->lay.K, kv_layer_bytes(c), layer);
    p.V = layer_ptr(c, c->lay.V, kv_layer_bytes(c), layer);
    set_paging(c, layer, p);
    p.word = reinterpret_cast<uint32_t*>(layer_ptr(c, c->lay.word, U * C * 4, layer));
    p.pos = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.pos, U * C * 4, layer));
    p.live_in = live_buf(c, layer, c->parity[layer]);
    p.live_out = live_buf(c, layer, c->parity[layer] ^ 1);
    p.base_tokens = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.base_tokens, (size_t)cf.batch * 4, layer));
    p.base_obs = reinterpret_cast<int32_t*>(layer_ptr(c, c->lay.base_obs, (size_t)cf.batch * 4, layer));
    p.counters = reinterpret_cast<unsigned long long*>(layer_ptr(c, c->lay.counters, CNT_COUNT * 8, layer));
    p.status = reinterpret_cast<int32_t*>(c->arena + c->lay.status);
    p.stash = reinterpret_cast<double*>(scratch);
    p.partials = scratch + stash_bytes;
    p.ticket = reinterpret_cast<uint32_t*>(scratch + stash_bytes + partial_bytes);
    p.q = q; p.k_new = k_new; p.v_new = v_new; p.out = out;
    p.U = (int)U; p.Hkv = cf.n_kv_heads; p.C = cf.max_tokens; p.max_splits = n_splits; p.split_len = split_len;
    p.step = c->steps[layer]; p.w = cf.window_w; p.r = cf.recent_r;
    p.log_alpha = log_alpha_of(c);
    // the array keeps whatever the previous call (of any cache) left: the arrival counters must start at zero;
    // logits and partial records are fully rewritten before they are read
    CORM_CUDA(cudaMemsetAsync(p.ticket, 0, U * 4, st));
    rc = dispatch(c, [&](auto* tp, auto dd, auto gg) -> corm_status_t {
        using T = std::remove_pointer_t<decltype(tp)>;
        constexpr int DD = decltype(dd)::value, GG = decltype(gg)::value;
        const size_t smem = generic_decode_smem(DD, GG, cf.max_tokens, c->pool_pages != 0);
        auto kern = decode_generic_kernel<T, DD, GG>;
        CORM_CUDA(ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem));
        kern<<<dim3(n_splits, (unsigned)U), kGenericThreads, smem, st>>>(p);
        CORM_CUDA(cudaGetLastError());
        return CORM_OK;
    });
    if (rc != CORM_OK) return rc;
    c->launches += 1;
    c->chain_ok[layer] = 0;
    c->parity[layer] ^= 1;
    c->steps[layer] += 1;
    c->live_upper[layer] = std::min(cf.max_tokens, c->live_upper[layer] + 1);
    return monitor_similarity(c, layer, q, st);
}

corm_status_t corm_cache_live_lens(corm_cache_t* c, int32_t layer, int32_t* live_host, void* stream) {
    if (!layer_ok(c, layer) || !live_host) return CORM_ERR_INVALID_ARG;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CORM_CUDA(cudaMemcpyAsync(live_host, live_buf(c, layer, c->parity[layer]), (size_t)c->U * 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaStreamSynchronize(st));
    return CORM_OK;
}

corm_status_t corm_cache_stats(corm_cache_t* c, corm_stats_t* out_host, void* stream) {
    NvtxRange nvtx_range("corm_cache_stats");
    if (!c || !out_host) return CORM_ERR_INVALID_ARG;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int L = c->cfg.n_layers;
    std::vector<int32_t> live((size_t)L * 2 * c->U);
    std::vector<unsigned long long> cnt((size_t)L * CNT_COUNT);
    int32_t status = 0;
    CORM_CUDA(cudaMemcpyAsync(live.data(), c->arena + c->lay.live, live.size() * 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaMemcpyAsync(cnt.data(), c->arena + c->lay.counters, cnt.size() * 8, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaMemcpyAsync(&status, c->arena + c->lay.status, 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaStreamSynchronize(st));
    corm_stats_t s{};
    for (int l = 0; l < L; ++l) {
        const int32_t* lv = live.data() + ((size_t)c->parity[l] * L + l) * c->U;
        for (int u = 0; u < c->U; ++u) s.live_keys += lv[u];
        s.appended_keys += (int64_t)cnt[(size_t)l * CNT_COUNT + CNT_APPENDED];
        s.evicted_keys += (int64_t)cnt[(size_t)l * CNT_COUNT + CNT_EVICTED];
        s.moved_rows += (int64_t)cnt[(size_t)l * CNT_COUNT + CNT_MOVED];
        s.attended_keys += (int64_t)cnt[(size_t)l * CNT_COUNT + CNT_ATTENDED];
        s.important_keys += (int64_t)cnt[(size_t)l * CNT_COUNT + CNT_IMPORTANT];
        s.near_threshold += (int64_t)cnt[(size_t)l * CNT_COUNT + CNT_NEAR];
    }
    s.retention = s.appended_keys ? (double)s.live_keys / (double)s.appended_keys : 1.0;
    s.kv_bytes_live = s.live_keys * 2 * c->cfg.head_dim * (int64_t)c->e;
    s.aux_bytes_live = s.live_keys * 8;
    s.device_status = status;
    *out_host = s;
    return CORM_OK;
}

corm_status_t corm_cache_export_state(corm_cache_t* c, int32_t layer, int32_t seq, int32_t kv_head, void* k_host,
                                      void* v_host, uint32_t* word_host, int32_t* pos_host, int32_t* live_len,
                                      int32_t* n_tokens, int32_t* n_obs, void* stream) {
    if (!layer_ok(c, layer) || seq < 0 || seq >= c->cfg.batch || kv_head < 0 || kv_head >= c->cfg.n_kv_heads)
        return CORM_ERR_INVALID_ARG;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const corm_config_t& cf = c->cfg;
    const size_t C = cf.max_tokens, D = cf.head_dim, U = c->U, u = (size_t)seq * cf.n_kv_heads + kv_head;
    const size_t row_bytes = C * D * c->e;
    int32_t bt = 0, bo = 0, lv = 0;
    if (c->pool_pages) {   // page by page, in slot order; slots of pages the unit does not own are left as they are
        std::vector<int32_t> pt(c->pt_stride);
        CORM_CUDA(cudaMemcpyAsync(pt.data(), page_table_ptr(c, layer) + u * c->pt_stride, pt.size() * 4, cudaMemcpyDeviceToHost, st));
        CORM_CUDA(cudaStreamSynchronize(st));
        const size_t page_bytes = (size_t)kPageKeys * D * c->e;
        for (int i = 0; i < c->pt_stride; ++i) {
            if (pt[i] <= 0 || pt[i] > c->pool_pages) continue;
            const size_t n = std::min(page_bytes, row_bytes - (size_t)i * page_bytes);
            const size_t at = (size_t)(pt[i] - 1) * page_bytes;
            if (k_host) CORM_CUDA(cudaMemcpyAsync(static_cast<unsigned char*>(k_host) + (size_t)i * page_bytes, layer_ptr(c, c->lay.K, kv_layer_bytes(c), layer) + at, n, cudaMemcpyDeviceToHost, st));
            if (v_host) CORM_CUDA(cudaMemcpyAsync(static_cast<unsigned char*>(v_host) + (size_t)i * page_bytes, layer_ptr(c, c->lay.V, kv_layer_bytes(c), layer) + at, n, cudaMemcpyDeviceToHost, st));
        }
    } else {
        if (k_host) CORM_CUDA(cudaMemcpyAsync(k_host, layer_ptr(c, c->lay.K, U * row_bytes, layer) + u * row_bytes, row_bytes, cudaMemcpyDeviceToHost, st));
        if (v_host) CORM_CUDA(cudaMemcpyAsync(v_host, layer_ptr(c, c->lay.V, U * row_bytes, layer) + u * row_bytes, row_bytes, cudaMemcpyDeviceToHost, st));
    }
    if (word_host) CORM_CUDA(cudaMemcpyAsync(word_host, layer_ptr(c, c->lay.word, U * C * 4, layer) + u * C * 4, C * 4, cudaMemcpyDeviceToHost, st));
    if (pos_host) CORM_CUDA(cudaMemcpyAsync(pos_host, layer_ptr(c, c->lay.pos, U * C * 4, layer) + u * C * 4, C * 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaMemcpyAsync(&lv, live_buf(c, layer, c->parity[layer]) + u, 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaMemcpyAsync(&bt, layer_ptr(c, c->lay.base_tokens, (size_t)cf.batch * 4, layer) + (size_t)seq * 4, 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaMemcpyAsync(&bo, layer_ptr(c, c->lay.base_obs, (size_t)cf.batch * 4, layer) + (size_t)seq * 4, 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaStreamSynchronize(st));
    if (live_len) *live_len = lv;
    if (n_tokens) *n_tokens = bt + c->steps[layer];
    if (n_obs) *n_obs = std::min(cf.window_w, bo + c->steps[layer]);
    return CORM_OK;
}

corm_status_t corm_cache_import_state(corm_cache_t* c, int32_t layer, int32_t seq, int32_t kv_head, const void* k_host,
                                      const void* v_host, const uint32_t* word_host, const int32_t* pos_host,
                                      int32_t live_len, int32_t n_tokens, int32_t n_obs, void* stream) {
    if (!layer_ok(c, layer) || seq < 0 || seq >= c->cfg.batch || kv_head < 0 || kv_head >= c->cfg.n_kv_heads)
        return CORM_ERR_INVALID_ARG;
    const corm_config_t& cf = c->cfg;
    if (live_len < 0 || n_tokens < 0 || n_obs < 0 || n_obs > cf.window_w) return CORM_ERR_INVALID_ARG;
    if (live_len > cf.max_tokens) return CORM_ERR_CAPACITY;
    if (live_len > 0 && (!k_host || !v_host || !word_host || !pos_host)) return CORM_ERR_INVALID_ARG;
    DeviceGuard guard(cf.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t C = cf.max_tokens, D = cf.head_dim, U = c->U, u = (size_t)seq * cf.n_kv_heads + kv_head;
    const size_t row_bytes = C * D * c->e, n = (size_t)live_len;
    if (c->pool_pages) {
        // The host edits the layer's page bitmap and this unit's page table itself (nothing else runs meanwhile: the
        // stream is drained first): the unit's old pages are returned, live_len / 32 + 1 pages are claimed, rows are
        // copied page by page.
        CORM_CUDA(cudaStreamSynchronize(st));
        std::vector<int32_t> pt(c->pt_stride);
        std::vector<uint32_t> bits(c->pool_pages / 32);
        int32_t* pt_dev = page_table_ptr(c, layer) + u * c->pt_stride;
        CORM_CUDA(cudaMemcpy(pt.data(), pt_dev, pt.size() * 4, cudaMemcpyDeviceToHost));
        CORM_CUDA(cudaMemcpy(bits.data(), page_bits_ptr(c, layer), bits.size() * 4, cudaMemcpyDeviceToHost));
        for (int i = 0; i < c->pt_stride; ++i) {
            if (pt[i] > 0 && pt[i] <= c->pool_pages) bits[(pt[i] - 1) >> 5] &= ~(1u << ((pt[i] - 1) & 31));
            pt[i] = 0;
        }
        const int need = std::min(live_len / kPageKeys + 1, c->pt_stride);
        int next = 0;
        for (int i = 0; i < need; ++i) {
            while (next < c->pool_pages && (bits[next >> 5] >> (next & 31) & 1u)) ++next;
            if (next >= c->pool_pages) return CORM_ERR_CAPACITY;          // nothing has been written to the device yet
            bits[next >> 5] |= 1u << (next & 31);
            pt[i] = next + 1;
        }
        CORM_CUDA(cudaMemcpy(pt_dev, pt.data(), pt.size() * 4, cudaMemcpyHostToDevice));
        CORM_CUDA(cudaMemcpy(page_bits_ptr(c, layer), bits.data(), bits.size() * 4, cudaMemcpyHostToDevice));
        const int32_t has_room = 1;
        CORM_CUDA(cudaMemcpy(page_room_ptr(c, layer) + u, &has_room, 4, cudaMemcpyHostToDevice));
        const size_t page_bytes = (size_t)kPageKeys * D * c->e;
        for (size_t i = 0; i * kPageKeys < n; ++i) {
            const size_t bytes = std::min(page_bytes, n * D * c->e - i * page_bytes), at = (size_t)(pt[i] - 1) * page_bytes;
            CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.K, kv_layer_bytes(c), layer) + at, static_cast<const unsigned char*>(k_host) + i * page_bytes, bytes, cudaMemcpyHostToDevice, st));
            CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.V, kv_layer_bytes(c), layer) + at, static_cast<const unsigned char*>(v_host) + i * page_bytes, bytes, cudaMemcpyHostToDevice, st));
        }
        if (n) {
            CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.word, U * C * 4, layer) + u * C * 4, word_host, n * 4, cudaMemcpyHostToDevice, st));
            CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.pos, U * C * 4, layer) + u * C * 4, pos_host, n * 4, cudaMemcpyHostToDevice, st));
        }
    } else if (n) {
        CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.K, U * row_bytes, layer) + u * row_bytes, k_host, n * D * c->e, cudaMemcpyHostToDevice, st));
        CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.V, U * row_bytes, layer) + u * row_bytes, v_host, n * D * c->e, cudaMemcpyHostToDevice, st));
        CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.word, U * C * 4, layer) + u * C * 4, word_host, n * 4, cudaMemcpyHostToDevice, st));
        CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.pos, U * C * 4, layer) + u * C * 4, pos_host, n * 4, cudaMemcpyHostToDevice, st));
    }
    // the kernels see tokens = base + steps and rows = min(w, base + steps): rebase this sequence
    const int32_t bt = n_tokens - c->steps[layer], bo = n_obs - c->steps[layer], lv = live_len;
    CORM_CUDA(cudaMemcpyAsync(live_buf(c, layer, c->parity[layer]) + u, &lv, 4, cudaMemcpyHostToDevice, st));
    CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.base_tokens, (size_t)cf.batch * 4, layer) + (size_t)seq * 4, &bt, 4, cudaMemcpyHostToDevice, st));
    CORM_CUDA(cudaMemcpyAsync(layer_ptr(c, c->lay.base_obs, (size_t)cf.batch * 4, layer) + (size_t)seq * 4, &bo, 4, cudaMemcpyHostToDevice, st));
    CORM_CUDA(cudaStreamSynchronize(st));
    c->ready[layer] = 1;
    c->readback_pending[layer] = 0;   // a read-back enqueued before this import knows nothing of it
    c->live_upper[layer] = std::max(c->live_upper[layer], live_len);
    c->live_mean[layer] = 0;                      // unknown until the next read-back
    c->step_group[layer] = -2;                    // lengths changed behind the kernels' backs: the layer keeps its own bound
    c->group_upper[layer] = INT_MAX;
    c->chain_ok[layer] = 0;                       // ... and its units' stamps no longer describe them
    return CORM_OK;
}

corm_status_t corm_cache_pool_usage(corm_cache_t* c, int32_t layer, int64_t* pages_in_use, int64_t* pages_total, void* stream) {
    if (!layer_ok(c, layer) || !pages_in_use || !pages_total) return CORM_ERR_INVALID_ARG;
    *pages_in_use = 0;
    *pages_total = c->pool_pages;
    if (!c->pool_pages) return CORM_OK;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<uint32_t> bits(c->pool_pages / 32);
    CORM_CUDA(cudaMemcpyAsync(bits.data(), page_bits_ptr(c, layer), bits.size() * 4, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaStreamSynchronize(st));
    for (uint32_t w : bits) *pages_in_use += __builtin_popcount(w);
    return CORM_OK;
}

corm_status_t corm_cache_set_tuning(corm_cache_t* c, int32_t split_len, int32_t allow_fast_path) {
    if (!c || split_len < 0 || (split_len % 32) || (split_len && split_len < kMinSplit)) return CORM_ERR_INVALID_ARG;
    c->tune_split_len = split_len;
    if (allow_fast_path < 0 || allow_fast_path > 6) return CORM_ERR_INVALID_ARG;
    c->allow_fast = allow_fast_path;
    return CORM_OK;
}

corm_status_t corm_cache_set_similarity_monitor(corm_cache_t* c, int32_t enabled) {
    if (!c) return CORM_ERR_INVALID_ARG;
    c->monitor_similarity = enabled ? 1 : 0;
    if (!enabled) std::fill(c->have_q_prev.begin(), c->have_q_prev.end(), 0);   // a gap breaks the chain of adjacent steps
    return CORM_OK;
}

corm_status_t corm_cache_similarity(corm_cache_t* c, double* sum_host, int64_t* count_host, void* stream) {
    if (!c || !sum_host || !count_host) return CORM_ERR_INVALID_ARG;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return CORM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char buf[16];
    CORM_CUDA(cudaMemcpyAsync(buf, c->arena + c->lay.sim_acc, 16, cudaMemcpyDeviceToHost, st));
    CORM_CUDA(cudaStreamSynchronize(st));
    std::memcpy(sum_host, buf, 8);
    unsigned long long n;
    std::memcpy(&n, buf + 8, 8);
    *count_host = (int64_t)n;
    return CORM_OK;
}

corm_status_t corm_cache_set_bound_scale(corm_cache_t* c, double scale) {
    if (!c || !(scale >= 1.0) || !std::isfinite(scale)) return CORM_ERR_INVALID_ARG;
    c->bound_scale = scale;
    return CORM_OK;
}

int64_t corm_cache_kernel_launches(const corm_cache_t* c) { return c ? c->launches : 0; }

const char* corm_status_string(corm_status_t s) {
    switch (s) {
        case CORM_OK: return "ok";
        case CORM_ERR_INVALID_ARG: return "invalid argument";
        case CORM_ERR_UNSUPPORTED: return "unsupported configuration";
        case CORM_ERR_ARENA_TOO_SMALL: return "arena too small";
        case CORM_ERR_STATE: return "call out of order (no prompt pass for this layer)";
        case CORM_ERR_CUDA: return "CUDA runtime error";
        case CORM_ERR_CAPACITY: return "slab capacity exceeded";
        case CORM_ERR_TIMEOUT: return "bounded wait expired";
        case CORM_ERR_INTERNAL: return "internal invariant broken (index outside its range)";
    }
    return "unknown status";
}

}  // extern "C"
