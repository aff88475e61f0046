// C ABI of the offloaded-MoE decode step (see include/spm.h): context, slot pools, copy-stream
// scheduling with CUDA events, kernel launches. All arithmetic of the path runs in the kernels
// of ffn_gemv.cuh / router_adapter.cuh; this file is host control only.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <deque>
#include <string>
#include <utility>
#include <vector>

#include <cuda_runtime.h>
#include <immintrin.h>

#include "../../include/spm.h"
#include "ffn_gemv.cuh"
#include "ffn_gemv_q4.cuh"
#include "ffn_grouped.cuh"
#include "ffn_grouped_q4.cuh"
#include "router_adapter.cuh"
#include "tma_maps.h"
#include "gg_plan.h"
#include "slot_table.h"

using namespace spm;

namespace {

thread_local std::string g_init_error;

struct bf16_t { uint16_t v; };

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

enum ClockKind : uint8_t { kClkFfn = 0, kClkRouter = 1, kClkReduce = 2 };   // owners of in-kernel clock slots

struct Timing {            // CUDA events of one step, per layer
    std::vector<cudaEvent_t> k1_done, ffn_start, ffn_end;
    std::vector<uint8_t> used;
};

}  // namespace

struct spm_ctx {
    spm_model_cfg cfg{};
    int S = 0, budget = 0, policy = SPM_POLICY_ADAPTER;
    spm_buffers buf{};
    cudaStream_t compute = nullptr, copy = nullptr;
    SlotTable* table = nullptr;
    size_t elem = 2, blob = 0, row_bytes = 0;
    int nseg = 0, depth = 2, num_sms = 148, ffn_ctas = 0;
    // arena carve-up
    unsigned char* pools = nullptr;
    float *ws_x = nullptr, *ws_logits = nullptr, *ws_pihat = nullptr, *ws_w = nullptr;
    float *ws_scores = nullptr, *ws_partial = nullptr, *ws_h = nullptr;
    int32_t *ws_ids = nullptr, *ws_order = nullptr;
    unsigned* ws_counters = nullptr;
    int* ws_status = nullptr;
    unsigned long long* ws_clock = nullptr;
    int clock_used = 0;
    std::vector<uint8_t> clock_kind;          // which kernel each armed clock slot belongs to (ClockKind)
    double window_us = 0, router_window_us = 0, reduce_window_us = 0, gap_us = 0;
    // batched tensor-core path (bf16, max_batch > 1, no shared experts, I and D multiples of 128)
    bool tc_ok = false;
    int batched_path = 0;                 // 0: tensor cores when possible, 1: always the per-token GEMV
    int rows_cap = 0, n_jt = 0, max_units = 0;
    CUtensorMap wmap{};
    GgTokenMaps xmaps{};
    CUtensorMap qmapn{}, qmapsc{};            // 4-bit blobs: nibble box of 128 bytes, scale box of 16 bytes
    __nv_bfloat16* tc_xs = nullptr;
    float *tc_wrow = nullptr, *tc_partial = nullptr;
    unsigned char* tc_desc_dev = nullptr;     // kDescRing wave descriptors
    unsigned char* tc_desc_host = nullptr;    // pinned staging, same layout
    int* tc_counts = nullptr;                 // {units, rows} of a wave planned on the device
    size_t tc_desc_bytes = 0, tc_off_rows = 0, tc_off_rowmap = 0, tc_off_chunks = 0, tc_chunk_cap = 0, tc_off_wait = 0;
    int wave_row_off = 0;                     // rows of the sorted token arrays taken by the earlier waves of this layer
    std::vector<int32_t> wave_rowmap;         // [nb][SPM_MAX_TOPK] row of each (token, k) pair over all waves so far
    unsigned char* tc_act = nullptr;          // [max_units][16 KB] A^T slots of the bf16 grouped kernel
    int* tc_ready = nullptr;                  // [1 + max_units] chunk counter, then the slots' arrival counters
    std::vector<GgTaskHost> plan_chunks;
    std::vector<cudaEvent_t> tc_desc_ev;
    std::vector<uint8_t> tc_desc_ev_valid;
    size_t tc_desc_pos = 0;
    uint64_t tc_launches = 0;
    // mailbox
    Mailbox* mb_host = nullptr;
    Mailbox* mb_dev = nullptr;
    uint32_t seq = 0;
    int deadline_ms = 5000;
    // per-slot copy events
    std::vector<cudaEvent_t> slot_ev;
    std::vector<uint8_t> slot_pending;
    std::vector<size_t> slot_dep;             // slot whose event covers the batch this slot's latest copy belongs to
    std::vector<cudaEvent_t> pool_free;       // recorded after the last FFN that read pool l
    std::vector<uint8_t> pool_free_valid;
    cudaEvent_t wave_done = nullptr;
    // timing
    bool timing = false;
    Timing tim[2];
    int tim_cur = 0;
    std::vector<double> layer_stall_us, layer_ffn_us;
    uint64_t timed_steps = 0;
    // spm_moe_ffn called on its own: ring of event pairs around the FFN kernel
    std::vector<cudaEvent_t> ring_start, ring_end;
    std::vector<uint8_t> ring_used;
    size_t ring_pos = 0;
    double ring_us = 0;
    // policy inputs
    std::vector<int32_t> hint, hint_count;
    int hint_steps = 0, hint_stride = 0;
    int drop_modulo = 0;
    int stub_us = 0;                          // attention stand-in before each layer's router
    int copy_delay_us = 0;                    // emulated slower storage tier: extra wait after every expert copy
    bool device_wait = false;                 // batch-1 FFN launched at once, waits for its copies on the device
    double prof_window_us = 0, prof_xfer_us = 0;   // what the last spm_profile_window measured (0: never run)
    int prof_raw = 0;
    unsigned long long wait_limit_ns = 0;     // limit of every device-side wait in the expert kernels (0: their 2 s default)
    int withhold_arrivals = 0;                // test hook: this many arrival-counter bumps are skipped (a wait then runs out)
    unsigned* ws_slot_gen = nullptr;          // [L][S] arrival counters, bumped by the copy stream
    std::vector<uint32_t> slot_gen_host;      // arrival counter of a slot as a batch leader: batches it has led so far
    std::vector<uint32_t> slot_want;          // counter value of its batch leader at which a slot's latest copy has landed
    // host-free steps: once every expert of every layer is resident, a step is enqueued without
    // waiting for any routing result; the routing kernel leaves slot numbers for the expert kernel
    // in device memory and its ids / ranking in a ring of host-mapped trace mailboxes, from which
    // the slot table's bookkeeping is replayed later, in order
    bool host_free = true, fast_ready = false;
    short* ws_slot_map = nullptr;             // [L][n] slot of each expert (valid while fast_ready)
    short* ws_codes = nullptr;                // [L][max_batch][K] slots of the routed experts of the step in flight
    Mailbox* tr_host = nullptr;               // [kTraceRing][L]
    Mailbox* tr_dev = nullptr;
    std::vector<cudaEvent_t> tr_ev;
    std::deque<std::pair<int, int>> tr_pending;   // (ring slot, nb) of steps enqueued but not yet replayed
    uint64_t tr_count = 0, host_free_steps = 0;
    struct HostFreeGraph {                    // a captured host-free step and what one replay adds to the launch counters
        int slot, nb; const float* h_out; bool predict; int G, batched_path;
        uint64_t kernels, ffns, tcs;
        cudaGraphExec_t exec;
    };
    std::vector<HostFreeGraph> hf_graphs;
    bool graph_replay = true, hf_warm = false;
    std::vector<std::vector<int32_t>> prev_rank;   // Naive Prefetch: experts the preceding step used, per layer
    std::vector<std::vector<int32_t>> pending_protect;
    std::vector<uint8_t> has_plan;
    std::vector<int32_t> prev_order;          // ranking produced at the previous layer of this step
    bool prev_order_valid = false;
    // scratch
    std::vector<Placement> placements;
    std::vector<int32_t> need, sel, protect, slots_tmp;
    std::vector<int16_t> wave_slot;
    std::vector<int32_t> plan_first;
    uint64_t extra_late = 0, h2d_bytes = 0, ffn_launches = 0, kernel_launches = 0, tokens = 0;
    double ready_sum = 0, recall_sum = 0;
    double recall_at[3] = {0, 0, 0};          // ExpertRecall@M for M = K/2, K, K+2 (same terms as recall_sum)
    uint64_t ready_count = 0, recall_count = 0;
    std::string err;
};

namespace {

int fail(spm_ctx* c, int code, const char* fmt, ...) {
    char b[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(b, sizeof b, fmt, ap);
    va_end(ap);
    if (c) c->err = b; else g_init_error = b;
    return code;
}

int take_clock(spm_ctx* c, ClockKind kind, unsigned long long** out);

#define CU(c, call)                                                                        \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess)                                                             \
            return fail((c), SPM_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

int check_cfg(const spm_model_cfg* m, int S, spm_ctx* c) {
    if (!m) return fail(c, SPM_ERR_INVALID_ARG, "cfg is null");
    if (m->dtype != SPM_DTYPE_FP32 && m->dtype != SPM_DTYPE_BF16 && m->dtype != SPM_DTYPE_Q4)
        return fail(c, SPM_ERR_CONFIG, "unknown dtype %d", m->dtype);
    const int seg = m->dtype == SPM_DTYPE_FP32 ? 128 : 256;
    if (m->n_layers < 1 || m->hidden < seg || m->hidden % seg || m->hidden / seg > 8)
        return fail(c, SPM_ERR_CONFIG, "hidden %d unsupported: need a multiple of %d, at most %d", m->hidden, seg, 8 * seg);
    if (m->n_experts < 1 || m->n_experts > SPM_MAX_EXPERTS) return fail(c, SPM_ERR_CONFIG, "n_experts %d out of range", m->n_experts);
    if (m->top_k < 1 || m->top_k > m->n_experts || m->n_shared < 0 || m->top_k + m->n_shared > SPM_MAX_TOPK)
        return fail(c, SPM_ERR_CONFIG, "top_k %d + n_shared %d unsupported (max %d)", m->top_k, m->n_shared, SPM_MAX_TOPK);
    if (m->inter < 1) return fail(c, SPM_ERR_CONFIG, "inter %d", m->inter);
    if (m->adapter_rank < 1 || m->adapter_rank > 256 || m->n_experts * m->adapter_rank > 32768)
        return fail(c, SPM_ERR_CONFIG, "adapter_rank %d out of range (n_experts * rank <= 32768)", m->adapter_rank);
    if (m->max_batch < 1 || m->max_batch > SPM_MAX_BATCH) return fail(c, SPM_ERR_CONFIG, "max_batch %d out of range", m->max_batch);
    if (S < 1 || S > 32767) return fail(c, SPM_ERR_CONFIG, "slots_per_layer %d out of range", S);
    if (m->max_batch == 1 && S < m->top_k) return fail(c, SPM_ERR_CONFIG, "slots_per_layer %d < top_k %d at batch 1", S, m->top_k);
    return SPM_OK;
}

size_t blob_bytes_of(const spm_model_cfg* m) {
    if (m->dtype == SPM_DTYPE_Q4) return size_t(3) * m->inter * (size_t(m->hidden) / 2 + size_t(m->hidden) / 16);
    return size_t(3) * m->inter * m->hidden * (m->dtype == SPM_DTYPE_BF16 ? 2 : 4);
}

constexpr int kMaxCtasBatch1 = 296;
constexpr int kClockSlots = 12288;    // in-kernel {start, end} pairs between two harvests
constexpr int kDescRing = 8;          // wave descriptors in flight for the batched tensor-core path
constexpr int kTraceRing = 8;         // host-free steps whose bookkeeping may be outstanding
static_assert(sizeof(GgTask) == sizeof(GgTaskHost), "host plan and device task share one layout");

// The grouped tcgen05 kernels handle bf16 or 4-bit weights, more than one sequence per step, no
// shared experts, and intermediate / hidden sizes that tile by 128.
bool tc_supported(const spm_model_cfg* m) {
    // the 4-bit kernel takes the scales of 256 columns (16 bytes per row) at a time
    const int col_step = m->dtype == SPM_DTYPE_Q4 ? 2 * kGgTileRows : kGgTileRows;
    return (m->dtype == SPM_DTYPE_BF16 || m->dtype == SPM_DTYPE_Q4) && m->max_batch > 1 && m->n_shared == 0 &&
           m->inter % kGgTileRows == 0 && m->hidden % col_step == 0;
}
static_assert(kMaxCtasBatch1 <= kReduceGroups * kReduceMaxRows, "reduce kernel covers every grid size");
static_assert(kReduceGroups == kReduceGroupsR && kReduceGroupsR == kRouterWarps, "the routing kernel folds partial rows in the combine kernel's order");

int ffn_grid_for(const spm_ctx* c, int nb) {
    if (nb == 1) return c->ffn_ctas > 0 ? std::min(c->ffn_ctas, kMaxCtasBatch1) : c->num_sms;
    return std::max(1, kMaxCtasBatch1 / nb);
}

struct Carve {
    size_t off = 0;
    size_t take(size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; }
};

struct Layout {
    size_t pools, slot_gen, x, logits, pihat, w, scores, partial, h, ids, order, clock, slot_map, codes, counters, status, total;
    size_t tc_xs, tc_wrow, tc_partial, tc_desc, tc_counts, tc_act, tc_ready;       // batched tensor-core path only
    size_t desc_bytes, off_rows, off_rowmap, off_chunks, chunk_cap, off_wait;
    int rows_cap, n_jt, max_units;
    bool tc;
};

Layout layout_of(const spm_model_cfg* m, int S) {
    Layout l{};
    Carve c;
    const size_t nb = m->max_batch, D = m->hidden, n = m->n_experts;
    l.pools = c.take(size_t(m->n_layers) * S * blob_bytes_of(m));
    l.slot_gen = c.take(size_t(m->n_layers) * S * 4);
    l.x = c.take(nb * D * 4);
    l.logits = c.take(nb * n * 4);
    l.pihat = c.take(nb * n * 4);
    l.w = c.take(nb * SPM_MAX_TOPK * 4);
    l.scores = c.take(n * 4);
    l.partial = c.take((kMaxCtasBatch1 + nb) * D * 4);
    l.h = c.take(nb * D * 4);
    l.ids = c.take(nb * SPM_MAX_TOPK * 4);
    l.order = c.take(n * 4);
    l.clock = c.take(size_t(kClockSlots) * 16);
    l.slot_map = c.take(size_t(m->n_layers) * n * sizeof(short));
    l.codes = c.take(size_t(m->n_layers) * nb * SPM_MAX_TOPK * sizeof(short));
    l.tc = tc_supported(m);
    if (l.tc) {
        l.rows_cap = m->max_batch * m->top_k;
        l.n_jt = m->inter / kGgTileRows;
        l.max_units = std::min(S, m->n_experts) * l.n_jt;
        l.off_rows = align_up(size_t(l.max_units) * sizeof(GgUnit), 256);
        l.off_rowmap = l.off_rows + align_up(size_t(l.rows_cap) * sizeof(GgRow), 256);
        // phase-2 chunk list of the bf16 kernel: at most one chunk per kGgMinChunk d-tiles, at least one per unit
        l.off_chunks = l.off_rowmap + align_up(size_t(m->max_batch) * SPM_MAX_TOPK * 4, 256);
        l.chunk_cap = size_t(l.max_units) * size_t(std::max(1, (m->hidden / kGgTileRows + kGgMinChunk - 1) / kGgMinChunk));
        l.off_wait = l.off_chunks + align_up(l.chunk_cap * sizeof(GgTask), 256);      // per unit: what its expert's copy is awaited by
        l.desc_bytes = l.off_wait + align_up(size_t(l.max_units) * sizeof(GgWait), 256);
        l.tc_xs = c.take(size_t(l.rows_cap + kGgTokens) * D * 2);
        l.tc_wrow = c.take(size_t(l.rows_cap) * 4);
        l.tc_partial = c.take(size_t(l.n_jt) * l.rows_cap * D * 4);
        l.tc_desc = c.take(size_t(kDescRing) * l.desc_bytes);
        l.tc_counts = c.take(2 * sizeof(int));
        l.tc_act = c.take(size_t(l.max_units) * kGgActBytes);
        l.tc_ready = c.take(size_t(l.max_units + 1) * sizeof(int));
    }
    l.counters = c.take(256);
    l.status = c.take(4);
    l.total = c.off;
    return l;
}

// ---- kernel dispatch -------------------------------------------------------
// Launch with an optional programmatic-serialisation attribute: the kernel may then start while
// the preceding kernel of the stream is still running and orders itself with grid_dep_wait().
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl, Args&&... args) {
    cudaLaunchConfig_t lc{};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute at[1];
    if (pdl) {
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at;
        lc.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&lc, kern, std::forward<Args>(args)...);
}

template <typename WT, int NSEG, int MAXNB>
cudaError_t launch_gemv_t(const FfnArgs<MAXNB>& a, int G, int nb, int warps, int depth, size_t smem, cudaStream_t st, bool pdl) {
    static bool attr_set[64] = {};          // the attribute is per device
    auto kern = ffn_gemv_kernel<WT, NSEG, MAXNB>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kFfnSmemLimit));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    return launch_k(kern, dim3(G, nb), dim3(warps * 32), smem, st, pdl, a, depth);
}

template <typename WT, int MAXNB>
cudaError_t launch_gemv_seg(int nseg, const FfnArgs<MAXNB>& a, int G, int nb, int warps, int depth, size_t smem, cudaStream_t st, bool pdl) {
    switch (nseg) {
        case 1: return launch_gemv_t<WT, 1, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
        case 2: return launch_gemv_t<WT, 2, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
        case 3: return launch_gemv_t<WT, 3, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
        case 4: return launch_gemv_t<WT, 4, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
        case 5: return launch_gemv_t<WT, 5, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
        case 6: return launch_gemv_t<WT, 6, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
        case 7: return launch_gemv_t<WT, 7, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
        case 8: return launch_gemv_t<WT, 8, MAXNB>(a, G, nb, warps, depth, smem, st, pdl);
    }
    return cudaErrorInvalidValue;
}

template <int NCH, int MAXNB>
cudaError_t launch_gemv_q4_t(int D, const FfnArgs<MAXNB>& a, int G, int nb, int warps, int depth, size_t smem, cudaStream_t st, bool pdl) {
    static bool attr_set[64] = {};
    auto kern = ffn_gemv_q4_kernel<NCH, MAXNB>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kFfnSmemLimit));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    return launch_k(kern, dim3(G, nb), dim3(warps * 32), smem, st, pdl, a, depth, D);
}

template <int MAXNB>
cudaError_t launch_gemv_q4(int D, const FfnArgs<MAXNB>& a, int G, int nb, int warps, int depth, size_t smem, cudaStream_t st, bool pdl) {
    if (D <= 1024) return launch_gemv_q4_t<1, MAXNB>(D, a, G, nb, warps, depth, smem, st, pdl);
    return launch_gemv_q4_t<2, MAXNB>(D, a, G, nb, warps, depth, smem, st, pdl);
}

template <int MAXNB>
cudaError_t launch_gemv(const spm_ctx* c, const FfnArgs<MAXNB>& a, int G, int nb, bool pdl = false) {
    int max_cnt = 1;
    for (int t = 0; t < nb; ++t) max_cnt = std::max(max_cnt, int(a.count[t]));
    const int rows_per_cta = (max_cnt * c->cfg.inter + G - 1) / G;
    int warps = 8, depth = 2;
    if (c->cfg.dtype == SPM_DTYPE_Q4) {
        size_t smem = 0;
        ffn_gemv_q4_shape(c->row_bytes, c->cfg.hidden, rows_per_cta, &warps, &depth, &smem);
        return launch_gemv_q4<MAXNB>(c->cfg.hidden, a, G, nb, warps, depth, smem, c->compute, pdl);
    }
    ffn_gemv_shape(c->row_bytes, rows_per_cta, &warps, &depth);
    const size_t smem = ffn_gemv_smem(c->row_bytes, warps, depth);
    if (c->cfg.dtype == SPM_DTYPE_BF16) return launch_gemv_seg<bf16_t, MAXNB>(c->nseg, a, G, nb, warps, depth, smem, c->compute, pdl);
    return launch_gemv_seg<float, MAXNB>(c->nseg, a, G, nb, warps, depth, smem, c->compute, pdl);
}

// Where a routing launch leaves its results besides the workspace: by default the context's
// mailbox, which the host polls; a host-free step names a trace mailbox, the device-side slot
// map and the slot-code row of its layer, and lets the kernel start ahead of its predecessor's end.
struct RouterRoute {
    Mailbox* mailbox_dev;
    const short* slot_map;
    short* codes_out;
    bool pdl;
    const float* partial;      // partial rows of the preceding layer's expert kernel to fold into the hidden row, or null
    int G;
};

int launch_router(spm_ctx* c, int layer, const float* h, const float* x_in, int nb, float* x_norm,
                  float* logits_out, bool do_router, bool do_adapter, const RouterRoute* route = nullptr, bool publish_seq = true) {
    const spm_model_cfg& m = c->cfg;
    RouterArgs a{};
    const size_t D = m.hidden, n = m.n_experts, r = m.adapter_rank;
    a.h = h;
    a.x_in = x_in;
    a.gamma = static_cast<const float*>(c->buf.rms_gamma) + size_t(layer) * D;
    a.router_w = static_cast<const unsigned char*>(c->buf.router_w) + size_t(layer) * n * D * c->elem;
    if (do_adapter) {
        a.adapter_a = static_cast<const unsigned char*>(c->buf.adapter_a) + size_t(layer) * r * D * c->elem;
        a.adapter_b = static_cast<const unsigned char*>(c->buf.adapter_b) + size_t(layer) * n * r * c->elem;
    }
    a.x_norm = x_norm;
    a.logits = c->ws_logits;
    a.logits_out = logits_out;
    a.pihat = c->ws_pihat;
    a.ids = c->ws_ids;
    a.w = c->ws_w;
    a.scores = c->ws_scores;
    a.order = c->ws_order;
    a.counters = c->ws_counters;
    a.status = c->ws_status;
    a.mailbox = route ? route->mailbox_dev : c->mb_dev;
    a.slot_map = route ? route->slot_map : nullptr;
    a.codes_out = route ? route->codes_out : nullptr;
    a.partial = route ? route->partial : nullptr;
    a.G = route ? route->G : 0;
    a.h_out = const_cast<float*>(h);
    a.publish_seq = publish_seq;
    if (int rc = take_clock(c, kClkRouter, &a.clock)) return rc;
    // Sequence numbers whose low 16 bits are zero are skipped, and the words this launch will
    // publish are zeroed first, so a word left by an older launch can never carry the current tag.
    ++c->seq;
    if ((c->seq & 0xffffu) == 0) ++c->seq;
    if (!route || route->mailbox_dev == c->mb_dev) {
        if (do_router) memset(const_cast<int32_t*>(c->mb_host->ids), 0, size_t(nb) * m.top_k * sizeof(int32_t));
        if (do_adapter) memset(const_cast<int32_t*>(c->mb_host->order), 0, size_t(m.n_experts) * sizeof(int32_t));
    }
    a.seq = c->seq;
    a.D = m.hidden; a.n = m.n_experts; a.K = m.top_k; a.r = m.adapter_rank; a.nb = nb;
    a.renorm = m.renormalize; a.do_router = do_router; a.do_adapter = do_adapter;
    a.eps = m.rms_eps;
    const size_t smem = router_smem_bytes(m.hidden, m.n_experts, m.adapter_rank);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(kRouterCluster, nb);
    lc.blockDim = dim3(kRouterThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = c->compute;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kRouterCluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    if (route && route->pdl) {
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        lc.numAttrs = 2;
    }
    // more CTAs than SMs: the variant compiled for two CTAs per SM halves the number of waves
    const bool dense = kRouterCluster * nb > c->num_sms && !a.partial;
    auto go = [&](auto kern) -> int {
        if (smem > 48 * 1024) CU(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        CU(c, cudaLaunchKernelEx(&lc, kern, a));
        return SPM_OK;
    };
    int rc;
    if (m.dtype != SPM_DTYPE_FP32) rc = dense ? go(router_adapter_kernel<bf16_t, 2>) : go(router_adapter_kernel<bf16_t, 1>);
    else rc = dense ? go(router_adapter_kernel<float, 2>) : go(router_adapter_kernel<float, 1>);
    if (rc) return rc;
    CU(c, cudaGetLastError());
    c->kernel_launches++;
    return SPM_OK;
}

// Wait (bounded) until the routing kernel of the current sequence number has published.
int wait_mailbox(spm_ctx* c) {
    const uint32_t want = c->seq;
    const auto t0 = std::chrono::steady_clock::now();
    uint64_t spins = 0;
    while (c->mb_host->seq != want) {
        _mm_pause();
        if ((++spins & 0x3fff) == 0) {
            cudaError_t q = cudaStreamQuery(c->compute);
            if (q != cudaSuccess && q != cudaErrorNotReady)
                return fail(c, SPM_ERR_CUDA, "compute stream failed while waiting for the router: %s", cudaGetErrorString(q));
            auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count();
            if (ms > c->deadline_ms)
                return fail(c, SPM_ERR_TIMEOUT, "routing kernel did not report within %d ms", c->deadline_ms);
        }
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    return SPM_OK;
}

// Wait (bounded) until `count` self-tagged mailbox words carry the current launch's tag, then
// return their payloads. The device writes each word as (sequence << 16) | value, so no fence or
// separate flag is involved: a word is either stale (old tag) or complete.
int wait_tagged(spm_ctx* c, const volatile int32_t* words, int count, int32_t* out, const char* what) {
    const uint32_t tag = c->seq & 0xffffu;
    const auto t0 = std::chrono::steady_clock::now();
    uint64_t spins = 0;
    int done = 0;
    while (done < count) {
        const uint32_t wv = uint32_t(words[done]);
        if ((wv >> 16) == tag) { out[done++] = int32_t(wv & 0xffffu); continue; }
        _mm_pause();
        if ((++spins & 0x3fff) == 0) {
            cudaError_t q = cudaStreamQuery(c->compute);
            if (q != cudaSuccess && q != cudaErrorNotReady)
                return fail(c, SPM_ERR_CUDA, "compute stream failed while waiting for the %s: %s", what, cudaGetErrorString(q));
            auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count();
            if (ms > c->deadline_ms)
                return fail(c, SPM_ERR_TIMEOUT, "routing kernel did not deliver the %s within %d ms", what, c->deadline_ms);
        }
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    return SPM_OK;
}

// Read-only streaming probe: every thread folds its 16-byte words into a checksum.
__global__ void __launch_bounds__(512)
read_probe_kernel(const uint4* __restrict__ p, size_t n16, unsigned* sink) {
    unsigned acc = 0;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n16; i += 4 * stride) {      // four independent loads in flight per thread
        const uint4 a = __ldcs(p + i), b = __ldcs(p + i + stride), c2 = __ldcs(p + i + 2 * stride), d = __ldcs(p + i + 3 * stride);
        acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c2.x ^ c2.y ^ c2.z ^ c2.w ^ d.x ^ d.y ^ d.z ^ d.w;
    }
    for (; i < n16; i += stride) { const uint4 a = __ldcs(p + i); acc ^= a.x ^ a.y ^ a.z ^ a.w; }
    if (acc == 0x9e3779b9u) *sink = acc;      // keeps the loads alive; practically never taken
}

// A kernel that only waits: one thread watches %globaltimer until `ns` have passed. Used as the
// stand-in for the omitted attention block and as the extra delay of an emulated slower storage tier.
__global__ void attention_stub_kernel(unsigned long long ns) {
    const unsigned long long t0 = global_timer_ns();
    while (global_timer_ns() - t0 < ns) __nanosleep(200);
}

unsigned char* slot_ptr(spm_ctx* c, int layer, int slot) {
    return c->pools + (size_t(layer) * c->S + slot) * c->blob;
}
const unsigned char* host_blob(spm_ctx* c, int layer, int e) {
    const int k = c->buf.host_store_layers;
    const int src = (k > 0 && k < c->cfg.n_layers) ? layer % k : layer;
    return static_cast<const unsigned char*>(c->buf.host_experts) + (size_t(src) * c->cfg.n_experts + e) * c->blob;
}

// Enqueue one expert transfer on the copy stream. Transfers are issued in batches (the misses of a
// wave, the selections of a prefetch) that are awaited as a whole, so only the last transfer of a
// batch records an event (`lead` = the slot whose event covers the batch): every stream operation
// between two copies costs a few microseconds of link time. With device-side waiting the last
// transfer also bumps the lead slot's arrival counter, which the kernel watches for the whole batch.
int issue_copy(spm_ctx* c, int layer, int e, int slot, size_t lead, bool last_of_batch) {
    const size_t k = size_t(layer) * c->S + slot;
    CU(c, cudaMemcpyAsync(slot_ptr(c, layer, slot), host_blob(c, layer, e), c->blob, cudaMemcpyHostToDevice, c->copy));
    if (c->copy_delay_us > 0) {
        attention_stub_kernel<<<1, 1, 0, c->copy>>>(uint64_t(c->copy_delay_us) * 1000ull);   // emulated slower tier
        CU(c, cudaGetLastError());
    }
    if (last_of_batch) {
        CU(c, cudaEventRecord(c->slot_ev[lead], c->copy));
        if (c->device_wait) {
            // stream-ordered bump of the lead slot's arrival counter, for launches that wait on the device
            StreamWriteValue32Fn wr = stream_write32_fn();
            if (!wr) return fail(c, SPM_ERR_CUDA, "cuStreamWriteValue32 is not available");
            if (c->withhold_arrivals > 0) {
                --c->withhold_arrivals;        // host-side fault injection: the bytes land, the counter never says so
            } else if (wr(reinterpret_cast<CUstream>(c->copy), reinterpret_cast<CUdeviceptr>(c->ws_slot_gen + lead), c->slot_gen_host[lead] + 1, 0) != CUDA_SUCCESS)
                return fail(c, SPM_ERR_CUDA, "cuStreamWriteValue32 failed");
        }
        ++c->slot_gen_host[lead];        // every slot of the batch was given this value as its target below
    }
    c->slot_want[k] = c->slot_gen_host[lead] + (last_of_batch ? 0 : 1);
    c->slot_dep[k] = lead;
    c->slot_pending[k] = 1;
    c->h2d_bytes += c->blob;
    return SPM_OK;
}

// The copy stream may overwrite pool `layer` only after the last kernel that read it.
int order_copy_after_readers(spm_ctx* c, int layer) {
    if (c->pool_free_valid[layer]) CU(c, cudaStreamWaitEvent(c->copy, c->pool_free[layer], 0));
    return SPM_OK;
}

void harvest(spm_ctx* c, Timing& t) {
    const int L = c->cfg.n_layers;
    bool any = false;
    for (int l = 0; l < L; ++l) {
        if (!t.used[l]) continue;
        float a = 0, b = 0;
        cudaEventSynchronize(t.ffn_end[l]);
        if (cudaEventElapsedTime(&a, t.k1_done[l], t.ffn_start[l]) == cudaSuccess) c->layer_stall_us[l] += a * 1e3;
        if (cudaEventElapsedTime(&b, t.ffn_start[l], t.ffn_end[l]) == cudaSuccess) c->layer_ffn_us[l] += b * 1e3;
        t.used[l] = 0;
        any = true;
    }
    if (any) c->timed_steps++;
}

// Read back the in-kernel {first start, last end} pairs written so far and re-arm the slots.
// Slots are handed out in stream order, so the distance from one kernel's end to the next one's
// start is the idle time between them on the device (launch gaps, host turns, waits for copies).
int harvest_clock(spm_ctx* c) {
    if (c->clock_used == 0) return SPM_OK;
    std::vector<unsigned long long> h(size_t(c->clock_used) * 2);
    CU(c, cudaStreamSynchronize(c->compute));
    CU(c, cudaMemcpy(h.data(), c->ws_clock, h.size() * 8, cudaMemcpyDeviceToHost));
    for (int i = 0; i < c->clock_used; ++i) {
        if (h[2 * i + 1] <= h[2 * i]) continue;
        const double us = double(h[2 * i + 1] - h[2 * i]) * 1e-3;
        (c->clock_kind[i] == kClkFfn ? c->window_us : c->clock_kind[i] == kClkRouter ? c->router_window_us : c->reduce_window_us) += us;
        if (i > 0 && h[2 * i - 1] > h[2 * i - 2] && h[2 * i] > h[2 * i - 1]) c->gap_us += double(h[2 * i] - h[2 * i - 1]) * 1e-3;
    }
    for (int i = 0; i < c->clock_used; ++i) { h[2 * i] = ~0ull; h[2 * i + 1] = 0; }
    CU(c, cudaMemcpy(c->ws_clock, h.data(), h.size() * 8, cudaMemcpyHostToDevice));
    c->clock_used = 0;
    return SPM_OK;
}

// Next clock slot for a kernel of the given kind (null when timing is off).
int take_clock(spm_ctx* c, ClockKind kind, unsigned long long** out) {
    *out = nullptr;
    if (!c->timing) return SPM_OK;
    if (c->clock_used == kClockSlots) if (int rc = harvest_clock(c)) return rc;
    c->clock_kind[c->clock_used] = kind;
    *out = c->ws_clock + 2 * size_t(c->clock_used++);
    return SPM_OK;
}

int arm_clock(spm_ctx* c) {   // whole ring to {max, 0}
    std::vector<unsigned long long> h(size_t(kClockSlots) * 2);
    for (int i = 0; i < kClockSlots; ++i) { h[2 * i] = ~0ull; h[2 * i + 1] = 0; }
    CU(c, cudaMemcpy(c->ws_clock, h.data(), h.size() * 8, cudaMemcpyHostToDevice));
    c->clock_used = 0;
    return SPM_OK;
}

void harvest_ring(spm_ctx* c, size_t i) {
    if (!c->ring_used[i]) return;
    float ms = 0;
    cudaEventSynchronize(c->ring_end[i]);
    if (cudaEventElapsedTime(&ms, c->ring_start[i], c->ring_end[i]) == cudaSuccess) c->ring_us += ms * 1e3;
    c->ring_used[i] = 0;
}

// One wave of the batched tensor-core path: sort the (token, k) pairs of this wave's experts by
// expert, upload the wave descriptor, then gather -> grouped tcgen05 FFN -> combine.
int launch_grouped_wave(spm_ctx* c, int layer, const float* x_norm, const int32_t* ids, const float* w, int nb,
                        float* h_inout, const std::vector<int16_t>& slot_of_expert, bool first, bool last,
                        Timing* t, int ring, bool dev_wait) {
    const spm_model_cfg& m = c->cfg;
    const int K = m.top_k;
    const size_t d = c->tc_desc_pos++ % kDescRing;
    if (c->tc_desc_ev_valid[d]) CU(c, cudaEventSynchronize(c->tc_desc_ev[d]));   // staging slot free again
    unsigned char* hd = c->tc_desc_host + d * c->tc_desc_bytes;
    unsigned char* dd = c->tc_desc_dev + d * c->tc_desc_bytes;
    GgUnit* units = reinterpret_cast<GgUnit*>(hd);
    GgRow* rows = reinterpret_cast<GgRow*>(hd + c->tc_off_rows);
    int32_t* rowmap = reinterpret_cast<int32_t*>(hd + c->tc_off_rowmap);
    GgWait* waits = reinterpret_cast<GgWait*>(hd + c->tc_off_wait);
    // Every (token, k) pair of the layer gets a row of its own in the sorted token arrays and in the partial
    // outputs, whatever wave its expert is computed in: the waves append their rows, and one combine after the
    // last wave adds each token's experts in k order. The sum then does not depend on which experts shared a
    // wave, i.e. on the cache state: batched outputs are bit-identical with and without offloading.
    if (first) {
        c->wave_row_off = 0;
        c->wave_rowmap.assign(size_t(nb) * SPM_MAX_TOPK, -1);
    }
    const int off = c->wave_row_off;
    // counting sort of the wave's (token, k) pairs by expert: rows of an expert keep token-major order
    int n_rows = 0, n_units = 0;
    std::vector<int32_t>& row_of = c->plan_first;       // per expert: pairs in this wave, then the next free row of its run
    row_of.assign(size_t(m.n_experts) + 1, 0);
    for (int i = 0; i < nb * K; ++i)
        if (slot_of_expert[ids[i]] >= 0) ++row_of[ids[i] + 1];
    for (int e = 0; e < m.n_experts; ++e) {
        const int cnt = row_of[e + 1];
        row_of[e + 1] = row_of[e] + cnt;
        if (cnt == 0) continue;
        // with device-side waiting a slot whose copy had not landed when the host looked stays pending: the
        // producer warp of its units waits for the batch's arrival counter
        const size_t ks = size_t(layer) * c->S + slot_of_expert[e];
        const GgWait uw = (dev_wait && c->slot_pending[ks]) ? GgWait{int32_t(c->slot_dep[ks]), c->slot_want[ks]} : GgWait{-1, 0u};
        for (int jt = 0; jt < c->n_jt; ++jt) {
            waits[n_units] = uw;
            units[n_units++] = GgUnit{layer * c->S + slot_of_expert[e], jt, off + row_of[e], cnt};
        }
    }
    n_rows = row_of[m.n_experts];
    for (int tk = 0; tk < nb; ++tk)
        for (int k = 0; k < K; ++k) {
            const int e = ids[tk * K + k];
            if (slot_of_expert[e] < 0) continue;
            const int r = row_of[e]++;
            c->wave_rowmap[tk * SPM_MAX_TOPK + k] = off + r;
            rows[r] = GgRow{tk, k};
        }
    if (off + n_rows > c->rows_cap) return fail(c, SPM_ERR_STATE, "token rows of a layer exceed the workspace");
    std::memcpy(rowmap, c->wave_rowmap.data(), size_t(nb) * SPM_MAX_TOPK * sizeof(int32_t));
    c->wave_row_off = off + n_rows;
    if (n_units == 0 && !last) return SPM_OK;
    const bool q4 = m.dtype == SPM_DTYPE_Q4;
    if (!q4) {
        // bf16 kernel: phase-2 chunks, finer towards the end, so that every SM streams until the launch ends
        gg_plan_chunks(n_units, m.hidden / kGgTileRows, c->num_sms, c->plan_chunks);
        if (c->plan_chunks.size() > c->tc_chunk_cap) return fail(c, SPM_ERR_STATE, "grouped-kernel chunk list exceeds its buffer");
        std::memcpy(hd + c->tc_off_chunks, c->plan_chunks.data(), c->plan_chunks.size() * sizeof(GgTaskHost));
    }
    CU(c, cudaMemcpyAsync(dd, hd, c->tc_desc_bytes, cudaMemcpyHostToDevice, c->compute));
    CU(c, cudaEventRecord(c->tc_desc_ev[d], c->compute));
    c->tc_desc_ev_valid[d] = 1;
    // (all three kernels of a wave are launched so that their preambles may overlap their predecessor's tail)
    CU(c, launch_k(gg_gather_kernel, dim3(std::max(n_rows, 1)), dim3(128), 0, c->compute, true, x_norm, w,
                   reinterpret_cast<const GgRow*>(dd + c->tc_off_rows), n_rows, (const int*)nullptr, m.hidden, K,
                   c->tc_xs + size_t(off) * m.hidden, c->tc_wrow + off,
                   q4 ? 1 : 0, q4 ? (int*)nullptr : c->tc_ready, q4 ? 0 : n_units + 1));
    if (t && first) CU(c, cudaEventRecord(t->ffn_start[layer], c->compute));
    if (ring >= 0 && first) CU(c, cudaEventRecord(c->ring_start[ring], c->compute));
    GgArgs a{reinterpret_cast<const GgUnit*>(dd), n_units, nullptr, c->tc_wrow, c->tc_partial, c->rows_cap, m.hidden, m.inter, c->ws_status, c->wait_limit_ns,
             nullptr, 0, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    if (int rc = take_clock(c, kClkFfn, &a.clock)) return rc;
    if (dev_wait) {
        a.unit_wait = reinterpret_cast<const GgWait*>(dd + c->tc_off_wait);
        a.ready = c->ws_slot_gen;
    }
    if (n_units == 0) {
        // (nothing to compute in this wave; the combine below still closes the layer)
    } else if (q4) {
        CU(c, launch_k(ffn_grouped_q4_kernel, dim3(std::min(c->num_sms, n_units)), dim3(kQgThreads), ffn_grouped_q4_smem(), c->compute, true,
                       c->qmapn, c->qmapsc, c->xmaps, a));
    } else {
        a.chunks = reinterpret_cast<const GgTask*>(dd + c->tc_off_chunks);
        a.n_chunks = int(c->plan_chunks.size());
        a.next_chunk = c->tc_ready;
        a.act_ready = c->tc_ready + 1;
        a.act_g = c->tc_act;
        // every SM takes part: CTAs without a unit of their own still run phase-2 chunks
        CU(c, launch_k(ffn_grouped_kernel, dim3(c->num_sms), dim3(kGgThreads), ffn_grouped_smem(), c->compute, true, c->wmap, c->xmaps, a));
    }
    if (t && last) CU(c, cudaEventRecord(t->ffn_end[layer], c->compute));
    if (ring >= 0 && last) { CU(c, cudaEventRecord(c->ring_end[ring], c->compute)); c->ring_used[ring] = 1; }
    if (last)
        CU(c, launch_k(gg_combine_kernel, gg_combine_grid(m.hidden, nb), gg_combine_block(K), 0, c->compute, true,
                       (const float*)c->tc_partial, reinterpret_cast<const int32_t*>(dd + c->tc_off_rowmap), K, c->n_jt, c->rows_cap, m.hidden, h_inout));
    c->kernel_launches += last ? 3 : 2;
    c->ffn_launches++;
    c->tc_launches++;
    return SPM_OK;
}

// Demand resolution, on-demand copies, stream waits and FFN launches of one layer.
// `t` (may be null) receives the timing events of this layer; `ring` >= 0 selects an event pair
// of the stand-alone timing ring instead.
// With `launch` false only the slot table's side runs (the kernels of a host-free step were
// enqueued earlier); a miss there would mean the step computed with a stale slot map.
// With `leave_partial` the partial rows of the last wave stay in the workspace for the next
// layer's routing kernel to fold into the hidden row (GEMV path only; reported through *left).
int run_ffn(spm_ctx* c, int layer, const float* x_norm, const int32_t* ids, const float* w, int nb,
            float* h_inout, Timing* t, int ring = -1, bool launch = true, bool leave_partial = false, bool* left = nullptr) {
    const spm_model_cfg& m = c->cfg;
    const int K = m.top_k;
    SlotTable& tb = *c->table;

    c->need.clear();
    for (int i = 0; i < nb * K; ++i) {
        if (ids[i] < 0 || ids[i] >= m.n_experts) return fail(c, SPM_ERR_INVALID_ARG, "expert id %d out of range", ids[i]);
        c->need.push_back(ids[i]);
    }
    if (layer >= 1) {   // logical ReadyRecall: needed experts that already have a slot
        for (int tk = 0; tk < nb; ++tk) {
            int have = 0;
            for (int k = 0; k < K; ++k) have += tb.slot_of(layer, ids[tk * K + k]) >= 0;
            c->ready_sum += double(have) / K;
            c->ready_count++;
        }
    }
    int n_waves = 1;
    tb.demand(layer, c->need.data(), int(c->need.size()), c->placements, &n_waves);
    if (!launch) {
        for (const Placement& p : c->placements)
            if (p.missed) return fail(c, SPM_ERR_STATE, "host-free step met a non-resident expert (layer %d, expert %d)", layer, p.expert);
        return SPM_OK;
    }

    const int G = ffn_grid_for(c, nb);
    const bool use_tc = nb > 1 && c->tc_ok && c->batched_path == 0;
    // kernels that can wait for a copy themselves: the batch-1 GEMV kernels and the grouped tensor-core kernels
    const bool dev_wait = c->device_wait && (nb == 1 || use_tc) && stream_write32_fn() != nullptr;
    std::vector<int16_t>& slot_of_expert = c->wave_slot;   // experts computed in the current wave
    for (int wave = 0; wave < n_waves; ++wave) {
        slot_of_expert.assign(m.n_experts, -1);
        int n_missed = 0, last_missed = -1;
        for (size_t i = 0; i < c->placements.size(); ++i) {
            const Placement& p = c->placements[i];
            if (p.wave != wave) continue;
            slot_of_expert[p.expert] = int16_t(p.slot);
            if (p.missed) { ++n_missed; last_missed = int(i); }
        }
        if (n_missed > 0) {
            if (int rc = order_copy_after_readers(c, layer)) return rc;
            if (wave > 0) CU(c, cudaStreamWaitEvent(c->copy, c->wave_done, 0));
            const size_t lead = size_t(layer) * c->S + c->placements[last_missed].slot;
            for (size_t i = 0; i < c->placements.size(); ++i) {
                const Placement& p = c->placements[i];
                if (p.wave != wave || !p.missed) continue;
                if (int rc = issue_copy(c, layer, p.expert, p.slot, lead, int(i) == last_missed)) return rc;
            }
        }
        for (size_t i = 0; i < c->placements.size(); ++i) {
            const Placement& p = c->placements[i];
            if (p.wave != wave) continue;
            const size_t k = size_t(layer) * c->S + p.slot;
            if (!c->slot_pending[k]) continue;
            const size_t dep = c->slot_dep[k];       // (an event re-recorded by a later batch only waits longer)
            cudaError_t q = cudaEventQuery(c->slot_ev[dep]);
            if (q == cudaErrorNotReady) {
                if (!p.missed) c->extra_late++;
                if (dev_wait) continue;      // the kernel itself waits for this slot; it stays pending for later launches
                CU(c, cudaStreamWaitEvent(c->compute, c->slot_ev[dep], 0));
            } else if (q != cudaSuccess) {
                return fail(c, SPM_ERR_CUDA, "copy event query: %s", cudaGetErrorString(q));
            }
            c->slot_pending[k] = 0;
        }

        const bool first = wave == 0, last = wave == n_waves - 1;
        unsigned long long* clock_slot = nullptr;
        if (!use_tc) if (int rc = take_clock(c, kClkFfn, &clock_slot)) return rc;
        auto fill = [&](auto& a) {
            a.pool = slot_ptr(c, layer, 0);
            a.shared = m.n_shared ? static_cast<const unsigned char*>(c->buf.shared_experts) + size_t(layer) * m.n_shared * c->blob : nullptr;
            a.x = x_norm;
            a.w = w;
            a.partial = c->ws_partial;
            a.status = c->ws_status;
            a.clock = clock_slot;
            a.ready = dev_wait ? c->ws_slot_gen + size_t(layer) * c->S : nullptr;
            a.wait_limit_ns = c->wait_limit_ns;
            a.early = 1;               // slot numbers are launch arguments: the first weight copies need not wait for the preceding kernel
            a.blob_bytes = c->blob;
            a.I = m.inter; a.K = K; a.n_slots = c->S; a.n_shared = m.n_shared;
            for (int tk = 0; tk < nb; ++tk) {
                int cnt = 0;
                for (int k = 0; k < K; ++k) {
                    const int s = slot_of_expert[ids[tk * K + k]];
                    if (s < 0) continue;
                    a.code[tk * SPM_MAX_TOPK + cnt] = short(s);
                    a.kidx[tk * SPM_MAX_TOPK + cnt] = (unsigned char)k;
                    if (dev_wait) {
                        const size_t ks = size_t(layer) * c->S + s;
                        a.want[cnt] = c->slot_want[ks];
                        a.watch[cnt] = short(c->slot_dep[ks] - size_t(layer) * c->S);
                    }
                    ++cnt;
                }
                if (first)
                    for (int s = 0; s < m.n_shared; ++s) {
                        a.code[tk * SPM_MAX_TOPK + cnt] = short(-1 - s);
                        a.kidx[tk * SPM_MAX_TOPK + cnt] = 255;
                        ++cnt;
                    }
                a.count[tk] = (unsigned char)cnt;
            }
        };
        if (use_tc) {
            if (int rc = launch_grouped_wave(c, layer, x_norm, ids, w, nb, h_inout, slot_of_expert, first, last, t, ring, dev_wait)) return rc;
        } else {
            if (t && first) CU(c, cudaEventRecord(t->ffn_start[layer], c->compute));
            if (ring >= 0 && first) CU(c, cudaEventRecord(c->ring_start[ring], c->compute));
            if (nb == 1) {
                FfnArgs<1> a{};
                fill(a);
                CU(c, launch_gemv<1>(c, a, G, nb, true));
            } else {
                FfnArgs<SPM_MAX_BATCH> a{};
                fill(a);
                CU(c, launch_gemv<SPM_MAX_BATCH>(c, a, G, nb, true));
            }
            if (t && last) CU(c, cudaEventRecord(t->ffn_end[layer], c->compute));
            if (ring >= 0 && last) { CU(c, cudaEventRecord(c->ring_end[ring], c->compute)); c->ring_used[ring] = 1; }
            if (last && leave_partial) {
                if (left) *left = true;
                c->kernel_launches += 1;
            } else {
                unsigned long long* reduce_clock = nullptr;
                if (int rc = take_clock(c, kClkReduce, &reduce_clock)) return rc;
                CU(c, launch_k(ffn_reduce_kernel, dim3((m.hidden + kReduceCols - 1) / kReduceCols, nb), dim3(kReduceCols * kReduceGroups), 0,
                               c->compute, true, (const float*)c->ws_partial, (const float*)h_inout, h_inout, G, m.hidden, reduce_clock));
                c->kernel_launches += 2;
            }
            c->ffn_launches++;
        }
        if (!last) CU(c, cudaEventRecord(c->wave_done, c->compute));
    }
    CU(c, cudaEventRecord(c->pool_free[layer], c->compute));
    c->pool_free_valid[layer] = 1;
    if (t) t->used[layer] = 1;
    return SPM_OK;
}

int do_prefetch(spm_ctx* c, int target, const int32_t* ids, int count, const int32_t* protect, int n_protect,
                int* out_issued) {
    SlotTable& tb = *c->table;
    c->slots_tmp.assign(size_t(std::max(count, 1)), -1);
    const int issued = tb.prefetch(target, ids, count, protect, n_protect, c->drop_modulo, c->slots_tmp.data());
    if (issued > 0) {
        if (int rc = order_copy_after_readers(c, target)) return rc;
        int last = -1;
        for (int i = 0; i < count; ++i) if (c->slots_tmp[i] >= 0) last = i;
        const size_t lead = size_t(target) * c->S + c->slots_tmp[last];
        for (int i = 0; i < count; ++i)
            if (c->slots_tmp[i] >= 0)
                if (int rc = issue_copy(c, target, ids[i], c->slots_tmp[i], lead, i == last)) return rc;
    }
    if (out_issued) *out_issued = issued;
    return SPM_OK;
}

// Experts of this step's routing at one layer, ranked by sum over tokens of (K - rank position).
void borda_rank(const int32_t* ids, int nb, int K, int n, std::vector<int32_t>& out) {
    std::vector<int32_t> score(n, 0);
    for (int t = 0; t < nb; ++t)
        for (int k = 0; k < K; ++k) score[ids[t * K + k]] += K - k;
    out.clear();
    for (int e = 0; e < n; ++e) if (score[e] > 0) out.push_back(e);
    std::stable_sort(out.begin(), out.end(), [&](int32_t x, int32_t y) { return score[x] > score[y]; });
}


// The layers of one decode step. With `trace` null the kernels are launched and the routing results
// awaited layer by layer; with a trace (the mailboxes a host-free step filled) only the host side
// runs: accounting, slot-table updates, selection — the same calls in the same order.
int step_layers(spm_ctx* c, float* h_out, int nb, Timing* t, const Mailbox* trace) {
    const spm_model_cfg& m = c->cfg;
    const int L = m.n_layers, K = m.top_k, n = m.n_experts;
    SlotTable& tb = *c->table;
    const bool predict = c->policy == SPM_POLICY_ADAPTER || c->policy == SPM_POLICY_PRED0;
    c->prev_order_valid = false;
    std::vector<int32_t> ids(size_t(nb) * K);
    std::vector<int32_t> this_rank;
    // The routing kernel of layer l + 1 depends only on layer l's kernels, so it is enqueued as soon as
    // they are and before the host plans and issues layer l + 1's prefetch (several driver calls):
    // the device never waits for that host work. The mailbox words of layer l are read before.
    bool partial_left = false;       // the preceding layer's partial rows are still to be folded into the hidden row
    auto enqueue_router = [&](int l) -> int {
        if (c->stub_us > 0) {
            attention_stub_kernel<<<1, 1, 0, c->compute>>>(uint64_t(c->stub_us) * 1000ull);
            CU(c, cudaGetLastError());
            c->kernel_launches++;
        }
        RouterRoute fold{c->mb_dev, nullptr, nullptr, false, c->ws_partial, ffn_grid_for(c, nb)};
        if (int rc = launch_router(c, l, h_out, nullptr, nb, c->ws_x, nullptr, true, predict && l <= L - 2,
                                   partial_left ? &fold : nullptr, false)) return rc;
        partial_left = false;
        if (t) CU(c, cudaEventRecord(t->k1_done[l], c->compute));
        return SPM_OK;
    };
    // GEMV path: only the last layer runs the combine kernel, the others leave it to the next routing kernel
    const bool gemv_path = !(nb > 1 && c->tc_ok && c->batched_path == 0);
    if (!trace) if (int rc = enqueue_router(0)) return rc;
    for (int l = 0; l < L; ++l) {
        const bool has_adapter = l <= L - 2;
        if (!trace) {
            if (int rc = wait_tagged(c, c->mb_host->ids, nb * K, ids.data(), "expert ids")) return rc;
        } else {
            for (int i = 0; i < nb * K; ++i) ids[i] = trace[l].ids[i] & 0xffff;
        }

        if (c->prev_order_valid) {   // ExpertRecall@M of the previous layer's prediction, M = budget
            const int M = std::min(c->budget, n);
            for (int tk = 0; tk < nb; ++tk) {
                int hit = 0;
                for (int k = 0; k < K; ++k)
                    for (int q = 0; q < M; ++q) hit += c->prev_order[q] == ids[tk * K + k];
                c->recall_sum += double(hit) / K;
                c->recall_count++;
                const int Ms[3] = {std::max(1, K / 2), K, K + 2};      // the coverage levels the paper tabulates
                for (int j = 0; j < 3; ++j) {
                    int h2 = 0;
                    const int Mj = std::min(Ms[j], n);
                    for (int k = 0; k < K; ++k)
                        for (int q = 0; q < Mj; ++q) h2 += c->prev_order[q] == ids[tk * K + k];
                    c->recall_at[j] += double(h2) / K;
                }
            }
        }
        if (int rc = run_ffn(c, l, c->ws_x, ids.data(), c->ws_w, nb, h_out, t, -1, trace == nullptr,
                             gemv_path && l + 1 < L && c->stub_us == 0, &partial_left)) return rc;
        if (c->policy == SPM_POLICY_NAIVE) borda_rank(ids.data(), nb, K, n, this_rank);

        c->prev_order_valid = false;
        const bool reads_order = has_adapter && (c->policy == SPM_POLICY_ADAPTER || c->policy == SPM_POLICY_PRED0);
        if (!trace && !reads_order && l + 1 < L) {       // nothing left to read from layer l's mailbox
            if (int rc = enqueue_router(l + 1)) return rc;
        }
        if (has_adapter && c->policy != SPM_POLICY_ON_DEMAND) {
            const int32_t* ranking;
            int n_ranked;
            bool protect_all = false;
            if (c->policy == SPM_POLICY_HINT_TRACE) {
                const size_t cell = size_t(tb.step()) * L + (l + 1);
                ranking = c->hint.data() + cell * c->hint_stride;
                n_ranked = c->hint_count[cell];
                protect_all = true;
            } else if (c->policy == SPM_POLICY_NAIVE) {
                ranking = c->prev_rank[l + 1].data();      // what the preceding step used at layer l+1
                n_ranked = int(c->prev_rank[l + 1].size());
            } else {
                c->prev_order.resize(n);
                if (!trace) {
                    if (int rc = wait_tagged(c, c->mb_host->order, n, c->prev_order.data(), "expert ranking")) return rc;
                    if (int rc = enqueue_router(l + 1)) return rc;      // has_adapter: layer l + 1 exists
                } else {
                    for (int e = 0; e < n; ++e) c->prev_order[e] = trace[l].order[e] & 0xffff;
                }
                c->prev_order_valid = true;
                ranking = c->prev_order.data();
                n_ranked = n;
            }
            tb.plan(l + 1, ranking, n_ranked, c->budget, protect_all, c->sel, c->protect);
            if (c->policy == SPM_POLICY_PRED0) {
                tb.plan_only(l + 1, c->sel.data(), int(c->sel.size()));
            } else {
                if (int rc = do_prefetch(c, l + 1, c->sel.data(), int(c->sel.size()), c->protect.data(),
                                         int(c->protect.size()), nullptr)) return rc;
            }
        }
        if (c->policy == SPM_POLICY_NAIVE) c->prev_rank[l] = this_rank;
    }
    tb.end_step();
    tb.stats().steps++;
    c->tokens += nb;
    return SPM_OK;
}

// ---- host-free steps ---------------------------------------------------------
// Replay the bookkeeping of the oldest enqueued host-free step (waits for its kernels).
int replay_oldest(spm_ctx* c) {
    const auto [slot, nb] = c->tr_pending.front();
    CU(c, cudaEventSynchronize(c->tr_ev[slot]));
    c->tr_pending.pop_front();
    return step_layers(c, nullptr, nb, nullptr, c->tr_host + size_t(slot) * c->cfg.n_layers);
}

int flush_trace(spm_ctx* c) {
    while (!c->tr_pending.empty())
        if (int rc = replay_oldest(c)) return rc;
    return SPM_OK;
}

// A step may skip the host when no routing result can change what the host would do: every expert
// of every layer holds a slot and every copy has landed, so any demand is a hit and no selection
// finds a candidate. On the batched tensor-core path the wave plan is then built by a kernel.
int host_free_ready(spm_ctx* c, int nb, bool* out) {
    const spm_model_cfg& m = c->cfg;
    *out = false;
    if (!c->host_free || c->S < m.n_experts) return SPM_OK;
    if (!c->fast_ready) {
        SlotTable& tb = *c->table;
        for (int l = 0; l < m.n_layers; ++l)
            for (int e = 0; e < m.n_experts; ++e)
                if (tb.slot_of(l, e) < 0) return SPM_OK;
        for (size_t k = 0; k < c->slot_pending.size(); ++k)
            if (c->slot_pending[k]) {
                CU(c, cudaStreamWaitEvent(c->compute, c->slot_ev[c->slot_dep[k]], 0));
                c->slot_pending[k] = 0;
            }
        std::vector<short> map(size_t(m.n_layers) * m.n_experts);
        for (int l = 0; l < m.n_layers; ++l)
            for (int e = 0; e < m.n_experts; ++e) map[size_t(l) * m.n_experts + e] = short(tb.slot_of(l, e));
        CU(c, cudaMemcpyAsync(c->ws_slot_map, map.data(), map.size() * sizeof(short), cudaMemcpyHostToDevice, c->compute));
        CU(c, cudaStreamSynchronize(c->compute));      // `map` is a temporary
        c->fast_ready = true;
    }
    *out = true;
    return SPM_OK;
}

// The kernels of all layers of one host-free step, enqueued on the compute stream (or captured).
int enqueue_host_free_layers(spm_ctx* c, int nb, float* h_out, int slot, bool predict) {
    const spm_model_cfg& m = c->cfg;
    const int L = m.n_layers, K = m.top_k, n = m.n_experts;
    const int G = ffn_grid_for(c, nb);
    for (int l = 0; l < L; ++l) {
        if (c->stub_us > 0) {
            attention_stub_kernel<<<1, 1, 0, c->compute>>>(uint64_t(c->stub_us) * 1000ull);
            CU(c, cudaGetLastError());
            c->kernel_launches++;
        }
        short* codes = c->ws_codes + size_t(l) * m.max_batch * SPM_MAX_TOPK;
        // On the GEMV path the routing kernel of layer l + 1 also folds layer l's partial rows into the
        // hidden row, so only the last layer needs the combine kernel.
        const bool use_tc = nb > 1 && c->tc_ok && c->batched_path == 0;
        const bool fold = !use_tc && l > 0 && c->stub_us == 0;
        RouterRoute route{c->tr_dev + size_t(slot) * L + l, c->ws_slot_map + size_t(l) * n, codes, true,
                          fold ? c->ws_partial : nullptr, G};
        if (int rc = launch_router(c, l, h_out, nullptr, nb, c->ws_x, nullptr, true, predict && l <= L - 2, &route, false)) return rc;
        unsigned long long* clock_slot = nullptr;
        if (int rc = take_clock(c, kClkFfn, &clock_slot)) return rc;
        auto fill = [&](auto& a) {
            a.pool = slot_ptr(c, l, 0);
            a.shared = m.n_shared ? static_cast<const unsigned char*>(c->buf.shared_experts) + size_t(l) * m.n_shared * c->blob : nullptr;
            a.x = c->ws_x;
            a.w = c->ws_w;
            a.partial = c->ws_partial;
            a.status = c->ws_status;
            a.clock = clock_slot;
            a.ready = nullptr;
            a.wait_limit_ns = c->wait_limit_ns;
            a.dev_code = codes;
            a.blob_bytes = c->blob;
            a.I = m.inter; a.K = K; a.n_slots = c->S; a.n_shared = m.n_shared;
            for (int tk = 0; tk < nb; ++tk) a.count[tk] = (unsigned char)(K + m.n_shared);   // launch shape only
        };
        if (use_tc) {
            // wave plan on the device, then gather -> grouped tcgen05 FFN -> combine
            unsigned char* dd = c->tc_desc_dev;        // stream-ordered reuse of the first descriptor slot
            GgUnit* units = reinterpret_cast<GgUnit*>(dd);
            GgRow* rows = reinterpret_cast<GgRow*>(dd + c->tc_off_rows);
            int32_t* rowmap = reinterpret_cast<int32_t*>(dd + c->tc_off_rowmap);
            CU(c, launch_k(gg_plan_kernel, dim3(1), dim3(kGgPlanThreads), gg_plan_smem(n), c->compute, true,
                           (const int32_t*)c->ws_ids, (const short*)(c->ws_slot_map + size_t(l) * n), l * c->S, nb, K, n, c->n_jt,
                           units, rows, rowmap, c->tc_counts, c->ws_status));
            CU(c, launch_k(gg_gather_kernel, dim3(nb * K), dim3(128), 0, c->compute, true, (const float*)c->ws_x, (const float*)c->ws_w,
                           (const GgRow*)rows, 0, (const int*)(c->tc_counts + 1), m.hidden, K, c->tc_xs, c->tc_wrow,
                           m.dtype == SPM_DTYPE_Q4 ? 1 : 0, m.dtype == SPM_DTYPE_Q4 ? (int*)nullptr : c->tc_ready,
                           m.dtype == SPM_DTYPE_Q4 ? 0 : c->max_units + 1));
            // (no chunk list here: the plan is built on the device, a chunk is a whole unit)
            GgArgs ga{units, 0, c->tc_counts, c->tc_wrow, c->tc_partial, c->rows_cap, m.hidden, m.inter, c->ws_status, c->wait_limit_ns,
                      nullptr, 0, c->tc_ready, c->tc_act, c->tc_ready + 1, clock_slot};
            if (m.dtype == SPM_DTYPE_Q4)
                CU(c, launch_k(ffn_grouped_q4_kernel, dim3(c->num_sms), dim3(kQgThreads), ffn_grouped_q4_smem(), c->compute, true,
                               c->qmapn, c->qmapsc, c->xmaps, ga));
            else
                CU(c, launch_k(ffn_grouped_kernel, dim3(c->num_sms), dim3(kGgThreads), ffn_grouped_smem(), c->compute, true, c->wmap, c->xmaps, ga));
            CU(c, launch_k(gg_combine_kernel, gg_combine_grid(m.hidden, nb), gg_combine_block(K), 0, c->compute, true,
                           (const float*)c->tc_partial, (const int32_t*)rowmap, K, c->n_jt, c->rows_cap, m.hidden, h_out));
            c->kernel_launches += 5;
            c->ffn_launches++;
            c->tc_launches++;
            continue;
        }
        if (nb == 1) {
            FfnArgs<1> a{};
            fill(a);
            CU(c, launch_gemv<1>(c, a, G, nb, true));
        } else {
            FfnArgs<SPM_MAX_BATCH> a{};
            fill(a);
            CU(c, launch_gemv<SPM_MAX_BATCH>(c, a, G, nb, true));
        }
        if (l == L - 1 || c->stub_us > 0) {
            unsigned long long* reduce_clock = nullptr;
            if (int rc = take_clock(c, kClkReduce, &reduce_clock)) return rc;
            CU(c, launch_k(ffn_reduce_kernel, dim3((m.hidden + kReduceCols - 1) / kReduceCols, nb), dim3(kReduceCols * kReduceGroups), 0,
                           c->compute, true, (const float*)c->ws_partial, (const float*)h_out, h_out, G, m.hidden, reduce_clock));
            c->kernel_launches++;
        }
        c->kernel_launches += 2;
        c->ffn_launches++;
    }
    return SPM_OK;
}

// A host-free step is the same sequence of launches every time (for a given trace slot, batch size,
// output buffer, prediction on/off and launch geometry), so it is captured once into a CUDA graph
// and replayed: one submission instead of 2-5 per layer. Steps with timing or an attention
// stand-in are enqueued launch by launch.
int enqueue_host_free_step(spm_ctx* c, const float* h_in, int nb, float* h_out) {
    const spm_model_cfg& m = c->cfg;
    if (int(c->tr_pending.size()) == kTraceRing)
        if (int rc = replay_oldest(c)) return rc;
    const int slot = int(c->tr_count++ % kTraceRing);
    if (h_out != h_in)
        CU(c, cudaMemcpyAsync(h_out, h_in, size_t(nb) * m.hidden * 4, cudaMemcpyDeviceToDevice, c->compute));
    const bool predict = c->policy == SPM_POLICY_ADAPTER || c->policy == SPM_POLICY_PRED0;
    bool done = false;
    if (c->graph_replay && !c->timing && c->stub_us == 0) {
        const int G = ffn_grid_for(c, nb);
        spm_ctx::HostFreeGraph* g = nullptr;
        for (auto& x : c->hf_graphs)
            if (x.slot == slot && x.nb == nb && x.h_out == h_out && x.predict == predict && x.G == G && x.batched_path == c->batched_path) g = &x;
        if (!g && c->hf_warm && c->hf_graphs.size() < 64) {
            // (the first host-free step ran launch by launch, so every kernel attribute is already set)
            spm_ctx::HostFreeGraph ng{slot, nb, h_out, predict, G, c->batched_path, 0, 0, 0, nullptr};
            const uint64_t k0 = c->kernel_launches, f0 = c->ffn_launches, t0 = c->tc_launches;
            cudaGraph_t graph = nullptr;
            int rc = SPM_ERR_CUDA;
            cudaError_t ce = cudaStreamBeginCapture(c->compute, cudaStreamCaptureModeRelaxed);   // (fails on the legacy default stream)
            if (ce == cudaSuccess) {
                rc = enqueue_host_free_layers(c, nb, h_out, slot, predict);
                ce = cudaStreamEndCapture(c->compute, &graph);
            }
            ng.kernels = c->kernel_launches - k0; ng.ffns = c->ffn_launches - f0; ng.tcs = c->tc_launches - t0;
            c->kernel_launches = k0; c->ffn_launches = f0; c->tc_launches = t0;
            if (rc == SPM_OK && ce == cudaSuccess && graph && cudaGraphInstantiate(&ng.exec, graph, 0) == cudaSuccess) {
                c->hf_graphs.push_back(ng);
                g = &c->hf_graphs.back();
            } else {
                cudaGetLastError();
                c->graph_replay = false;       // capture is not possible here: keep enqueueing launch by launch
            }
            if (graph) cudaGraphDestroy(graph);
        }
        if (g) {
            CU(c, cudaGraphLaunch(g->exec, c->compute));
            c->kernel_launches += g->kernels; c->ffn_launches += g->ffns; c->tc_launches += g->tcs;
            done = true;
        }
    }
    if (!done) {
        if (int rc = enqueue_host_free_layers(c, nb, h_out, slot, predict)) return rc;
        c->hf_warm = true;
    }
    CU(c, cudaEventRecord(c->tr_ev[slot], c->compute));
    c->tr_pending.emplace_back(slot, nb);
    c->host_free_steps++;
    // bookkeeping of steps whose kernels have already finished, while the device works on this one
    while (!c->tr_pending.empty() && cudaEventQuery(c->tr_ev[c->tr_pending.front().first]) == cudaSuccess)
        if (int rc = replay_oldest(c)) return rc;
    return SPM_OK;
}

int check_layer(spm_ctx* c, int layer, int nb) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, SPM_ERR_INVALID_ARG, "layer %d out of range", layer);
    if (nb < 1 || nb > c->cfg.max_batch) return fail(c, SPM_ERR_INVALID_ARG, "nb %d out of range (max_batch %d)", nb, c->cfg.max_batch);
    return SPM_OK;
}

int check_status(spm_ctx* c) {
    int st = 0;
    CU(c, cudaMemcpy(&st, c->ws_status, sizeof st, cudaMemcpyDeviceToHost));
    if (st == 0) return SPM_OK;
    CU(c, cudaMemset(c->ws_status, 0, sizeof st));      // reported once; the context stays usable
    if (st & kStatusCopyTimeout) return fail(c, SPM_ERR_TIMEOUT, "expert FFN kernel gave up waiting for a weight copy");
    if (st & kStatusBadSlot) return fail(c, SPM_ERR_NOT_RESIDENT, "expert FFN kernel received a slot number outside the pool");
    if (st & kStatusGroupedTimeout) return fail(c, SPM_ERR_TIMEOUT, "grouped expert FFN kernel gave up waiting on a pipeline barrier");
    if (st & kStatusNonFinite) return fail(c, SPM_ERR_NUMERIC, "a routing kernel met a non-finite logit (NaN or Inf in the hidden rows or the weights)");
    return SPM_OK;
}

}  // namespace

namespace spm {
// lets other translation units of the library leave a message for spm_last_error(NULL)
void set_thread_error(const std::string& msg) { g_init_error = msg; }
}  // namespace spm

// ============================================================================
extern "C" {

int spm_expert_blob_bytes(const spm_model_cfg* cfg, size_t* bytes) {
    if (!cfg || !bytes) return SPM_ERR_INVALID_ARG;
    *bytes = blob_bytes_of(cfg);
    return SPM_OK;
}

int spm_query_arena(const spm_model_cfg* cfg, int slots_per_layer, size_t* bytes) {
    if (!bytes) return SPM_ERR_INVALID_ARG;
    if (int rc = check_cfg(cfg, slots_per_layer, nullptr)) return rc;
    *bytes = layout_of(cfg, slots_per_layer).total;
    return SPM_OK;
}

const char* spm_last_error(const spm_ctx* ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

int spm_init(const spm_model_cfg* cfg, int slots_per_layer, int budget, const spm_buffers* b, spm_ctx** out) {
    if (!out || !b) return fail(nullptr, SPM_ERR_INVALID_ARG, "null argument");
    *out = nullptr;
    if (int rc = check_cfg(cfg, slots_per_layer, nullptr)) return rc;
    if (budget < -1) return fail(nullptr, SPM_ERR_INVALID_ARG, "budget %d", budget);
    if (!b->rms_gamma || !b->router_w || !b->host_experts || !b->arena) return fail(nullptr, SPM_ERR_INVALID_ARG, "a required buffer is null");
    if (cfg->n_layers > 1 && (!b->adapter_a || !b->adapter_b)) return fail(nullptr, SPM_ERR_INVALID_ARG, "adapter buffers are null");
    if (cfg->n_shared > 0 && !b->shared_experts) return fail(nullptr, SPM_ERR_INVALID_ARG, "shared_experts is null");
    if (b->compute_stream == b->copy_stream) return fail(nullptr, SPM_ERR_INVALID_ARG, "compute and copy stream must differ");
    if (b->host_store_layers < 0 || b->host_store_layers > cfg->n_layers) return fail(nullptr, SPM_ERR_INVALID_ARG, "host_store_layers out of range");
    if (reinterpret_cast<uintptr_t>(b->arena) % 256) return fail(nullptr, SPM_ERR_INVALID_ARG, "arena must be 256-byte aligned");
    const Layout lay = layout_of(cfg, slots_per_layer);
    if (b->arena_bytes < lay.total) return fail(nullptr, SPM_ERR_INVALID_ARG, "arena too small: %zu < %zu", b->arena_bytes, lay.total);

    int dev_count = 0;
    cudaError_t e = cudaGetDeviceCount(&dev_count);
    if (e != cudaSuccess || dev_count == 0)
        return fail(nullptr, SPM_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(e));

    spm_ctx* c = new spm_ctx();
    c->cfg = *cfg;
    c->S = slots_per_layer;
    c->buf = *b;
    c->compute = static_cast<cudaStream_t>(b->compute_stream);
    c->copy = static_cast<cudaStream_t>(b->copy_stream);
    c->elem = cfg->dtype == SPM_DTYPE_FP32 ? 4 : 2;       // router / adapter element size
    c->blob = blob_bytes_of(cfg);
    c->row_bytes = c->blob / size_t(cfg->inter);
    c->nseg = cfg->hidden / (cfg->dtype == SPM_DTYPE_FP32 ? 128 : 256);
    c->depth = int((kFfnSmemLimit - 1024) / (4 * c->row_bytes));   // ring depth with the fewest warps
    auto bail = [&](int rc) { g_init_error = c->err; spm_destroy(c); return rc; };
    if (c->depth < 1) { c->err = "hidden too large for the shared-memory ring"; return bail(SPM_ERR_CONFIG); }
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceProp prop{};
    if (cudaGetDeviceProperties(&prop, dev) == cudaSuccess) c->num_sms = prop.multiProcessorCount;
    if (prop.major != 10) { c->err = "this library is built for sm_100a (B200) only"; return bail(SPM_ERR_CONFIG); }

    unsigned char* base = static_cast<unsigned char*>(b->arena);
    c->pools = base + lay.pools;
    c->ws_slot_gen = reinterpret_cast<unsigned*>(base + lay.slot_gen);
    c->ws_x = reinterpret_cast<float*>(base + lay.x);
    c->ws_logits = reinterpret_cast<float*>(base + lay.logits);
    c->ws_pihat = reinterpret_cast<float*>(base + lay.pihat);
    c->ws_w = reinterpret_cast<float*>(base + lay.w);
    c->ws_scores = reinterpret_cast<float*>(base + lay.scores);
    c->ws_partial = reinterpret_cast<float*>(base + lay.partial);
    c->ws_h = reinterpret_cast<float*>(base + lay.h);
    c->ws_ids = reinterpret_cast<int32_t*>(base + lay.ids);
    c->ws_order = reinterpret_cast<int32_t*>(base + lay.order);
    c->ws_clock = reinterpret_cast<unsigned long long*>(base + lay.clock);
    c->ws_slot_map = reinterpret_cast<short*>(base + lay.slot_map);
    c->ws_codes = reinterpret_cast<short*>(base + lay.codes);
    c->ws_counters = reinterpret_cast<unsigned*>(base + lay.counters);
    c->ws_status = reinterpret_cast<int*>(base + lay.status);

    const int L = cfg->n_layers;
    c->table = new SlotTable(L, cfg->n_experts, c->S, false);
    c->pending_protect.resize(L);
    c->prev_rank.assign(L, {});
    c->has_plan.assign(L, 0);
    c->layer_stall_us.assign(L, 0.0);
    c->layer_ffn_us.assign(L, 0.0);
    c->slot_pending.assign(size_t(L) * c->S, 0);
    c->slot_dep.assign(size_t(L) * c->S, 0);
    c->slot_gen_host.assign(size_t(L) * c->S, 0);
    c->slot_want.assign(size_t(L) * c->S, 0);
    c->pool_free_valid.assign(L, 0);

    auto cu = [&](cudaError_t err, const char* what) {
        if (err == cudaSuccess) return true;
        c->err = std::string(what) + " failed: " + cudaGetErrorString(err);
        return false;
    };
    if (!cu(cudaMemsetAsync(base + lay.counters, 0, lay.total - lay.counters, c->compute), "cudaMemsetAsync")) return bail(SPM_ERR_CUDA);
    if (!cu(cudaMemsetAsync(c->ws_slot_gen, 0, size_t(L) * c->S * 4, c->compute), "cudaMemsetAsync")) return bail(SPM_ERR_CUDA);
    if (!cu(cudaHostAlloc(reinterpret_cast<void**>(&c->mb_host), sizeof(Mailbox), cudaHostAllocMapped), "cudaHostAlloc(mailbox)")) return bail(SPM_ERR_CUDA);
    memset(c->mb_host, 0, sizeof(Mailbox));
    if (!cu(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->mb_dev), c->mb_host, 0), "cudaHostGetDevicePointer")) return bail(SPM_ERR_CUDA);
    if (!cu(cudaHostAlloc(reinterpret_cast<void**>(&c->tr_host), sizeof(Mailbox) * kTraceRing * L, cudaHostAllocMapped), "cudaHostAlloc(trace)")) return bail(SPM_ERR_CUDA);
    memset(c->tr_host, 0, sizeof(Mailbox) * kTraceRing * L);
    if (!cu(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->tr_dev), c->tr_host, 0), "cudaHostGetDevicePointer")) return bail(SPM_ERR_CUDA);
    c->tr_ev.resize(kTraceRing);
    for (auto& ev : c->tr_ev) if (!cu(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming), "cudaEventCreate")) return bail(SPM_ERR_CUDA);
    c->slot_ev.resize(size_t(L) * c->S);
    for (auto& ev : c->slot_ev) if (!cu(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming), "cudaEventCreate")) return bail(SPM_ERR_CUDA);
    c->pool_free.resize(L);
    for (auto& ev : c->pool_free) if (!cu(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming), "cudaEventCreate")) return bail(SPM_ERR_CUDA);
    if (!cu(cudaEventCreateWithFlags(&c->wave_done, cudaEventDisableTiming), "cudaEventCreate")) return bail(SPM_ERR_CUDA);
    for (auto& t : c->tim) {
        t.k1_done.resize(L); t.ffn_start.resize(L); t.ffn_end.resize(L); t.used.assign(L, 0);
        for (int l = 0; l < L; ++l)
            if (!cu(cudaEventCreate(&t.k1_done[l]), "cudaEventCreate") || !cu(cudaEventCreate(&t.ffn_start[l]), "cudaEventCreate") ||
                !cu(cudaEventCreate(&t.ffn_end[l]), "cudaEventCreate")) return bail(SPM_ERR_CUDA);
    }
    if (lay.tc) {
        c->rows_cap = lay.rows_cap; c->n_jt = lay.n_jt; c->max_units = lay.max_units;
        c->tc_xs = reinterpret_cast<__nv_bfloat16*>(base + lay.tc_xs);
        c->tc_wrow = reinterpret_cast<float*>(base + lay.tc_wrow);
        c->tc_partial = reinterpret_cast<float*>(base + lay.tc_partial);
        c->tc_desc_dev = base + lay.tc_desc;
        c->tc_counts = reinterpret_cast<int*>(base + lay.tc_counts);
        c->tc_desc_bytes = lay.desc_bytes; c->tc_off_rows = lay.off_rows; c->tc_off_rowmap = lay.off_rowmap;
        c->tc_off_chunks = lay.off_chunks; c->tc_chunk_cap = lay.chunk_cap; c->tc_off_wait = lay.off_wait;
        c->tc_act = base + lay.tc_act;
        c->tc_ready = reinterpret_cast<int*>(base + lay.tc_ready);
        if (!cu(cudaMemsetAsync(c->tc_xs, 0, size_t(lay.rows_cap + kGgTokens) * cfg->hidden * 2, c->compute), "cudaMemsetAsync")) return bail(SPM_ERR_CUDA);
        if (!cu(cudaHostAlloc(reinterpret_cast<void**>(&c->tc_desc_host), size_t(kDescRing) * lay.desc_bytes, cudaHostAllocDefault), "cudaHostAlloc(descriptors)")) return bail(SPM_ERR_CUDA);
        c->tc_desc_ev.resize(kDescRing);
        c->tc_desc_ev_valid.assign(kDescRing, 0);
        for (auto& ev : c->tc_desc_ev) if (!cu(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming), "cudaEventCreate")) return bail(SPM_ERR_CUDA);
        const bool maps_ok = cfg->dtype == SPM_DTYPE_Q4
            ? make_q4_maps(&c->qmapn, &c->qmapsc, c->pools, cfg->hidden, cfg->inter, uint64_t(L) * c->S)
            : make_weight_map(&c->wmap, c->pools, cfg->hidden, cfg->inter, uint64_t(L) * c->S);
        bool xmaps_ok = true;
        for (int b = 0; b < 3; ++b)
            xmaps_ok = xmaps_ok && make_token_map(&c->xmaps.m[b], c->tc_xs, cfg->hidden, uint64_t(lay.rows_cap + kGgTokens), 16u << b);
        if (!maps_ok || !xmaps_ok) {
            c->err = "cuTensorMapEncodeTiled failed";
            return bail(SPM_ERR_CUDA);
        }
        if (!cu(cudaFuncSetAttribute(ffn_grouped_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(ffn_grouped_smem())), "cudaFuncSetAttribute")) return bail(SPM_ERR_CUDA);
        if (!cu(cudaFuncSetAttribute(ffn_grouped_q4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(ffn_grouped_q4_smem())), "cudaFuncSetAttribute")) return bail(SPM_ERR_CUDA);
        if (gg_plan_smem(cfg->n_experts) > 48 * 1024 &&
            !cu(cudaFuncSetAttribute(gg_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(gg_plan_smem(cfg->n_experts))), "cudaFuncSetAttribute")) return bail(SPM_ERR_CUDA);
        c->tc_ok = true;
    }
    c->ring_start.resize(64); c->ring_end.resize(64); c->ring_used.assign(64, 0);
    for (size_t i = 0; i < 64; ++i)
        if (!cu(cudaEventCreate(&c->ring_start[i]), "cudaEventCreate") || !cu(cudaEventCreate(&c->ring_end[i]), "cudaEventCreate")) return bail(SPM_ERR_CUDA);
    if (!cu(cudaStreamSynchronize(c->compute), "cudaStreamSynchronize")) return bail(SPM_ERR_CUDA);

    c->clock_kind.assign(kClockSlots, kClkFfn);
    if (arm_clock(c) != SPM_OK) return bail(SPM_ERR_CUDA);
    c->budget = budget < 0 ? 1 : budget;
    if (budget < 0) {
        double W = 0, tx = 0;
        int raw = 0;
        int rc = spm_profile_window(c, &W, &tx, &raw);
        if (rc) return bail(rc);
        c->budget = std::max(1, raw);
    }
    *out = c;
    return SPM_OK;
}

int spm_destroy(spm_ctx* c) {
    if (!c) return SPM_OK;
    if (c->compute) cudaStreamSynchronize(c->compute);
    if (c->copy) cudaStreamSynchronize(c->copy);
    for (auto ev : c->slot_ev) if (ev) cudaEventDestroy(ev);
    for (auto ev : c->pool_free) if (ev) cudaEventDestroy(ev);
    if (c->wave_done) cudaEventDestroy(c->wave_done);
    for (auto& t : c->tim) {
        for (auto ev : t.k1_done) if (ev) cudaEventDestroy(ev);
        for (auto ev : t.ffn_start) if (ev) cudaEventDestroy(ev);
        for (auto ev : t.ffn_end) if (ev) cudaEventDestroy(ev);
    }
    for (auto ev : c->tc_desc_ev) if (ev) cudaEventDestroy(ev);
    if (c->tc_desc_host) cudaFreeHost(c->tc_desc_host);
    for (auto ev : c->ring_start) if (ev) cudaEventDestroy(ev);
    for (auto ev : c->ring_end) if (ev) cudaEventDestroy(ev);
    if (c->mb_host) cudaFreeHost(c->mb_host);
    for (auto ev : c->tr_ev) if (ev) cudaEventDestroy(ev);
    for (auto& g : c->hf_graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
    if (c->tr_host) cudaFreeHost(c->tr_host);
    delete c->table;
    delete c;
    return SPM_OK;
}

int spm_router_topk(spm_ctx* c, int layer, const float* h, int nb, float* x_norm, int32_t* ids, float* w,
                    float* logits) {
    if (int rc = check_layer(c, layer, nb)) return rc;
    if (int rc = flush_trace(c)) return rc;
    if (!h || !x_norm || !ids || !w) return fail(c, SPM_ERR_INVALID_ARG, "null argument");
    if (int rc = launch_router(c, layer, h, nullptr, nb, x_norm, logits, true, false)) return rc;
    CU(c, cudaMemcpyAsync(w, c->ws_w, size_t(nb) * c->cfg.top_k * 4, cudaMemcpyDeviceToDevice, c->compute));
    if (int rc = wait_mailbox(c)) return rc;
    for (int i = 0; i < nb * c->cfg.top_k; ++i) ids[i] = c->mb_host->ids[i] & 0xffff;
    return SPM_OK;
}

int spm_adapter_predict(spm_ctx* c, int layer, const float* x_norm, int nb, float* scores, int32_t* order) {
    if (int rc = check_layer(c, layer, nb)) return rc;
    if (int rc = flush_trace(c)) return rc;
    if (layer > c->cfg.n_layers - 2) return fail(c, SPM_ERR_INVALID_ARG, "layer %d has no adapter (L-1 adapters)", layer);
    if (!x_norm || !scores || !order) return fail(c, SPM_ERR_INVALID_ARG, "null argument");
    if (int rc = launch_router(c, layer, nullptr, x_norm, nb, nullptr, nullptr, false, true)) return rc;
    if (int rc = wait_mailbox(c)) return rc;
    memcpy(scores, c->mb_host->scores, size_t(c->cfg.n_experts) * 4);
    for (int i = 0; i < c->cfg.n_experts; ++i) order[i] = c->mb_host->order[i] & 0xffff;
    return SPM_OK;
}

int spm_budget_select(spm_ctx* c, int target, const int32_t* order, int n_ranked, int budget, int protect_all,
                      int32_t* out_ids, int* out_count) {
    if (int rc = check_layer(c, target, 1)) return rc;
    if (int rc = flush_trace(c)) return rc;
    if (!order || !out_ids || !out_count || n_ranked < 0 || n_ranked > c->cfg.n_experts)
        return fail(c, SPM_ERR_INVALID_ARG, "bad ranking argument");
    for (int i = 0; i < n_ranked; ++i)
        if (order[i] < 0 || order[i] >= c->cfg.n_experts) return fail(c, SPM_ERR_INVALID_ARG, "expert id %d out of range", order[i]);
    const int bud = budget < 0 ? c->budget : budget;
    c->table->plan(target, order, n_ranked, bud, protect_all != 0, c->sel, c->pending_protect[target]);
    c->has_plan[target] = 1;
    std::copy(c->sel.begin(), c->sel.end(), out_ids);
    *out_count = int(c->sel.size());
    return SPM_OK;
}

int spm_prefetch_async(spm_ctx* c, int target, const int32_t* ids, int count, int* out_issued) {
    if (int rc = check_layer(c, target, 1)) return rc;
    if (int rc = flush_trace(c)) return rc;
    if (count < 0 || (count > 0 && !ids)) return fail(c, SPM_ERR_INVALID_ARG, "bad id list");
    for (int i = 0; i < count; ++i)
        if (ids[i] < 0 || ids[i] >= c->cfg.n_experts) return fail(c, SPM_ERR_INVALID_ARG, "expert id %d out of range", ids[i]);
    const std::vector<int32_t> none;
    const std::vector<int32_t>& prot = c->has_plan[target] ? c->pending_protect[target] : none;
    int rc = do_prefetch(c, target, ids, count, prot.data(), int(prot.size()), out_issued);
    c->has_plan[target] = 0;
    return rc;
}

int spm_moe_ffn(spm_ctx* c, int layer, const float* x_norm, const int32_t* ids, const float* w, int nb, float* h_inout) {
    if (int rc = check_layer(c, layer, nb)) return rc;
    if (int rc = flush_trace(c)) return rc;
    if (!x_norm || !ids || !w || !h_inout) return fail(c, SPM_ERR_INVALID_ARG, "null argument");
    int ring = -1;
    if (c->timing) {
        ring = int(c->ring_pos++ % c->ring_start.size());
        harvest_ring(c, size_t(ring));
    }
    return run_ffn(c, layer, x_norm, ids, w, nb, h_inout, nullptr, ring);
}

int spm_decode_step(spm_ctx* c, const float* h_in, int nb, float* h_out) {
    if (int rc = check_layer(c, 0, nb)) return rc;
    if (!h_in || !h_out) return fail(c, SPM_ERR_INVALID_ARG, "null argument");
    const spm_model_cfg& m = c->cfg;
    if (c->policy == SPM_POLICY_HINT_TRACE && c->table->step() + int(c->tr_pending.size()) >= c->hint_steps)
        return fail(c, SPM_ERR_STATE, "no hint trace for step %d", c->table->step() + int(c->tr_pending.size()));
    bool fast = false;
    if (int rc = host_free_ready(c, nb, &fast)) return rc;
    if (fast) return enqueue_host_free_step(c, h_in, nb, h_out);
    if (int rc = flush_trace(c)) return rc;
    if (h_out != h_in)
        CU(c, cudaMemcpyAsync(h_out, h_in, size_t(nb) * m.hidden * 4, cudaMemcpyDeviceToDevice, c->compute));
    Timing* t = nullptr;
    if (c->timing) {
        c->tim_cur ^= 1;
        t = &c->tim[c->tim_cur];
        harvest(c, *t);
    }
    return step_layers(c, h_out, nb, t, nullptr);
}

int spm_decode_step_host(spm_ctx* c, const float* h_in_host, int nb, float* h_out_host) {
    if (int rc = check_layer(c, 0, nb)) return rc;
    if (!h_in_host || !h_out_host) return fail(c, SPM_ERR_INVALID_ARG, "null argument");
    const size_t bytes = size_t(nb) * c->cfg.hidden * 4;
    CU(c, cudaMemcpyAsync(c->ws_h, h_in_host, bytes, cudaMemcpyHostToDevice, c->compute));
    if (int rc = spm_decode_step(c, c->ws_h, nb, c->ws_h)) return rc;
    CU(c, cudaMemcpyAsync(h_out_host, c->ws_h, bytes, cudaMemcpyDeviceToHost, c->compute));
    CU(c, cudaStreamSynchronize(c->compute));
    return SPM_OK;
}

// ---- control --------------------------------------------------------------
int spm_set_policy(spm_ctx* c, int policy) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    if (policy < SPM_POLICY_ADAPTER || policy > SPM_POLICY_NAIVE) return fail(c, SPM_ERR_INVALID_ARG, "policy %d", policy);
    if ((policy == SPM_POLICY_ADAPTER || policy == SPM_POLICY_PRED0) && c->cfg.n_layers > 1 && (!c->buf.adapter_a || !c->buf.adapter_b))
        return fail(c, SPM_ERR_STATE, "no adapter weights");
    c->policy = policy;
    return SPM_OK;
}
int spm_set_budget(spm_ctx* c, int budget) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    if (budget < 0) return fail(c, SPM_ERR_INVALID_ARG, "budget %d", budget);
    c->budget = budget;
    return SPM_OK;
}
int spm_get_budget(spm_ctx* c, int* budget) {
    if (!c || !budget) return SPM_ERR_INVALID_ARG;
    *budget = c->budget;
    return SPM_OK;
}
int spm_set_plain_lru(spm_ctx* c, int on) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    c->table->set_plain_lru(on != 0);
    return SPM_OK;
}
int spm_set_timing(spm_ctx* c, int on) {
    if (!c) return SPM_ERR_INVALID_ARG;
    c->timing = on != 0;
    return SPM_OK;
}
int spm_set_ffn_ctas(spm_ctx* c, int ctas) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (ctas < 0 || ctas > kMaxCtasBatch1) return fail(c, SPM_ERR_INVALID_ARG, "ctas %d (max %d)", ctas, kMaxCtasBatch1);
    c->ffn_ctas = ctas;
    return SPM_OK;
}
int spm_set_batched_path(spm_ctx* c, int mode) {
    if (!c || mode < 0 || mode > 1) return SPM_ERR_INVALID_ARG;
    c->batched_path = mode;
    return SPM_OK;
}
int spm_set_hint_trace(spm_ctx* c, const int32_t* hint, const int32_t* count, int n_steps, int stride) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    if (!hint || !count || n_steps < 0 || stride < 1) return fail(c, SPM_ERR_INVALID_ARG, "bad hint trace");
    const size_t cells = size_t(n_steps) * c->cfg.n_layers;
    for (size_t i = 0; i < cells; ++i) {
        if (count[i] < 0 || count[i] > stride) return fail(c, SPM_ERR_INVALID_ARG, "hint count out of range");
        for (int q = 0; q < count[i]; ++q)
            if (hint[i * stride + q] < 0 || hint[i * stride + q] >= c->cfg.n_experts)
                return fail(c, SPM_ERR_INVALID_ARG, "hint expert id out of range");
    }
    c->hint.assign(hint, hint + cells * stride);
    c->hint_count.assign(count, count + cells);
    c->hint_steps = n_steps;
    c->hint_stride = stride;
    return SPM_OK;
}
int spm_set_drop_modulo(spm_ctx* c, int modulo) {
    if (!c || modulo < 0) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    c->drop_modulo = modulo;
    return SPM_OK;
}
int spm_set_copy_delay_us(spm_ctx* c, int us) {
    if (!c || us < 0 || us > 100000) return SPM_ERR_INVALID_ARG;
    c->copy_delay_us = us;
    return SPM_OK;
}
int spm_set_device_wait(spm_ctx* c, int on) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (on && !stream_write32_fn()) return fail(c, SPM_ERR_CUDA, "cuStreamWriteValue32 is not available on this driver");
    if (int rc = flush_trace(c)) return rc;
    if ((on != 0) != c->device_wait) {
        // transfers issued in the other mode carry no arrival counters (or no per-slot meaning): let them land first
        CU(c, cudaStreamSynchronize(c->copy));
        CU(c, cudaStreamSynchronize(c->compute));
        std::fill(c->slot_pending.begin(), c->slot_pending.end(), 0);
        // batches led while the option was off did not bump the device-side counters
        if (on) CU(c, cudaMemcpy(c->ws_slot_gen, c->slot_gen_host.data(), c->slot_gen_host.size() * sizeof(uint32_t), cudaMemcpyHostToDevice));
    }
    c->device_wait = on != 0;
    return SPM_OK;
}
int spm_set_host_free(spm_ctx* c, int on) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    c->host_free = on != 0;
    return SPM_OK;
}
int spm_set_graph_replay(spm_ctx* c, int on) {
    if (!c) return SPM_ERR_INVALID_ARG;
    c->graph_replay = on != 0;
    return SPM_OK;
}
int spm_set_attention_stub_us(spm_ctx* c, int us) {
    if (!c || us < 0 || us > 100000) return SPM_ERR_INVALID_ARG;
    c->stub_us = us;
    return SPM_OK;
}
int spm_set_deadline_ms(spm_ctx* c, int ms) {
    if (!c || ms < 1) return SPM_ERR_INVALID_ARG;
    c->deadline_ms = ms;
    return SPM_OK;
}

int spm_set_event_log_limit(spm_ctx* c, size_t max_events) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    c->table->set_event_cap(max_events);
    return SPM_OK;
}
int spm_set_device_wait_limit_us(spm_ctx* c, int us) {
    if (!c || us < 0) return SPM_ERR_INVALID_ARG;
    c->wait_limit_ns = uint64_t(us) * 1000ull;
    return SPM_OK;
}
int spm_test_withhold_arrivals(spm_ctx* c, int count) {
    if (!c || count < 0) return SPM_ERR_INVALID_ARG;
    c->withhold_arrivals = count;
    return SPM_OK;
}

int spm_synchronize(spm_ctx* c) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    CU(c, cudaStreamSynchronize(c->copy));
    CU(c, cudaStreamSynchronize(c->compute));
    return check_status(c);
}

int spm_reset_stats(spm_ctx* c) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    CU(c, cudaStreamSynchronize(c->copy));
    CU(c, cudaStreamSynchronize(c->compute));
    for (auto& t : c->tim) std::fill(t.used.begin(), t.used.end(), 0);
    c->table->reset_accounting();
    std::fill(c->ring_used.begin(), c->ring_used.end(), 0);
    c->ring_us = 0;
    if (int rc = arm_clock(c)) return rc;
    c->window_us = c->router_window_us = c->reduce_window_us = c->gap_us = 0;
    std::fill(c->layer_stall_us.begin(), c->layer_stall_us.end(), 0.0);
    std::fill(c->layer_ffn_us.begin(), c->layer_ffn_us.end(), 0.0);
    c->timed_steps = 0;
    c->extra_late = c->h2d_bytes = c->ffn_launches = c->kernel_launches = c->tokens = 0;
    c->host_free_steps = 0;
    c->ready_sum = c->recall_sum = 0;
    c->recall_at[0] = c->recall_at[1] = c->recall_at[2] = 0;
    c->ready_count = c->recall_count = 0;
    return SPM_OK;
}

int spm_cache_reset(spm_ctx* c) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    CU(c, cudaStreamSynchronize(c->copy));
    CU(c, cudaStreamSynchronize(c->compute));
    for (auto& t : c->tim) std::fill(t.used.begin(), t.used.end(), 0);
    c->table->reset();
    c->fast_ready = false;
    for (auto& r : c->prev_rank) r.clear();
    std::fill(c->ring_used.begin(), c->ring_used.end(), 0);
    c->ring_us = 0;
    if (int rc = arm_clock(c)) return rc;
    c->window_us = c->router_window_us = c->reduce_window_us = c->gap_us = 0;
    std::fill(c->slot_pending.begin(), c->slot_pending.end(), 0);
    // arrival counters start over (both streams are idle): a counter bump lost to fault injection is forgotten here
    std::fill(c->slot_gen_host.begin(), c->slot_gen_host.end(), 0u);
    std::fill(c->slot_want.begin(), c->slot_want.end(), 0u);
    CU(c, cudaMemset(c->ws_slot_gen, 0, c->slot_gen_host.size() * sizeof(uint32_t)));
    c->withhold_arrivals = 0;
    std::fill(c->has_plan.begin(), c->has_plan.end(), 0);
    std::fill(c->layer_stall_us.begin(), c->layer_stall_us.end(), 0.0);
    std::fill(c->layer_ffn_us.begin(), c->layer_ffn_us.end(), 0.0);
    c->timed_steps = 0;
    c->extra_late = c->h2d_bytes = c->ffn_launches = c->kernel_launches = c->tokens = 0;
    c->ready_sum = c->recall_sum = 0;
    c->recall_at[0] = c->recall_at[1] = c->recall_at[2] = 0;
    c->ready_count = c->recall_count = 0;
    c->host_free_steps = 0;
    c->prev_order_valid = false;
    return SPM_OK;
}

int spm_check_invariants(spm_ctx* c, int with_device) {
    if (!c) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    const long long bad = c->table->check();
    if (bad >= 0) return fail(c, SPM_ERR_STATE, "slot table invariant violated at index %lld", bad);
    if (with_device) {
        CU(c, cudaStreamSynchronize(c->compute));
        return check_status(c);
    }
    return SPM_OK;
}

int spm_cache_export(spm_ctx* c, int64_t* state, size_t capacity, size_t* count) {
    if (!c || !count) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    *count = c->table->state_words();
    if (!state) return SPM_OK;
    if (capacity < *count) return fail(c, SPM_ERR_INVALID_ARG, "state buffer too small: %zu < %zu words", capacity, *count);
    c->table->export_state(state);
    return SPM_OK;
}

int spm_cache_import(spm_ctx* c, const int64_t* state, size_t count) {
    if (!c || !state) return SPM_ERR_INVALID_ARG;
    if (count != c->table->state_words()) return fail(c, SPM_ERR_INVALID_ARG, "state has %zu words, this context needs %zu", count, c->table->state_words());
    {   // validate on a scratch table first so that a bad state leaves the context untouched
        SlotTable probe(c->cfg.n_layers, c->cfg.n_experts, c->S, false);
        if (!probe.import_state(state, count)) return fail(c, SPM_ERR_INVALID_ARG, "state does not describe a valid slot table of this shape");
    }
    if (int rc = spm_cache_reset(c)) return rc;          // waits for both streams, clears accounting and pending copies
    c->table->import_state(state, count);
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        int last = -1;
        for (int sl = 0; sl < c->S; ++sl) if (c->table->expert_in(l, sl) >= 0) last = sl;
        if (last < 0) continue;
        const size_t lead = size_t(l) * c->S + last;
        for (int sl = 0; sl <= last; ++sl) {
            const int e = c->table->expert_in(l, sl);
            if (e >= 0) if (int rc = issue_copy(c, l, e, sl, lead, sl == last)) return rc;
        }
    }
    c->h2d_bytes = 0;        // restoring the cache is not decode traffic
    return SPM_OK;
}

int spm_profile_window(spm_ctx* c, double* window_us, double* t_xfer_us, int* budget_raw) {
    if (!c || !window_us || !t_xfer_us || !budget_raw) return SPM_ERR_INVALID_ARG;
    if (int rc = spm_cache_reset(c)) return rc;
    const spm_model_cfg& m = c->cfg;
    const int pools = std::min(m.n_layers, 4);
    cudaEvent_t e0, e1;
    CU(c, cudaEventCreate(&e0));
    CU(c, cudaEventCreate(&e1));
    // expert transfer: one blob from the pinned store into a slot, timed on the copy stream
    std::vector<float> tx;
    for (int it = 0; it < 11; ++it) {
        const int layer = it % pools, e = it % m.n_experts;
        CU(c, cudaEventRecord(e0, c->copy));
        CU(c, cudaMemcpyAsync(slot_ptr(c, layer, it % c->S), host_blob(c, layer, e), c->blob, cudaMemcpyHostToDevice, c->copy));
        if (c->copy_delay_us > 0) attention_stub_kernel<<<1, 1, 0, c->copy>>>(uint64_t(c->copy_delay_us) * 1000ull);
        CU(c, cudaEventRecord(e1, c->copy));
        CU(c, cudaEventSynchronize(e1));
        float ms = 0;
        CU(c, cudaEventElapsedTime(&ms, e0, e1));
        if (it >= 2) tx.push_back(ms * 1e3f);
    }
    // Window: the expert FFN of one layer at this context's batch size, through the same path a
    // decode step takes (slot table, kernel choice, combine), with every needed expert resident.
    // The pools of a few layers are cycled so that the weights come from HBM, not from L2.
    const int R = std::min(c->S, m.n_experts);
    const int nb = m.max_batch;
    {
        std::vector<int32_t> all(R);
        for (int e = 0; e < R; ++e) all[e] = e;
        for (int layer = 0; layer < pools; ++layer)
            if (int rc = do_prefetch(c, layer, all.data(), R, nullptr, 0, nullptr)) return rc;
        CU(c, cudaStreamSynchronize(c->copy));
    }
    std::vector<int32_t> pids(size_t(nb) * m.top_k);
    for (size_t i = 0; i < pids.size(); ++i) pids[i] = int32_t(i % size_t(R));
    std::vector<float> wv(size_t(nb) * m.top_k, 1.0f / m.top_k);
    CU(c, cudaMemcpyAsync(c->ws_w, wv.data(), wv.size() * 4, cudaMemcpyHostToDevice, c->compute));
    CU(c, cudaMemsetAsync(c->ws_x, 0, size_t(nb) * m.hidden * 4, c->compute));
    CU(c, cudaMemsetAsync(c->ws_h, 0, size_t(nb) * m.hidden * 4, c->compute));
    std::vector<float> wt;
    for (int it = 0; it < 14; ++it) {
        CU(c, cudaEventRecord(e0, c->compute));
        if (int rc = run_ffn(c, it % pools, c->ws_x, pids.data(), c->ws_w, nb, c->ws_h, nullptr)) return rc;
        CU(c, cudaEventRecord(e1, c->compute));
        CU(c, cudaEventSynchronize(e1));
        float ms = 0;
        CU(c, cudaEventElapsedTime(&ms, e0, e1));
        if (it >= 5) wt.push_back(ms * 1e3f);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    std::sort(tx.begin(), tx.end());
    std::sort(wt.begin(), wt.end());
    *t_xfer_us = tx[tx.size() / 2];
    *window_us = wt[wt.size() / 2] + c->stub_us;
    *budget_raw = int(*window_us / *t_xfer_us);
    c->prof_window_us = *window_us;
    c->prof_xfer_us = *t_xfer_us;
    c->prof_raw = *budget_raw;
    if (int rc = check_status(c)) return rc;
    return spm_cache_reset(c);
}

int spm_get_profile(spm_ctx* c, double* window_us, double* t_xfer_us, int* budget_raw) {
    if (!c || !window_us || !t_xfer_us || !budget_raw) return SPM_ERR_INVALID_ARG;
    if (c->prof_xfer_us <= 0) return fail(c, SPM_ERR_STATE, "the overlap window has not been profiled on this context");
    *window_us = c->prof_window_us;
    *t_xfer_us = c->prof_xfer_us;
    *budget_raw = c->prof_raw;
    return SPM_OK;
}

int spm_measure_read_bandwidth(spm_ctx* c, size_t bytes, int reps, double* gb_s) {
    if (!c || !gb_s || reps < 1) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    const size_t pool_bytes = size_t(c->cfg.n_layers) * c->S * c->blob;
    bytes = std::min(bytes, pool_bytes) / 16 * 16;
    if (bytes < (size_t(256) << 20)) return fail(c, SPM_ERR_INVALID_ARG, "need at least 256 MiB of slot pools to measure beyond L2");
    cudaEvent_t e0, e1;
    CU(c, cudaEventCreate(&e0));
    CU(c, cudaEventCreate(&e1));
    float best = 0.f;
    for (int r = 0; r < reps + 1; ++r) {        // first repetition is a warm-up
        CU(c, cudaEventRecord(e0, c->compute));
        read_probe_kernel<<<4 * c->num_sms, 512, 0, c->compute>>>(reinterpret_cast<const uint4*>(c->pools), bytes / 16,
                                                                  reinterpret_cast<unsigned*>(c->ws_counters + 8));
        CU(c, cudaGetLastError());
        CU(c, cudaEventRecord(e1, c->compute));
        CU(c, cudaEventSynchronize(e1));
        float ms = 0.f;
        CU(c, cudaEventElapsedTime(&ms, e0, e1));
        if (r > 0) best = std::max(best, float(double(bytes) / (double(ms) * 1e-3) / 1e9));
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *gb_s = best;
    return SPM_OK;
}

int spm_time_ffn_kernel(spm_ctx* c, int first_layer, const float* x_norm, const int32_t* ids, const float* w, int launches,
                        int chained, double* us_per_launch, double* window_us) {
    if (int rc = check_layer(c, first_layer, 1)) return rc;
    if (!x_norm || !ids || !w || !us_per_launch || launches < 1) return fail(c, SPM_ERR_INVALID_ARG, "bad argument");
    if (int rc = flush_trace(c)) return rc;
    const spm_model_cfg& m = c->cfg;
    const int K = m.top_k, L = m.n_layers;
    SlotTable& tb = *c->table;
    for (int i = 0; i < launches; ++i)
        for (int k = 0; k < K; ++k) {
            const int e = ids[size_t(i) * K + k];
            if (e < 0 || e >= m.n_experts) return fail(c, SPM_ERR_INVALID_ARG, "expert id %d out of range", e);
            if (tb.slot_of((first_layer + i) % L, e) < 0)
                return fail(c, SPM_ERR_NOT_RESIDENT, "expert %d of layer %d holds no slot: this probe loads nothing", e, (first_layer + i) % L);
        }
    CU(c, cudaStreamSynchronize(c->copy));          // every transfer issued so far has landed
    std::fill(c->slot_pending.begin(), c->slot_pending.end(), 0);
    const bool clocks = window_us != nullptr;
    if (clocks) { CU(c, cudaStreamSynchronize(c->compute)); if (int rc = arm_clock(c)) return rc; }
    const int G = ffn_grid_for(c, 1);
    cudaEvent_t e0, e1;
    CU(c, cudaEventCreate(&e0));
    CU(c, cudaEventCreate(&e1));
    int rc = SPM_OK;
    const bool pdl = (chained & 1) != 0, graph = chained >= 2;
    cudaGraph_t gr = nullptr;
    cudaGraphExec_t ge = nullptr;
    cudaError_t ce = cudaSuccess;
    if (graph) {
        // (kernel attributes are set outside the capture: one ordinary launch of this variant comes first)
        FfnArgs<1> warm{};
        warm.pool = slot_ptr(c, first_layer, 0); warm.x = x_norm; warm.w = w; warm.partial = c->ws_partial; warm.status = c->ws_status;
        warm.blob_bytes = c->blob; warm.I = m.inter; warm.K = K; warm.n_slots = c->S; warm.n_shared = 0; warm.count[0] = 0;
        ce = launch_gemv<1>(c, warm, G, 1, false);
        if (ce == cudaSuccess) ce = cudaStreamSynchronize(c->compute);
        if (ce == cudaSuccess) ce = cudaStreamBeginCapture(c->compute, cudaStreamCaptureModeThreadLocal);
    } else {
        ce = cudaEventRecord(e0, c->compute);
    }
    for (int i = 0; i < launches && ce == cudaSuccess; ++i) {
        const int layer = (first_layer + i) % L;
        FfnArgs<1> a{};
        a.pool = slot_ptr(c, layer, 0);
        a.shared = m.n_shared ? static_cast<const unsigned char*>(c->buf.shared_experts) + size_t(layer) * m.n_shared * c->blob : nullptr;
        a.x = x_norm;
        a.w = w;
        a.partial = c->ws_partial;
        a.status = c->ws_status;
        a.clock = clocks && i < kClockSlots ? c->ws_clock + 2 * size_t(i) : nullptr;
        a.wait_limit_ns = c->wait_limit_ns;
        a.early = pdl ? 1 : 0;
        a.blob_bytes = c->blob;
        a.I = m.inter; a.K = K; a.n_slots = c->S; a.n_shared = m.n_shared;
        int cnt = 0;
        for (int k = 0; k < K; ++k) {
            a.code[cnt] = short(tb.slot_of(layer, ids[size_t(i) * K + k]));
            a.kidx[cnt++] = (unsigned char)k;
        }
        for (int sh = 0; sh < m.n_shared; ++sh) { a.code[cnt] = short(-1 - sh); a.kidx[cnt++] = 255; }
        a.count[0] = (unsigned char)cnt;
        ce = launch_gemv<1>(c, a, G, 1, pdl);
    }
    if (graph) {
        cudaError_t end = cudaStreamEndCapture(c->compute, &gr);       // (always ends the capture, also after a failed launch)
        if (ce == cudaSuccess) ce = end;
        if (ce == cudaSuccess) ce = cudaGraphInstantiate(&ge, gr, 0);
        if (ce == cudaSuccess) ce = cudaEventRecord(e0, c->compute);
        if (ce == cudaSuccess) ce = cudaGraphLaunch(ge, c->compute);
    }
    if (ce == cudaSuccess) ce = cudaEventRecord(e1, c->compute);
    if (ce == cudaSuccess) ce = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (ce == cudaSuccess) ce = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (ge) cudaGraphExecDestroy(ge);
    if (gr) cudaGraphDestroy(gr);
    if (ce != cudaSuccess) return fail(c, SPM_ERR_CUDA, "expert kernel probe: %s", cudaGetErrorString(ce));
    c->kernel_launches += launches;
    *us_per_launch = double(ms) * 1e3 / launches;
    if (clocks) {
        const int n = std::min(launches, kClockSlots);
        std::vector<unsigned long long> h(size_t(n) * 2);
        CU(c, cudaMemcpy(h.data(), c->ws_clock, h.size() * 8, cudaMemcpyDeviceToHost));
        double sum = 0;
        int got = 0;
        for (int i = 0; i < n; ++i)
            if (h[2 * i + 1] > h[2 * i]) { sum += double(h[2 * i + 1] - h[2 * i]) * 1e-3; ++got; }
        *window_us = got ? sum / got : 0.0;
        rc = arm_clock(c);
    }
    if (rc) return rc;
    return check_status(c);
}

int spm_get_stats(spm_ctx* c, spm_stats* out) {
    if (!c || !out) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    CU(c, cudaStreamSynchronize(c->copy));
    CU(c, cudaStreamSynchronize(c->compute));
    for (auto& t : c->tim) harvest(c, t);
    for (size_t i = 0; i < c->ring_used.size(); ++i) harvest_ring(c, i);
    *out = c->table->stats();
    out->tokens = c->tokens;
    out->late_arrivals = c->extra_late;
    out->h2d_bytes = c->h2d_bytes;
    out->ffn_launches = c->ffn_launches;
    out->kernel_launches = c->kernel_launches;
    if (int rc = harvest_clock(c)) return rc;
    out->ffn_window_us = c->window_us;
    out->router_window_us = c->router_window_us;
    out->reduce_window_us = c->reduce_window_us;
    out->gap_us = c->gap_us;
    out->ffn_us = c->ring_us;
    out->stall_us = 0;
    for (int l = 0; l < c->cfg.n_layers; ++l) { out->ffn_us += c->layer_ffn_us[l]; out->stall_us += c->layer_stall_us[l]; }
    out->ready_sum = c->ready_sum; out->ready_count = c->ready_count;
    out->recall_sum = c->recall_sum; out->recall_count = c->recall_count;
    for (int j = 0; j < 3; ++j) out->recall_at[j] = c->recall_at[j];
    out->host_free_steps = c->host_free_steps;
    return check_status(c);
}

int spm_get_layer_times(spm_ctx* c, double* stall_us, double* ffn_us, uint64_t* steps) {
    if (!c || !stall_us || !ffn_us || !steps) return SPM_ERR_INVALID_ARG;
    CU(c, cudaStreamSynchronize(c->compute));
    for (auto& t : c->tim) harvest(c, t);
    for (int l = 0; l < c->cfg.n_layers; ++l) { stall_us[l] = c->layer_stall_us[l]; ffn_us[l] = c->layer_ffn_us[l]; }
    *steps = c->timed_steps;
    return SPM_OK;
}

int spm_get_events(spm_ctx* c, spm_event* out, size_t capacity, size_t* count) {
    if (!c || !count) return SPM_ERR_INVALID_ARG;
    if (int rc = flush_trace(c)) return rc;
    const auto& ev = c->table->events();
    *count = ev.size();
    if (out) memcpy(out, ev.data(), std::min(capacity, ev.size()) * sizeof(spm_event));
    return SPM_OK;
}

int spm_get_slot_table(spm_ctx* c, int layer, int32_t* slot_expert) {
    if (int rc = check_layer(c, layer, 1)) return rc;
    if (int rc = flush_trace(c)) return rc;
    if (!slot_expert) return SPM_ERR_INVALID_ARG;
    for (int s = 0; s < c->S; ++s) slot_expert[s] = c->table->expert_in(layer, s);
    return SPM_OK;
}

int spm_host_alloc(size_t bytes, void** out) {
    if (!out || bytes == 0) return SPM_ERR_INVALID_ARG;
    cudaError_t e = cudaHostAlloc(out, bytes, cudaHostAllocDefault);
    if (e != cudaSuccess) { g_init_error = std::string("cudaHostAlloc failed: ") + cudaGetErrorString(e); *out = nullptr; return SPM_ERR_CUDA; }
    return SPM_OK;
}
int spm_host_free(void* p) {
    if (!p) return SPM_OK;
    return cudaFreeHost(p) == cudaSuccess ? SPM_OK : SPM_ERR_CUDA;
}

// ---- host-only simulator ----------------------------------------------------
}  // extern "C"

struct spm_sim {
    SlotTable table;
    std::vector<Placement> placements;
    std::vector<int32_t> sel, protect;
    spm_sim(int L, int n, int S, bool plain) : table(L, n, S, plain) {}
};

extern "C" {

int spm_sim_create(int n_layers, int n_experts, int slots, int plain_lru, spm_sim** out) {
    if (!out || n_layers < 1 || n_experts < 1 || n_experts > SPM_MAX_EXPERTS || slots < 1) return SPM_ERR_INVALID_ARG;
    *out = new spm_sim(n_layers, n_experts, slots, plain_lru != 0);
    return SPM_OK;
}
int spm_sim_destroy(spm_sim* s) { delete s; return SPM_OK; }

int spm_plan_grouped_chunks(int n_units, int n_dt, int grid, int32_t* chunks, size_t capacity, size_t* count) {
    if (n_units < 1 || n_dt < 1 || n_dt > 32767 || grid < 1 || !chunks || !count) return SPM_ERR_INVALID_ARG;
    std::vector<GgTaskHost> list;
    gg_plan_chunks(n_units, n_dt, grid, list);
    *count = list.size();
    if (list.size() > capacity) return SPM_ERR_INVALID_ARG;
    for (size_t i = 0; i < list.size(); ++i) {
        chunks[3 * i] = list[i].unit;
        chunks[3 * i + 1] = list[i].dt0;
        chunks[3 * i + 2] = list[i].dt1;
    }
    return SPM_OK;
}

static bool sim_ids_ok(spm_sim* s, int layer, const int32_t* ids, int count) {
    if (!s || layer < 0 || layer >= s->table.layers() || count < 0 || (count > 0 && !ids)) return false;
    for (int i = 0; i < count; ++i) if (ids[i] < 0 || ids[i] >= s->table.experts()) return false;
    return true;
}

int spm_sim_demand(spm_sim* s, int layer, const int32_t* need, int count, int32_t* out_expert, int32_t* out_slot,
                   int32_t* out_wave, int32_t* out_missed, int* out_count, int* out_waves) {
    if (!sim_ids_ok(s, layer, need, count) || !out_expert || !out_slot || !out_wave || !out_missed || !out_count) return SPM_ERR_INVALID_ARG;
    int waves = 1;
    s->table.demand(layer, need, count, s->placements, &waves);
    for (size_t i = 0; i < s->placements.size(); ++i) {
        out_expert[i] = s->placements[i].expert; out_slot[i] = s->placements[i].slot;
        out_wave[i] = s->placements[i].wave; out_missed[i] = s->placements[i].missed;
    }
    *out_count = int(s->placements.size());
    if (out_waves) *out_waves = waves;
    return SPM_OK;
}

int spm_sim_plan(spm_sim* s, int layer, const int32_t* order, int n_ranked, int budget, int protect_all,
                 int32_t* out_ids, int* out_count, int32_t* out_protect, int* out_n_protect) {
    if (!sim_ids_ok(s, layer, order, n_ranked) || budget < 0 || !out_ids || !out_count || !out_protect || !out_n_protect) return SPM_ERR_INVALID_ARG;
    s->table.plan(layer, order, n_ranked, budget, protect_all != 0, s->sel, s->protect);
    std::copy(s->sel.begin(), s->sel.end(), out_ids);
    std::copy(s->protect.begin(), s->protect.end(), out_protect);
    *out_count = int(s->sel.size());
    *out_n_protect = int(s->protect.size());
    return SPM_OK;
}

int spm_sim_prefetch(spm_sim* s, int layer, const int32_t* ids, int count, const int32_t* protect, int n_protect,
                     int drop_modulo, int32_t* out_slots, int* out_issued) {
    if (!sim_ids_ok(s, layer, ids, count) || !sim_ids_ok(s, layer, protect, n_protect) || !out_slots || drop_modulo < 0) return SPM_ERR_INVALID_ARG;
    int issued = s->table.prefetch(layer, ids, count, protect, n_protect, drop_modulo, out_slots);
    if (out_issued) *out_issued = issued;
    return SPM_OK;
}

int spm_sim_plan_only(spm_sim* s, int layer, const int32_t* ids, int count) {
    if (!sim_ids_ok(s, layer, ids, count)) return SPM_ERR_INVALID_ARG;
    s->table.plan_only(layer, ids, count);
    return SPM_OK;
}

int spm_sim_end_step(spm_sim* s) {
    if (!s) return SPM_ERR_INVALID_ARG;
    s->table.end_step();
    s->table.stats().steps++;
    return SPM_OK;
}

int spm_sim_events(spm_sim* s, spm_event* out, size_t capacity, size_t* count) {
    if (!s || !count) return SPM_ERR_INVALID_ARG;
    const auto& ev = s->table.events();
    *count = ev.size();
    if (out) memcpy(out, ev.data(), std::min(capacity, ev.size()) * sizeof(spm_event));
    return SPM_OK;
}

int spm_sim_stats(spm_sim* s, spm_stats* out) {
    if (!s || !out) return SPM_ERR_INVALID_ARG;
    *out = s->table.stats();
    return SPM_OK;
}

int spm_sim_check(spm_sim* s) {
    if (!s) return SPM_ERR_INVALID_ARG;
    return s->table.check() < 0 ? SPM_OK : SPM_ERR_STATE;
}

int spm_sim_export(spm_sim* s, int64_t* state, size_t capacity, size_t* count) {
    if (!s || !count) return SPM_ERR_INVALID_ARG;
    *count = s->table.state_words();
    if (!state) return SPM_OK;
    if (capacity < *count) return SPM_ERR_INVALID_ARG;
    s->table.export_state(state);
    return SPM_OK;
}

int spm_sim_import(spm_sim* s, const int64_t* state, size_t count) {
    if (!s || !state) return SPM_ERR_INVALID_ARG;
    return s->table.import_state(state, count) ? SPM_OK : SPM_ERR_INVALID_ARG;
}

int spm_sim_slot_table(spm_sim* s, int layer, int32_t* slot_expert) {
    if (!s || !slot_expert || layer < 0 || layer >= s->table.layers()) return SPM_ERR_INVALID_ARG;
    for (int i = 0; i < s->table.slots(); ++i) slot_expert[i] = s->table.expert_in(layer, i);
    return SPM_OK;
}

}  // extern "C"
