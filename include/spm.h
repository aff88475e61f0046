/*
 * spm.h — C ABI of the offloaded sparse-MoE decode step with prediction-guided,
 * window-budgeted expert prefetch (SpecPrefetch), for one NVIDIA B200 (sm_100a).
 *
 * One decode step pushes nb hidden rows through L MoE layers. Per layer l:
 *   1. native router (frozen):  x = RMSNorm(h);  z = W_r x;  p = softmax(z);
 *      T = Top_K(z);  w_e = p_e / sum_{j in T} p_j            [Section 3.1, first equation]
 *   2. batch demand T_batch = union of the tokens' Top-K sets  [Section 3.1, second equation];
 *      experts of T_batch without a cache slot are copied on demand from the pinned
 *      host store (the fallback that Section 3.3's last paragraph prescribes for every
 *      needed expert the prefetch did not bring in)
 *   3. adapter (l <= L-2):  z^ = Bup (A x);  pi^ = softmax(z^);  s_e = sum over tokens of pi^_e
 *      [Section 3.2, equations 1, 3, 4]; the experts of layer l+1 are ranked by s
 *   4. budgeted selection  P = Top_{M_max}({ s_e : e not available, not in transfer }),
 *      issued asynchronously in descending priority, |P| <= M_max   [Section 3.3]
 *   5. routed (+ shared) SwiGLU experts read in place from their slots:
 *      h += sum_k w_k W_down( silu(W_gate x) * (W_up x) )
 * The prediction only moves transfers earlier; routing and outputs never depend on it
 * (Section 3.1, last paragraph).
 *
 * Conventions
 *   - every function returns an int status (SPM_OK or a negative SPM_ERR_*); nothing throws
 *     or aborts; results come back through out-pointers; spm_last_error() gives a message.
 *   - "dev" pointers are CUDA device pointers, "host" pointers ordinary host memory,
 *     "pinned" page-locked host memory. The library never frees or reallocates caller memory.
 *   - the caller owns all weights, the pinned expert store, the device arena and both CUDA
 *     streams (passed as cudaStream_t cast to void*); the library owns its context, the slot
 *     tables, its CUDA events and a small host-mapped mailbox.
 *   - one context per host thread. GPU work is enqueued on the caller's streams; a call
 *     returns as soon as the host has what it needs (calls that hand expert ids to the host
 *     wait, with a deadline, for the routing kernel only).
 *   - layers, experts, slots are 0-based. Adapter `l` scores layer l+1 and exists for l <= L-2.
 *   - all matrices are row-major. dtype applies to every weight matrix (router, adapter,
 *     experts); activations, logits, scores and routing weights are fp32.
 */
#ifndef SPM_H
#define SPM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ---------------------------------------------------- */
#define SPM_OK                 0
#define SPM_ERR_INVALID_ARG   (-1)  /* null pointer, index out of range                       */
#define SPM_ERR_CONFIG        (-2)  /* unsupported shape, slots < top_k at batch 1, ...        */
#define SPM_ERR_CUDA          (-3)  /* a CUDA runtime call failed (message has the detail)    */
#define SPM_ERR_TIMEOUT       (-4)  /* routing kernel did not report within the deadline      */
#define SPM_ERR_NOT_RESIDENT  (-5)  /* an expert handed to the FFN has no loaded slot         */
#define SPM_ERR_STATE         (-6)  /* call made in the wrong order (e.g. no hint trace set)  */
#define SPM_ERR_NUMERIC       (-7)  /* a routing kernel met a non-finite logit (NaN / Inf in h or weights) */

#define SPM_DTYPE_FP32 0
#define SPM_DTYPE_BF16 1
#define SPM_DTYPE_Q4   2   /* experts 4-bit (groups of 32 weights + one fp16 scale, value = scale * (q - 8)):
                              the paper's on-device precision; router, adapter matrices stay bf16 */

/* prefetch policies */
#define SPM_POLICY_ADAPTER    0   /* rank next-layer experts with the low-rank adapter (the method)    */
#define SPM_POLICY_ON_DEMAND  1   /* no prediction, no prefetch (the paper's OFF arm, Table 4)          */
#define SPM_POLICY_HINT_TRACE 2   /* perfect knowledge: ranking = recorded true next-layer experts      */
#define SPM_POLICY_PRED0      3   /* predict and select, issue no transfer (the paper's PRED0, Table 4) */
#define SPM_POLICY_NAIVE      4   /* prediction = the experts the preceding token used at that layer (the
                                     paper's Naive Prefetch, Table 5), ranked by sum over tokens of
                                     (K - rank position), ties to the lower id                          */

/* cache event kinds (spm_event.kind) */
#define SPM_EV_HIT            1   /* needed expert already has a slot                                   */
#define SPM_EV_HIT_PREFETCHED 2   /* ... and this is the first use of a prefetched expert               */
#define SPM_EV_MISS           3   /* loaded on demand into `slot`                                        */
#define SPM_EV_EVICT          4   /* `expert` removed from `slot`                                        */
#define SPM_EV_EVICT_WASTED   5   /* ... it had been prefetched and was never used                       */
#define SPM_EV_PREFETCH       6   /* prefetch of `expert` into `slot` issued                             */
#define SPM_EV_TOUCH_PRED     7   /* resident expert protected because the prediction ranks it high      */
#define SPM_EV_WAVE           8   /* demand exceeds the slots: a new wave starts (`expert` = wave index) */
#define SPM_EV_PLAN           9   /* PRED0: selected but not issued (`slot` = -1)                        */
#define SPM_EV_DROPPED        10  /* fault injection: prefetch request lost (`slot` = -1)                */

#define SPM_MAX_BATCH   64
#define SPM_MAX_TOPK    16        /* top_k + n_shared <= SPM_MAX_TOPK */
#define SPM_MAX_EXPERTS 1024

typedef struct spm_ctx spm_ctx;   /* GPU decode context           */
typedef struct spm_sim spm_sim;   /* host-only slot-table policy  */

typedef struct {
    int32_t n_layers;      /* L                                             */
    int32_t hidden;        /* D                                             */
    int32_t n_experts;     /* n routed experts per layer                    */
    int32_t inter;         /* I, SwiGLU intermediate size                   */
    int32_t top_k;         /* K                                             */
    int32_t n_shared;      /* always-resident shared experts per layer      */
    int32_t adapter_rank;  /* r                                             */
    int32_t dtype;         /* SPM_DTYPE_*                                   */
    int32_t renormalize;   /* 1: w_e = p_e / sum over the Top-K             */
    int32_t max_batch;     /* largest nb any call will pass (<= SPM_MAX_BATCH) */
    float   rms_eps;
} spm_model_cfg;

typedef struct {
    const void* rms_gamma;       /* dev   fp32 [L][D]                                            */
    const void* router_w;        /* dev   [L][n][D]                                              */
    const void* adapter_a;       /* dev   [L-1][r][D]   (may be NULL when L == 1)                */
    const void* adapter_b;       /* dev   [L-1][n][r]                                            */
    const void* shared_experts;  /* dev   [L][n_shared] packed blobs (NULL when n_shared == 0)   */
    const void* host_experts;    /* pinned [L][n] packed blobs: the offloaded expert store       */
    void*       arena;           /* dev, 256-byte aligned: slot pools + workspace                */
    size_t      arena_bytes;     /* >= spm_query_arena()                                         */
    void*       compute_stream;  /* cudaStream_t                                                 */
    void*       copy_stream;     /* cudaStream_t, different from compute_stream                  */
    int32_t     host_store_layers; /* 0 or L: host_experts holds all L layers. 0 < k < L: it holds only k
                                      layers and layer l reads the blobs of layer l % k (for hosts that
                                      cannot pin the whole store; the model then repeats its expert
                                      weights every k layers, sizes and traffic are unchanged)        */
} spm_buffers;

typedef struct { int32_t step, layer, kind, expert, slot; } spm_event;

typedef struct {
    uint64_t steps, tokens;
    uint64_t hits, hits_prefetched, misses, evictions, wasted;
    uint64_t prefetch_issued, touches, waves, planned, dropped;
    uint64_t late_arrivals;      /* needed expert whose prefetch copy was still in flight (timing only) */
    uint64_t h2d_bytes;          /* expert bytes copied host -> HBM                                      */
    uint64_t ffn_launches;       /* expert-FFN kernel launches timed below                               */
    uint64_t kernel_launches;    /* all kernels this context launched                                    */
    double   ffn_us;             /* summed CUDA-event time around those launches (needs spm_set_timing(ctx, 1)) */
    double   ffn_window_us;      /* same launches, first CTA start to last CTA end read from %globaltimer
                                    inside the kernel: excludes launch latency (profiling aid)            */
    double   stall_us;           /* summed gap "routing kernel done -> expert FFN may start" per layer    */
    double   ready_sum;          /* sum over (step, layer >= 1, token) of |T ∩ has-slot| / K at demand   */
    uint64_t ready_count;        /*   ... and the number of terms (ReadyRecall = ready_sum / ready_count) */
    double   recall_sum;         /* sum over (step, layer >= 1, token) of |T ∩ Top_M(s)| / K, M = budget  */
    uint64_t recall_count;       /*   ExpertRecall@M = recall_sum / recall_count  (Section 4.1)          */
    uint64_t host_free_steps;    /* decode steps enqueued without a host turn (spm_set_host_free)        */
    double router_window_us;     /* in-kernel windows of the routing kernels (first leader past its launch      */
    double reduce_window_us;     /*   dependency -> last leader done) and of the combine kernels, timing on     */
    double gap_us;               /* device idle time between consecutive clocked kernels of the compute stream  */
    double recall_at[3];         /* sums like recall_sum for M = max(1, K/2), K, K+2 (the coverage levels of
                                    the paper's model-level table); divide by recall_count                    */
    uint64_t events_dropped;     /* cache events not stored because the event log was full (spm_set_event_log_limit) */
} spm_stats;

/* ---- packed expert layout ------------------------------------------------
 * One expert = one contiguous blob of 3*I*D elements, identical in the host store, in a
 * cache slot and in shared_experts, so one transfer is one copy:
 *     blob[j][0][0..D) = W_gate[j][:]      j = 0..I-1
 *     blob[j][1][0..D) = W_up[j][:]
 *     blob[j][2][0..D) = W_down[:][j]      (column j of W_down[D][I])
 * With SPM_DTYPE_Q4 each of these rows is packed as D/2 bytes of nibbles (element 2b in the low
 * half of byte b, 2b+1 in the high half) followed by D/32 fp16 scales, one per 32 consecutive elements.
 * Writes the blob size to *bytes: 3*I*D*sizeof(element), or 3*I*(D/2 + D/16) for 4-bit experts. */
int spm_expert_blob_bytes(const spm_model_cfg* cfg, size_t* bytes);

/* Bytes of device arena needed for `slots_per_layer` routed slots per layer plus workspace. */
int spm_query_arena(const spm_model_cfg* cfg, int slots_per_layer, size_t* bytes);

/* Create a context. budget = M_max >= 0, or -1 to derive it from the profiled overlap window
 * (spm_profile_window is then run once here: max(1, floor(W / t_xfer)); Section 3.3, first
 * paragraphs). Slot tables start empty (cold cache). Fails with SPM_ERR_CONFIG when
 * max_batch == 1 and slots_per_layer < top_k, or when the shape is not supported by the
 * kernels (hidden must be a multiple of 256 and <= 2048 (bf16, 4-bit) / of 128 and <= 1024 (fp32)). */
int spm_init(const spm_model_cfg* cfg, int slots_per_layer, int budget,
             const spm_buffers* buffers, spm_ctx** out);
int spm_destroy(spm_ctx* ctx);
const char* spm_last_error(const spm_ctx* ctx);   /* ctx may be NULL: last error of spm_init */

/* Native router of `layer` (Section 3.1, first equation): RMSNorm, gate GEMV, softmax, Top-K,
 * renormalise.   h dev [nb][D] -> x_norm dev [nb][D], w dev [nb][K] (rank order),
 * logits dev [nb][n] (may be NULL), ids HOST [nb][K] (rank order: ties to the lower id).
 * Returns after the ids have reached the host (bounded wait, SPM_ERR_TIMEOUT). */
int spm_router_topk(spm_ctx* ctx, int layer, const float* h, int nb,
                    float* x_norm, int32_t* ids, float* w, float* logits);

/* Adapter of `layer` (Section 3.2): priorities of the experts of layer+1.
 * x_norm dev [nb][D] -> scores HOST [n] (s_e summed over the nb tokens in token order),
 * order HOST [n] (expert ids by (s descending, id ascending)). layer <= L-2. */
int spm_adapter_predict(spm_ctx* ctx, int layer, const float* x_norm, int nb,
                        float* scores, int32_t* order);

/* Selection of Section 3.3 for pool `target_layer`: walk `order` (host, n_ranked ids in
 * descending priority), skip experts that have a slot (available or in transfer), keep at
 * most `budget` (budget < 0: the context's M_max). Host logic only; nothing is issued.
 * protect_all = 0: the resident experts ranked above the last selected one are remembered for
 * the next spm_prefetch_async on this layer (predicted-use touch); 1: every resident expert in
 * `order` (use when `order` lists exactly the experts that will be needed).
 * out_ids host [>= min(budget, slots)], descending priority. */
int spm_budget_select(spm_ctx* ctx, int target_layer, const int32_t* order, int n_ranked,
                      int budget, int protect_all, int32_t* out_ids, int* out_count);

/* Asynchronous transfer of the selected experts (Section 3.3: the candidates of P are moved in
 * descending order of predicted priority while computation goes on). Issues host->HBM copies of
 * experts `ids` (host, descending priority) of `target_layer` on the copy stream into
 * least-recently-used slots of that layer's pool, in the order given; the copies of one call form
 * a batch with one CUDA event, recorded after its last copy, which later launches wait on.
 * Experts that already have a slot are skipped. Stops when no unprotected slot is left.
 * *out_issued (may be NULL) = number of copies enqueued. Asynchronous. */
int spm_prefetch_async(spm_ctx* ctx, int target_layer, const int32_t* ids, int count,
                       int* out_issued);

/* Expert computation of `layer` with the on-demand fallback (Section 3.1, second equation: the
 * batch demand T_batch; Section 3.3, last paragraph: whatever the router asks for and the cache
 * lacks is loaded at execution time, so outputs never depend on the prediction).
 * Routed + shared SwiGLU experts for nb tokens, slot-indexed (no gather):
 * resolves the batch demand against the slot table, loads misses on demand, makes the compute
 * stream wait for exactly the copy batches whose slots it reads, and enqueues
 * h_inout += sum_k w_k FFN_{ids_k}(x).
 * x_norm dev [nb][D], ids HOST [nb][K], w dev [nb][K], h_inout dev [nb][D]. Asynchronous.
 * When more distinct experts are needed than there are slots the work is split in waves. On the
 * batched tensor-core path the sum of a token's experts is taken in rank order whatever the waves
 * were, and at batch 1 a layer is one launch whenever slots >= top_k, so in both cases the result
 * does not depend on the cache state, bit for bit. */
int spm_moe_ffn(spm_ctx* ctx, int layer, const float* x_norm, const int32_t* ids,
                const float* w, int nb, float* h_inout);

/* One decode step through all L layers under the context's policy (Sections 3.1 - 3.3 in the order
 * of the paper's pipeline figure: route layer l, load what is missing, predict and prefetch for
 * layer l+1 while layer l's experts compute): h_in dev [nb][D] ->
 * h_out dev [nb][D] (may alias h_in). Equivalent to, per layer: spm_router_topk,
 * spm_adapter_predict, spm_moe_ffn, spm_budget_select + spm_prefetch_async for layer+1,
 * with router and adapter fused in one kernel. The last layer's work is left in flight. */
int spm_decode_step(spm_ctx* ctx, const float* h_in, int nb, float* h_out);

/* Same, with HOST buffers (pinned for speed): copies h_in to the device, runs the step, copies
 * h_out back and waits for it. */
int spm_decode_step_host(spm_ctx* ctx, const float* h_in_host, int nb, float* h_out_host);

/* ---- control, profiling, accounting ------------------------------------ */
int spm_set_policy(spm_ctx* ctx, int policy);
int spm_set_budget(spm_ctx* ctx, int budget);             /* M_max >= 0 */
int spm_get_budget(spm_ctx* ctx, int* budget);
int spm_set_plain_lru(spm_ctx* ctx, int on);              /* 1: no predicted-use touch */
int spm_set_timing(spm_ctx* ctx, int on);                 /* record CUDA events around FFN / stalls */
int spm_set_ffn_ctas(spm_ctx* ctx, int ctas);             /* CTAs per token of the GEMV FFN (0 = default) */
/* Expert FFN used when nb > 1. 0 (default): the grouped tensor-core kernel (tcgen05, bf16
 * activations, fp32 accumulation) whenever the shape allows it (bf16 or 4-bit weights, no shared
 * experts, inter a multiple of 128, hidden a multiple of 128 for bf16 and of 256 for 4-bit
 * weights, which are expanded to bf16 on the way to the tensor cores), else the GEMV kernel once
 * per token. 1: always the GEMV kernel per token (fp32 activations). */
int spm_set_batched_path(spm_ctx* ctx, int mode);
/* Perfect-knowledge ranking for SPM_POLICY_HINT_TRACE: for step s (counted from the last
 * spm_cache_reset) and layer l, hint[(s*L + l)*stride .. +count[s*L+l]) are the experts that
 * layer truly needs, in priority order. Copied. */
int spm_set_hint_trace(spm_ctx* ctx, const int32_t* hint, const int32_t* count,
                       int n_steps, int stride);
/* Fault injection on the host: every prefetch request with (step + expert) % modulo == 0 is
 * lost before it reaches the GPU (0 switches it off). The demand path must then load it. */
int spm_set_drop_modulo(spm_ctx* ctx, int modulo);
/* Emulated slower storage tier (the paper's controlled loading delays, Section 4.1): every expert
 * copy is followed on the copy stream by a wait of `us` microseconds (0 = off, at most 100000)
 * before the slot counts as loaded. Outputs are unchanged. */
int spm_set_copy_delay_us(spm_ctx* ctx, int us);
/* Device-side wait for the expert FFNs (default off): the batch-1 kernels (bf16, fp32 and 4-bit
 * experts) and the grouped tensor-core kernels of batched decode (bf16 and 4-bit experts). Off: the
 * compute stream waits on the event of the batch of copies that fills the slots a launch reads,
 * then the kernel starts. On: the kernel is launched at once and its warps (batch 1) or the producer
 * warp of each unit (grouped kernels) wait, bounded, SPM_ERR_TIMEOUT on expiry, on an arrival
 * counter that the copy stream bumps after the last copy of that batch has landed, so rows of
 * resident experts are streamed while missing ones are still in flight and no launch latency
 * follows the last copy. Outputs are bit-identical either way. With it on, the timed FFN duration
 * includes the wait for copies. Switching the option waits for both streams. */
int spm_set_device_wait(spm_ctx* ctx, int on);
/* Host-free decode steps (default on). Once every expert of every layer holds a slot and every
 * copy has landed (possible only with slots_per_layer >= n_experts), no routing result can change
 * what the prefetch controller does: each demand is a hit and no selection finds a non-resident
 * candidate (Section 3.3). spm_decode_step then enqueues all layers without waiting for any routing
 * result: the routing kernel leaves the slot numbers of the chosen experts in device memory for the
 * expert kernel that follows, each kernel is launched so that its preamble overlaps the end of its
 * predecessor, and the ids / rankings go to a ring of host-mapped trace mailboxes from which the
 * slot table's bookkeeping (hits, LRU ticks, recall statistics, event log) is replayed in order,
 * at the latest when a call reads or changes that state. Outputs, events and statistics are the
 * same as with the option off; per-layer event timings are not taken in such steps (the in-kernel
 * window still is). On the batched tensor-core path the wave plan (token rows sorted by expert,
 * work units, combine map) is then built by a kernel instead of the host.
 * spm_cache_reset() ends the state; it is re-entered once the pools are full again. */
int spm_set_host_free(spm_ctx* ctx, int on);
/* Replay host-free steps from CUDA graphs (default on): the launches of such a step are the same
 * every time for a given trace slot, batch size, output buffer and launch geometry, so each
 * combination is captured once (after one step enqueued launch by launch) and replayed with a
 * single submission. Off, or with timing / an attention stand-in set, every kernel is launched
 * individually. Results are identical. */
int spm_set_graph_replay(spm_ctx* ctx, int on);
/* Stand-in for the attention block the synthetic configurations omit: before each layer's router a
 * kernel that only waits `us` microseconds (0 = off, at most 100000) is enqueued on the compute
 * stream. It widens the overlap window W_l = t_exec(l+1) - t_pred(l) (Section 3.1) toward the
 * paper's regime; spm_profile_window adds it to the window it reports. Outputs are unchanged. */
int spm_set_attention_stub_us(spm_ctx* ctx, int us);
/* The cache-event log (spm_get_events) keeps at most `max_events` records between two calls of
 * spm_reset_stats / spm_cache_reset (default 1,048,576, about 20 MB of host memory; a Qwen3-shaped
 * step logs 400 - 800 events); events beyond that are only counted, in spm_stats.events_dropped.
 * 0 switches the log off. Counters and recall statistics do not depend on the log. */
int spm_set_event_log_limit(spm_ctx* ctx, size_t max_events);
/* Host deadline of the routing-kernel handshake, in milliseconds (default 5000). */
int spm_set_deadline_ms(spm_ctx* ctx, int ms);
/* Limit of every wait inside the expert kernels (for a weight copy to land in shared memory, for an
 * arrival counter with spm_set_device_wait, for a pipeline barrier of the grouped kernels), in
 * microseconds; 0 restores the default of 2 s. A wait that runs out sets a status bit, the kernel
 * winds down (no copy left in flight, tensor memory released) and returns; the next
 * spm_synchronize / spm_get_stats reports SPM_ERR_TIMEOUT once and the context stays usable
 * (spm_cache_reset brings slot table and arrival counters back to a known state). */
int spm_set_device_wait_limit_us(spm_ctx* ctx, int us);
/* Host-side fault injection for tests of that time-out: with spm_set_device_wait on, the next
 * `count` arrival-counter updates are not enqueued (the bytes still land; the counter never says
 * so), so the kernel that waits for that batch gives up after the limit. Nothing on the GPU
 * faults or hangs. Cleared by spm_cache_reset. */
int spm_test_withhold_arrivals(spm_ctx* ctx, int count);

/* Profile the overlap window (Section 3.3): window_us = median device time of the expert FFN of
 * one layer at max_batch tokens with every needed expert resident (kernel(s) + combine, the same
 * path a decode step takes), t_xfer_us = median time of one expert copy from the pinned store,
 * *budget_raw = floor(window / t_xfer). Uses and then empties the cache. */
int spm_profile_window(spm_ctx* ctx, double* window_us, double* t_xfer_us, int* budget_raw);
/* What the most recent spm_profile_window on this context measured, including the run inside
 * spm_init(budget = -1), whose budget is max(1, *budget_raw) (Section 3.3: the budget follows the
 * profiled window). SPM_ERR_STATE when the context has never been profiled. */
int spm_get_profile(spm_ctx* ctx, double* window_us, double* t_xfer_us, int* budget_raw);
/* Read-only HBM streaming rate of this device, as a second denominator beside the copy bandwidth:
 * a kernel that only reads (16-byte loads, grid of 4 CTAs per SM, every loaded word folded into a
 * checksum that is written once per thread) streams the first `bytes` of the slot pools (clamped
 * to their size, rounded down to 16 bytes; at least 256 MiB is needed so that L2 does not serve
 * it) `reps` >= 1 times on the compute stream; *gb_s is the best repetition by CUDA event pair.
 * The pool contents are not modified. Waits for the compute stream. */
int spm_measure_read_bandwidth(spm_ctx* ctx, size_t bytes, int reps, double* gb_s);
/* Device time of the batch-1 expert-FFN kernel by itself (measurement aid; the hidden row is not
 * updated and no combine kernel runs). Enqueues `launches` launches of the slot-indexed GEMV kernel
 * back to back on the compute stream, launch i on layer (first_layer + i) % L with the K experts
 * ids[i*K .. i*K+K) (HOST) plus the layer's shared experts, x_norm dev [D], w dev [K], between one
 * pair of CUDA events, and waits. Every expert named must already hold a slot
 * (SPM_ERR_NOT_RESIDENT otherwise: nothing is loaded here).
 * chained = 1: launched with the programmatic-serialisation attribute (as all kernels of a decode step are), so a
 * launch fetches its first weight rows while its predecessor drains; 0: plain launches, each
 * starts after the one before it has ended; 2 and 3: the same as 0 and 1 with the launches captured
 * into one CUDA graph and replayed (what a host-free decode step does), which takes the host's
 * launch path out of the gaps between kernels.
 * *us_per_launch = event span / launches. *window_us (may be NULL) = mean in-kernel window
 * (dependency resolved or first CTA started -> last CTA done, %globaltimer) of the first 12288
 * launches. The partial-row workspace and the in-kernel clock ring are overwritten. */
int spm_time_ffn_kernel(spm_ctx* ctx, int first_layer, const float* x_norm, const int32_t* ids,
                        const float* w, int launches, int chained, double* us_per_launch,
                        double* window_us);

int spm_cache_reset(spm_ctx* ctx);                         /* cold cache, step counter, stats, events */
/* Checkpoint / resume of the expert cache (Section 3.3's availability state; integers only, no
 * weights): which expert holds which slot, LRU ticks, prefetch-origin and first-use flags, the
 * global tick and the step counter, as 2 + 4 * n_layers * slots_per_layer 64-bit words.
 * export: `state` HOST [capacity] or NULL to query; *count receives the number of words; with a
 *   buffer that is too small nothing is written and SPM_ERR_INVALID_ARG is returned. Waits for
 *   outstanding bookkeeping, not for the GPU.
 * import: into a context of the same shape (else SPM_ERR_INVALID_ARG, context unchanged): waits
 *   for both streams, installs the table, clears statistics and the event log, and copies every
 *   listed expert from the host store into its slot on the copy stream (the next launch that
 *   reads a slot waits for it as for any other copy). Decoding then continues exactly as the
 *   exporting context would have: same hits, misses, evictions, outputs. */
int spm_cache_export(spm_ctx* ctx, int64_t* state, size_t capacity, size_t* count);
int spm_cache_import(spm_ctx* ctx, const int64_t* state, size_t count);
/* Debug aid: checks the slot table's structural invariants (slot -> expert and expert -> slot are
 * inverse maps, no expert in two slots of a layer, no LRU tick ahead of the global tick) and, when
 * `with_device` is non-zero, waits for the compute stream and checks the kernels' status word
 * (bad slot number, copy or pipeline time-out). SPM_OK, or SPM_ERR_STATE / the status error with a
 * message in spm_last_error. */
int spm_check_invariants(spm_ctx* ctx, int with_device);
int spm_reset_stats(spm_ctx* ctx);                         /* counters, timings and event log only; cache kept */
int spm_get_stats(spm_ctx* ctx, spm_stats* out);           /* waits for timed work to finish */
/* Per-layer sums since the last reset: stall_us[L], ffn_us[L], and the number of steps in them. */
int spm_get_layer_times(spm_ctx* ctx, double* stall_us, double* ffn_us, uint64_t* steps);
int spm_get_events(spm_ctx* ctx, spm_event* out, size_t capacity, size_t* count);
int spm_get_slot_table(spm_ctx* ctx, int layer, int32_t* slot_expert /* host [slots] */);
int spm_synchronize(spm_ctx* ctx);                         /* both streams idle */

/* Expert FFN for callers that may not allocate (the paper has no counterpart: this is a deployment
 * convenience of this library, not part of the method).
 *
 * Some callers cannot call cudaMalloc or anything that allocates: a serving loop that has frozen
 * its memory map, a process whose device memory is owned entirely by another allocator, code that
 * must not wait on the driver's allocation lock. They cannot create an spm_ctx either (that
 * creates CUDA events and pinned memory). For them this call computes, for ONE token,
 *     h_inout += sum_{i < count} w[i] * FFN_{which[i]}(x_norm)          (SwiGLU experts, as spm_moe_ffn)
 * reading packed expert blobs in place and using no memory but its arguments and a fixed scratch
 * array of SPM_NOALLOC_SCRATCH_BYTES that is part of the library image (every GPU that loads the
 * library holds that array until the process exits). It calls no cudaMalloc, cudaFree, event or
 * stream creation, nor any other allocating routine.
 *
 *   cfg       only dtype, hidden and inter are read. hidden: a multiple of 256 (bf16) / 128 (fp32),
 *             at most SPM_NOALLOC_MAX_HIDDEN (bf16) / 1024 (fp32); larger sizes are rejected with
 *             SPM_ERR_CONFIG and a message in spm_last_error(NULL), because the scratch array holds
 *             SPM_NOALLOC_MAX_CTAS partial rows of SPM_NOALLOC_MAX_HIDDEN floats and no more.
 *   blobs     dev: n_blobs packed expert blobs back to back (layout of spm_expert_blob_bytes), 16-byte aligned
 *   which     HOST [count]: index into `blobs` of each expert to apply, count <= SPM_MAX_TOPK
 *   w         dev fp32 [count] weights;  x_norm dev fp32 [hidden];  h_inout dev fp32 [hidden]
 *             blobs, x_norm and h_inout must be 16-byte aligned (the kernels use 16-byte copies and
 *             loads), w 4-byte aligned: a view that is not (an offset slice, say) is refused with
 *             SPM_ERR_INVALID_ARG before anything is enqueued
 *   stream    cudaStream_t; the work is enqueued there and the call returns, unless
 *   wait_and_check != 0: then the call also waits for the stream and returns SPM_ERR_TIMEOUT /
 *             SPM_ERR_NOT_RESIDENT if the kernel recorded a failure.
 *
 * The first call on a device looks up the scratch array's device address and sets the kernels'
 * shared-memory attribute for that device, for every supported shape at once (the device must be
 * current); make that first call before starting any stream capture. Only that set-up takes a
 * process-wide lock; the launches and an optional wait run outside it. All calls on a device share the one array and it keeps the previous call's contents: the
 * call clears the part that must start at zero itself, but two calls whose GPU work overlaps (two
 * streams, two threads) race on it and give wrong results -- keep them on one stream or otherwise
 * serialised. */
#define SPM_NOALLOC_MAX_CTAS      148
#define SPM_NOALLOC_MAX_HIDDEN    2048
#define SPM_NOALLOC_SCRATCH_BYTES (256 + SPM_NOALLOC_MAX_CTAS * SPM_NOALLOC_MAX_HIDDEN * 4)   /* 1,212,672 B */
int spm_ffn_noalloc(const spm_model_cfg* cfg, const void* blobs, int n_blobs, const int32_t* which,
                    const float* w, int count, const float* x_norm, float* h_inout, void* stream,
                    int wait_and_check);

/* Pinned host memory for the expert store (thin wrappers over cudaHostAlloc / cudaFreeHost). */
int spm_host_alloc(size_t bytes, void** out);
int spm_host_free(void* p);

/* Host logic of the batched tensor-core kernel's work distribution, exposed for tests (no GPU
 * needed). A launch has n_units units (expert x 128 intermediate rows); phase 1 of a unit runs on
 * CTA unit % grid, phase 2 is n_dt pipeline stages (one per 128 output columns) that may be cut
 * between d-tiles and are taken, chunk by chunk in list order, by whichever CTA is free. Writes the
 * chunk list: chunks[3 * i] = {unit, dt0, dt1} = d-tiles dt0 .. dt1-1 of that unit; *count = number
 * of chunks (SPM_ERR_INVALID_ARG when capacity is too small, *count still set). */
int spm_plan_grouped_chunks(int n_units, int n_dt, int grid, int32_t* chunks, size_t capacity,
                            size_t* count);

/* ---- host-only slot-table policy (no GPU needed) ------------------------
 * The same slot table the context uses, exposed so the cache policy can be driven and checked
 * on a machine without a GPU. Arrays are host memory.                                        */
int spm_sim_create(int n_layers, int n_experts, int slots, int plain_lru, spm_sim** out);
int spm_sim_destroy(spm_sim* sim);
/* Demand of `layer`: need[count] expert ids (any order, duplicates allowed). Outputs, one entry
 * per distinct expert in processing order: expert, slot, wave index, missed flag. */
int spm_sim_demand(spm_sim* sim, int layer, const int32_t* need, int count,
                   int32_t* out_expert, int32_t* out_slot, int32_t* out_wave,
                   int32_t* out_missed, int* out_count, int* out_waves);
int spm_sim_plan(spm_sim* sim, int layer, const int32_t* order, int n_ranked, int budget,
                 int protect_all, int32_t* out_ids, int* out_count,
                 int32_t* out_protect, int* out_n_protect);
int spm_sim_prefetch(spm_sim* sim, int layer, const int32_t* ids, int count,
                     const int32_t* protect, int n_protect, int drop_modulo,
                     int32_t* out_slots /* [count], -1 = not issued */, int* out_issued);
int spm_sim_plan_only(spm_sim* sim, int layer, const int32_t* ids, int count);
int spm_sim_end_step(spm_sim* sim);
int spm_sim_events(spm_sim* sim, spm_event* out, size_t capacity, size_t* count);
int spm_sim_stats(spm_sim* sim, spm_stats* out);
int spm_sim_slot_table(spm_sim* sim, int layer, int32_t* slot_expert /* [slots] */);
/* Same checkpoint words as spm_cache_export / spm_cache_import, for the host-only table. */
int spm_sim_check(spm_sim* sim);                            /* SPM_OK, or SPM_ERR_STATE when the table's invariants fail */
int spm_sim_export(spm_sim* sim, int64_t* state, size_t capacity, size_t* count);
int spm_sim_import(spm_sim* sim, const int64_t* state, size_t count);

#ifdef __cplusplus
}
#endif
#endif /* SPM_H */
