// Fused native router + prediction adapter for one layer and nb tokens.
//
// Router (Section 3.1): x = RMSNorm(h); z = W_r x; p = softmax(z); T = Top_K(z) with ties to the
// lower id; w_e = p_e / sum_{j in T} p_j.
// Adapter (Section 3.2): u = A x; z^ = Bup u; pi^ = softmax(z^); s_e = sum over tokens of pi^_e
// in token order; the experts of the next layer are ranked by (s descending, id ascending).
//
// One thread-block cluster per token: its CTAs split the n + r weight rows (one warp per row,
// 16-byte read-only loads all issued before the first use, shuffle reduction) and store the dot
// products into the leader CTA's shared memory over DSMEM; after one cluster barrier the leader
// does the token's tails, router (softmax / Top-K) and adapter (up-projection / softmax / ranking)
// side by side on its two half-blocks. With several tokens the last leader to finish (atomic
// ticket) does the batch aggregation. Expert ids and the ranking go to the host-mapped mailbox as
// self-tagged words (sequence number in the upper half) the moment they exist, so the host can
// act on the ids while the adapter tail is still running; a fenced sequence number follows for
// callers that also read the untagged scores.
// Every reduction has a fixed order, so results are bitwise reproducible.
#pragma once

#include "ptx.cuh"
#include "../../include/spm.h"

namespace spm {

constexpr int kRouterWarps = 8;
constexpr int kRouterThreads = kRouterWarps * 32;

// Host-mapped pinned mailbox (the device writes, the host polls `seq`).
struct Mailbox {
    volatile uint32_t seq;
    uint32_t pad[3];
    int32_t ids[SPM_MAX_BATCH * SPM_MAX_TOPK];   // [nb][K]
    int32_t order[SPM_MAX_EXPERTS];              // [n]
    float scores[SPM_MAX_EXPERTS];               // [n]
};

struct RouterArgs {
    const float* h;          // [nb][D] hidden rows (do_router) ...
    const float* x_in;       // ... or already-normalised rows (adapter only)
    const float* gamma;      // [D]
    const void* router_w;    // [n][D]
    const void* adapter_a;   // [r][D]
    const void* adapter_b;   // [n][r]
    float* x_norm;           // out [nb][D]
    float* logits;           // workspace [nb][n]
    float* logits_out;       // optional copy for the caller
    float* pihat;            // workspace [nb][n]
    int32_t* ids;            // out [nb][K]
    float* w;                // out [nb][K]
    float* scores;           // out [n]
    int32_t* order;          // out [n]
    unsigned* counters;      // [1] token-leader ticket, zero between launches
    Mailbox* mailbox;        // device view of a host-mapped mailbox (may be null)
    const short* slot_map;   // optional [n] slot of each expert of this layer (device memory) ...
    short* codes_out;        // ... and where to leave the slots of the routed experts, [nb][K]
    unsigned long long* clock;   // optional {first leader past its dependency wait, last leader done} in ns
    int* status;             // optional status word: kStatusNonFinite is set when a router logit is NaN or Inf
    const float* partial;    // optional [nb][G][D] partial rows of the preceding expert kernel: the hidden row is
    int G;                   //   then h + sum of them (summed here instead of by a combine kernel) ...
    float* h_out;            //   ... and written back here ([nb][D], may alias h)
    int publish_seq;         // fence and publish the sequence number for hosts that read untagged payload
    uint32_t seq;
    int D, n, K, r, nb, renorm, do_router, do_adapter;
    float eps;
};

__device__ __forceinline__ float block_reduce(float v, float* scratch, bool is_max) {
    // fixed-shape tree: shuffle inside warps, then warp 0 over the 8 warp results
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float t = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, t) : v + t;
    }
    __syncthreads();
    if (lane == 0) scratch[wi] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int i = 1; i < kRouterWarps; ++i) r = is_max ? fmaxf(r, scratch[i]) : r + scratch[i];
    return r;
}

// softmax of v[0..n) in shared memory, in place
__device__ __forceinline__ void block_softmax(float* v, int n, float* scratch) {
    float m = -INFINITY;
    for (int e = threadIdx.x; e < n; e += kRouterThreads) m = fmaxf(m, v[e]);
    m = block_reduce(m, scratch, true);
    float s = 0.f;
    for (int e = threadIdx.x; e < n; e += kRouterThreads) {
        const float t = expf(v[e] - m);
        v[e] = t;
        s += t;
    }
    s = block_reduce(s, scratch, false);
    for (int e = threadIdx.x; e < n; e += kRouterThreads) v[e] = v[e] / s;
    __syncthreads();
}

// Order-preserving integer image of a finite float (-0 counts as +0): a < b  <=>  key(a) < key(b).
__device__ __forceinline__ int order_key(float v) {
    const int b = __float_as_int(v + 0.0f);
    return b ^ ((b >> 31) & 0x7fffffff);
}

// Position of element e in the ordering (key descending, index ascending) of k[0..n): the number
// of elements that beat it. Element j beats e when k[j] > k[e], or k[j] == k[e] and j < e, i.e.
// when k[j] > k[e] - (j < e): branch-free, four independent counters. Keys never equal INT_MIN
// (that image belongs to a NaN, and non-finite values are replaced before ranking).
__device__ __forceinline__ int rank_of_key(const int* k, int n, int e) {
    const int ke = k[e];
    int c0 = 0, c1 = 0, c2 = 0, c3 = 0, j = 0;
    if ((reinterpret_cast<uintptr_t>(k) & 15) == 0) {
#pragma unroll 4
        for (; j + 4 <= n; j += 4) {
            const int4 t = *reinterpret_cast<const int4*>(k + j);
            const int d = e - j;                       // element j + i precedes e  <=>  i < d
            c0 += t.x > ke - int(0 < d);
            c1 += t.y > ke - int(1 < d);
            c2 += t.z > ke - int(2 < d);
            c3 += t.w > ke - int(3 < d);
        }
    }
    for (; j < n; ++j) c0 += k[j] > ke - int(j < e);
    return c0 + c1 + c2 + c3;
}

constexpr int kRouterCluster = 8;   // CTAs per token, one thread-block cluster
constexpr int kStatusNonFinite = 8; // status bit (the expert kernels own bits 1, 2 and 4)
constexpr int kReduceGroupsR = 8;   // runs of partial rows (= warps of a CTA); must equal the combine kernel's group count
constexpr int kReduceChunkR = 20;   // partial rows a lane keeps in flight

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// store one float into the shared memory of CTA `rank` of this cluster (same offset as `local`)
__device__ __forceinline__ void dsmem_store(float* local, uint32_t rank, float v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local)), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <typename WT>
__device__ __forceinline__ float load_weight(const WT* p, size_t i) {
    if (sizeof(WT) == 2) return __uint_as_float(uint32_t(reinterpret_cast<const uint16_t*>(p)[i]) << 16);
    return reinterpret_cast<const float*>(p)[i];
}

// 128-thread (half-block) reduction: shuffle inside warps, 4 warp results through `slot`, one
// named barrier. Each call site uses its own `slot`, so no barrier is needed before the write.
__device__ __forceinline__ float half_reduce(float v, float* slot, bool is_max, int bar_id) {
    const int lane = threadIdx.x & 31, wq = (threadIdx.x >> 5) & 3;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float t = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, t) : v + t;
    }
    if (lane == 0) slot[wq] = v;
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    float r = slot[0];
#pragma unroll
    for (int i = 1; i < 4; ++i) r = is_max ? fmaxf(r, slot[i]) : r + slot[i];
    return r;
}

// softmax of v[0..n) in shared memory by the 128 threads of one half-block, in place
__device__ __forceinline__ void half_softmax(float* v, int n, float* slots, int bar_id) {
    const int ht = threadIdx.x & 127;
    float m = -INFINITY;
    for (int e = ht; e < n; e += 128) m = fmaxf(m, v[e]);
    m = half_reduce(m, slots, true, bar_id);
    float s = 0.f;
    for (int e = ht; e < n; e += 128) {
        const float t = expf(v[e] - m);
        v[e] = t;
        s += t;
    }
    s = half_reduce(s, slots + 4, false, bar_id);
    for (int e = ht; e < n; e += 128) v[e] = v[e] / s;
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
}

// Mailbox words carry the launch's sequence number in their upper half, so the host can tell a
// fresh word from a stale one without any fence between payload and flag.
__device__ __forceinline__ int32_t tagged(uint32_t seq, int value) { return int32_t((seq << 16) | uint32_t(value)); }

// Grid (kRouterCluster, nb), cluster (kRouterCluster, 1, 1): the CTAs of a cluster split the n + r
// weight rows of one token and deliver their dot products straight into the leader CTA's shared
// memory; after one cluster barrier the leader runs the router tail (softmax, Top-K, renormalise)
// on its first four warps and the adapter tail (up-projection, softmax, ranking) on the other four.
// MINB = 1: all registers to one CTA per SM (the fold keeps 40 partial-row quads in flight);
// MINB = 2: register budget halved so two CTAs share an SM, for batches with more CTAs than SMs.
template <typename WT, int MINB>
__global__ void __launch_bounds__(kRouterThreads, MINB)
router_adapter_kernel(const __grid_constant__ RouterArgs a) {
    constexpr int VEC = 16 / int(sizeof(WT));
    constexpr int MAXIT = 8;        // hidden <= MAXIT * 32 * VEC
    constexpr int ROWS = 3;         // weight rows a warp fetches before it starts to multiply
    extern __shared__ __align__(16) float sm[];
    float* xs = sm;                 // [D]
    float* zs = xs + a.D;           // [n] logits (leader: filled by the whole cluster)
    float* ps = zs + a.n;           // [n] router probabilities
    float* qs = ps + a.n;           // [n] adapter logits -> probabilities -> priorities
    float* us = qs + a.n;           // [r] adapter hidden (leader: filled by the whole cluster)
    float* scratch = us + a.r;      // [16] reduction slots
    float* psel = scratch + 16;                                 // [K]
    int* isel = reinterpret_cast<int*>(psel + SPM_MAX_TOPK);    // [K]
    float* bs = reinterpret_cast<float*>(isel + SPM_MAX_TOPK);  // [n * r] adapter up-projection (leader)
    float* part = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(bs + a.n * a.r) + 15) & ~uintptr_t(15));   // [kReduceGroupsR][D / cluster] group sums of partial rows
    short* smap = reinterpret_cast<short*>(part + a.D);          // [n] slot of each expert (leader)
    __shared__ int s_last;

    const int tok = blockIdx.y;
    const uint32_t cr = cluster_ctarank();
    const bool leader = cr == 0;
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    const int D = a.D, n = a.n;
    const uint32_t tag = a.seq & 0xffffu;

    grid_dep_launch();
    // every CTA of the cluster must be running before anyone writes into the leader's shared
    // memory: arrive now, wait just before the first remote store
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");

    // ---- weights first: none of them depends on the kernel before this one, so in a launch that
    // overlaps its predecessor they are already in registers (or on their way into L2) when the
    // hidden row becomes readable. Router rows then adapter-A rows, one warp per row, ROWS rows in flight.
    const int n_r = a.do_router ? n : 0;
    const int rows = n_r + (a.do_adapter ? a.r : 0);
    constexpr int STRIDE = kRouterCluster * kRouterWarps;
    const bool fused = MINB == 1 && a.partial != nullptr;   // this launch also sums the preceding expert kernel's partial rows
    uint4 v[ROWS][MAXIT];
    auto row_ptr = [&](int row) {
        return row < n_r ? static_cast<const WT*>(a.router_w) + size_t(row) * D
                         : static_cast<const WT*>(a.adapter_a) + size_t(row - n_r) * D;
    };
    auto load_rows = [&](int row0) {
#pragma unroll
        for (int rr = 0; rr < ROWS; ++rr) {
            const int row = row0 + rr * STRIDE;
#pragma unroll
            for (int it = 0; it < MAXIT; ++it) {
                const int i = (it * 32 + lane) * VEC;
                v[rr][it] = (row < rows && i < D) ? __ldg(reinterpret_cast<const uint4*>(row_ptr(row) + i)) : make_uint4(0, 0, 0, 0);
            }
        }
    };
    int row0 = int(cr) * kRouterWarps + wi;
    if (!fused) {
        load_rows(row0);
    } else {
        // the registers are needed for the partial rows first: start the weights on their way into L2
#pragma unroll
        for (int rr = 0; rr < ROWS; ++rr) {
            const int row = row0 + rr * STRIDE;
            if (row < rows)
                for (int i = lane * 128; i < D * int(sizeof(WT)); i += 32 * 128)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(row_ptr(row)) + i));
        }
    }
    constexpr int NV4 = MAXIT * 32 * VEC / (kRouterThreads * 4);   // float4 per thread at the largest hidden size
    float4 gv[NV4];
    if (a.do_router) {
#pragma unroll
        for (int c = 0; c < NV4; ++c) {
            const int i = (c * kRouterThreads + threadIdx.x) * 4;
            if (i < D) gv[c] = *reinterpret_cast<const float4*>(a.gamma + i);
        }
    }
    // leader: the small adapter up-projection and the slot map are needed only in the tail
    if (leader && a.do_adapter) {
        const WT* B = static_cast<const WT*>(a.adapter_b);
        for (int i = threadIdx.x; i < n * a.r; i += kRouterThreads) bs[i] = load_weight(B, i);
    }
    if (leader && a.slot_map)
        for (int i = threadIdx.x; i < n; i += kRouterThreads) smap[i] = a.slot_map[i];

    // ---- router input: the hidden row (written by the preceding kernels) is normalised ----------
    grid_dep_wait();
    if (a.clock && leader && threadIdx.x == 0) atomicMin(a.clock, global_timer_ns());
    bool cluster_started = false;      // the start-of-kernel cluster barrier has been waited for
    if constexpr (MINB == 1) if (fused) {
        // h = h + sum over the expert kernel's CTAs of their partial rows, in the combine kernel's
        // order: kReduceGroupsR runs of consecutive rows, each summed front to back, the runs then
        // added in order, the residual last. This CTA owns D / cluster columns; warp g sums run g.
        const int slice = D / kRouterCluster, nq = slice / 4;
        const int col0 = int(cr) * slice;
        const int per = (a.G + kReduceGroupsR - 1) / kReduceGroupsR;
        const int c0 = wi * per, c1 = min(a.G, c0 + per);
        float hin = 0.f;
        if (threadIdx.x < slice) hin = a.h[size_t(tok) * D + col0 + threadIdx.x];
        const float* pbase = a.partial + size_t(tok) * a.G * D + col0;
        // a lane owns column quads lane and lane + 32 of the slice; all rows of its run are in
        // flight together for both before the first addition
        constexpr int QPL = 2;
        for (int r0 = c0; r0 < c1 || r0 == c0; r0 += kReduceChunkR) {
            float4 t[QPL][kReduceChunkR];
#pragma unroll
            for (int j = 0; j < QPL; ++j) {
                const int q = lane + 32 * j;
#pragma unroll
                for (int i = 0; i < kReduceChunkR; ++i)
                    t[j][i] = (q < nq && r0 + i < c1) ? __ldcg(reinterpret_cast<const float4*>(pbase + size_t(r0 + i) * D) + q)
                                                      : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < QPL; ++j) {
                const int q = lane + 32 * j;
                if (q >= nq) continue;
                float4 acc = r0 == c0 ? make_float4(0.f, 0.f, 0.f, 0.f) : *reinterpret_cast<const float4*>(part + wi * slice + q * 4);
#pragma unroll
                for (int i = 0; i < kReduceChunkR; ++i) { acc.x += t[j][i].x; acc.y += t[j][i].y; acc.z += t[j][i].z; acc.w += t[j][i].w; }
                *reinterpret_cast<float4*>(part + wi * slice + q * 4) = acc;
            }
        }
        __syncthreads();
        asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
        cluster_started = true;
        if (threadIdx.x < slice) {
            float tot = part[threadIdx.x];
#pragma unroll
            for (int g = 1; g < kReduceGroupsR; ++g) tot += part[g * slice + threadIdx.x];
            const float hv1 = hin + tot;
            a.h_out[size_t(tok) * D + col0 + threadIdx.x] = hv1;
#pragma unroll
            for (uint32_t dst = 0; dst < kRouterCluster; ++dst) dsmem_store(xs + col0 + threadIdx.x, dst, hv1);
        }
        load_rows(row0);                 // L2 hits by now; in flight across the barrier and the normalisation
        cluster_sync_all();              // every CTA holds the whole updated row in xs
    }
    if (a.do_router) {
        const float* ht = fused ? xs : a.h + size_t(tok) * D;
        float4 hv[NV4];
#pragma unroll
        for (int c = 0; c < NV4; ++c) {
            const int i = (c * kRouterThreads + threadIdx.x) * 4;
            if (i < D) hv[c] = *reinterpret_cast<const float4*>(ht + i);
        }
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < NV4; ++c) {
            const int i = (c * kRouterThreads + threadIdx.x) * 4;
            if (i < D) {
                ss = fmaf(hv[c].x, hv[c].x, ss); ss = fmaf(hv[c].y, hv[c].y, ss);
                ss = fmaf(hv[c].z, hv[c].z, ss); ss = fmaf(hv[c].w, hv[c].w, ss);
            }
        }
        ss = block_reduce(ss, scratch, false);
        const float inv = 1.0f / sqrtf(ss / float(D) + a.eps);
#pragma unroll
        for (int c = 0; c < NV4; ++c) {
            const int i = (c * kRouterThreads + threadIdx.x) * 4;
            if (i < D) {
                float4 o;
                o.x = hv[c].x * gv[c].x * inv; o.y = hv[c].y * gv[c].y * inv;
                o.z = hv[c].z * gv[c].z * inv; o.w = hv[c].w * gv[c].w * inv;
                *reinterpret_cast<float4*>(xs + i) = o;
                if (leader && a.x_norm) *reinterpret_cast<float4*>(a.x_norm + size_t(tok) * D + i) = o;
            }
        }
    } else {
        const float* xt = a.x_in + size_t(tok) * D;
        for (int i = threadIdx.x; i < D; i += kRouterThreads) xs[i] = xt[i];
    }
    __syncthreads();

    if (!cluster_started) asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
    while (row0 < rows) {
        // per row the products are accumulated in element order; the rows of a batch share each
        // 16-byte read of the activations
        float acc[ROWS];
#pragma unroll
        for (int rr = 0; rr < ROWS; ++rr) acc[rr] = 0.f;
#pragma unroll
        for (int it = 0; it < MAXIT; ++it) {
            const int i = (it * 32 + lane) * VEC;
            if (i < D) {
                float xv[VEC];
#pragma unroll
                for (int q = 0; q < VEC; q += 4) {
                    const float4 t = *reinterpret_cast<const float4*>(xs + i + q);
                    xv[q] = t.x; xv[q + 1] = t.y; xv[q + 2] = t.z; xv[q + 3] = t.w;
                }
#pragma unroll
                for (int rr = 0; rr < ROWS; ++rr) {
                    float f[VEC];
                    unpack16(v[rr][it], f);
#pragma unroll
                    for (int q = 0; q < VEC; ++q) acc[rr] = fmaf(f[q], xv[q], acc[rr]);
                }
            }
        }
#pragma unroll
        for (int rr = 0; rr < ROWS; ++rr) {
            const int row = row0 + rr * STRIDE;
            const float tot = warp_sum(acc[rr]);
            if (row < rows && lane == 0) dsmem_store(row < n_r ? zs + row : us + (row - n_r), 0, tot);
        }
        row0 += ROWS * STRIDE;
        if (row0 < rows) load_rows(row0);
    }
    cluster_sync_all();
    if (!leader) return;

    // ---- tails (leader CTA): router on warps 0-3, adapter on warps 4-7, concurrently ----------
    Mailbox* mb = a.mailbox;
    const int half = threadIdx.x >> 7, ht = threadIdx.x & 127;
    if (half == 0 && a.do_router) {
        if (ht < a.K) { isel[ht] = 0; psel[ht] = 0.f; }     // stays in range even if NaN logits leave a rank unfilled
        for (int e = ht; e < n; e += 128) {
            float z = zs[e];
            if (!isfinite(z)) {      // ids of this token are meaningless then; keep the ordering total so every rank is filled
                if (a.status) atomicOr(a.status, kStatusNonFinite);
                z = -3.0e38f;
            }
            ps[e] = z;
            reinterpret_cast<int*>(zs)[e] = order_key(z);       // the ranking below works on these
            a.logits[size_t(tok) * n + e] = z;
            if (a.logits_out) a.logits_out[size_t(tok) * n + e] = z;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        half_softmax(ps, n, scratch, 1);          // ps = p, zs = order keys of z (ranking is taken on the logits)
        for (int e = ht; e < n; e += 128) {
            const int rk = rank_of_key(reinterpret_cast<const int*>(zs), n, e);
            if (rk < a.K) { isel[rk] = e; psel[rk] = ps[e]; }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ht < a.K) {
            float tot = 0.f;
            for (int k = 0; k < a.K; ++k) tot += psel[k];
            a.ids[size_t(tok) * a.K + ht] = isel[ht];
            a.w[size_t(tok) * a.K + ht] = a.renorm ? psel[ht] / tot : psel[ht];
            if (mb) mb->ids[tok * a.K + ht] = tagged(tag, isel[ht]);      // the host may start on these at once
            // slot numbers for an expert kernel that follows without a host turn
            if (a.codes_out) a.codes_out[tok * a.K + ht] = smap[isel[ht]];
        }
    }
    if (half == 1 && a.do_adapter) {
        for (int e = ht; e < n; e += 128) {
            float acc = 0.f;
            for (int q = 0; q < a.r; ++q) acc = fmaf(bs[e * a.r + q], us[q], acc);
            if (!isfinite(acc)) {
                if (a.status) atomicOr(a.status, kStatusNonFinite);
                acc = -3.0e38f;
            }
            qs[e] = acc;
        }
        asm volatile("bar.sync 2, 128;" ::: "memory");
        half_softmax(qs, n, scratch + 8, 2);
        if (a.nb > 1) {
            for (int e = ht; e < n; e += 128) a.pihat[size_t(tok) * n + e] = qs[e];
        } else {
            for (int e = ht; e < n; e += 128) {        // one token: its distribution is the priority vector
                const int rk = rank_of_key(reinterpret_cast<const int*>(qs), n, e);   // non-negative floats order like their bits
                a.order[rk] = e;
                a.scores[e] = qs[e];
                if (mb) { mb->order[rk] = tagged(tag, e); mb->scores[e] = qs[e]; }
            }
        }
    }

    // ---- several tokens: the last leader to finish aggregates and ranks -------------------------
    if (a.nb > 1) {
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            if (a.clock) atomicMax(a.clock + 1, global_timer_ns());
            s_last = atomicAdd(&a.counters[0], 1u) == unsigned(a.nb - 1);
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        if (a.do_adapter) {
            for (int e = threadIdx.x; e < n; e += kRouterThreads) {
                float s = 0.f;
                for (int t = 0; t < a.nb; ++t) s += __ldcg(a.pihat + size_t(t) * n + e);
                qs[e] = s;
            }
            __syncthreads();
            for (int e = threadIdx.x; e < n; e += kRouterThreads) {
                const int rk = rank_of_key(reinterpret_cast<const int*>(qs), n, e);
                a.order[rk] = e;
                a.scores[e] = qs[e];
                if (mb) { mb->order[rk] = tagged(tag, e); mb->scores[e] = qs[e]; }
            }
        }
        if (threadIdx.x == 0) a.counters[0] = 0u;
    }
    // final flag for callers that read untagged payload (scores): fence, then the sequence number
    if (a.publish_seq) {
        __threadfence_system();
        __syncthreads();
        if (threadIdx.x == 0 && mb) mb->seq = a.seq;
    }
    if (threadIdx.x == 0 && a.clock) atomicMax(a.clock + 1, global_timer_ns());
}

inline size_t router_smem_bytes(int D, int n, int r) {
    return sizeof(float) * (2 * size_t(D) + 3 * size_t(n) + size_t(r) + 16 + 2 * SPM_MAX_TOPK + size_t(n) * r) +
           ((size_t(n) * sizeof(short) + 15) & ~size_t(15)) + 16;
}

}  // namespace spm
