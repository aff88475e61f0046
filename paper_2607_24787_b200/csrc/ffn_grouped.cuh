// Batched decode: slot-indexed grouped SwiGLU expert FFN on the 5th-generation tensor cores.
//
// When several sequences are decoded per step, the tokens routed to one expert form a small
// dense problem  G = X_e Wg^T, U = X_e Wu^T, A = silu(G)*U*w, Y_e = A Wd^T.  Weights stay the
// streamed operand (they go on the M side of the MMA, 128 rows at a time, read once from their
// cache slot by TMA), the expert's tokens (padded to 64) are the N side, accumulators live in
// TMEM. Activations are rounded to bf16 for the tensor cores; accumulation is fp32.
//
// Unit of work = (expert, 128 intermediate rows j). For a unit the CTA
//   phase 1: streams gate[j][:] and up[j][:] over K = hidden in 64-wide blocks together with
//            the matching block of the expert's token rows, accumulating G^T, U^T [128 x 64] in TMEM;
//            the epilogue warps read them, apply silu * up * routing weight, and write A^T as bf16
//            into shared memory (N-contiguous, 128-byte swizzle);
//   phase 2: streams column j of W_down for 128 hidden units d at a time ([128 j x 128 d], d
//            contiguous = an M-major A operand) and multiplies by A^T (K = the 128 j), one
//            accumulator [128 d x 64 tokens] per d-tile, double buffered; the epilogue writes the
//            rows of real tokens to the partial buffer P[j-tile][token row][d].
// A combine kernel then adds, per token, its K experts x (I/128) partial rows and the residual in
// a fixed order.
//
// Work is handed out as tasks, so that a launch with few units (a wave of 32 experts is 192 units
// on 148 SMs) still keeps every SM streaming until the end: a P1 task is phase 1 of one unit, a P2
// task ("chunk") is phase 2 of one unit for a range of d-tiles. P1 tasks are static: CTA b runs the
// units b, b + grid, ... first. P2 chunks are then taken from one list in order through an atomic
// counter, by whichever CTA is free: a chunk's output tiles are its own and are computed by the same
// sequence of MMAs whoever runs it, so results do not depend on who took what. A^T travels from the
// CTA that ran P1 to the CTA(s) that run P2 through a 16 KB slot of global memory (L2-resident)
// guarded by a per-unit arrival counter: the P1 epilogue warps store their rows, fence, and bump the
// counter; the P2 side's producer warp polls it (bounded), then pulls the slot into shared memory
// with one bulk copy. Every CTA finishes its P1 tasks before it takes its first chunk, so no CTA
// ever waits for a counter while its owner waits for it. The host cuts the chunks finer towards the
// end of the list (gg_plan_chunks) so that all CTAs finish together; without a list a chunk is a
// whole unit. The producer warp tells the other warps of its CTA what it took through a small queue
// in shared memory.
// One warp issues TMA, one thread issues tcgen05.mma, four warps run the epilogues;
// all of them talk through mbarriers, every wait is bounded and an abort flag lets the whole CTA
// leave together (freeing its TMEM) if a wait ever gives up. No multicast anywhere.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include "ptx.cuh"
#include "ffn_gemv.cuh"      // kWaitLimitNs, kernel status bits
#include "../../include/spm.h"

namespace spm {

constexpr int kGgThreads = 192;          // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int kGgStages = 5;
constexpr int kGgTokens = 64;            // N of every MMA: an expert's tokens, zero/garbage padded
constexpr int kGgTileRows = 128;         // M of every MMA
constexpr int kGgKBlock = 64;            // bf16 elements per 128-byte swizzled row
constexpr uint32_t kGgTileBytes = kGgTileRows * 128;          // one [128 x 128 B] weight box
constexpr uint32_t kGgXBytes = kGgTokens * 128;               // one [64 x 128 B] token box
constexpr uint32_t kGgStageBytes = 2 * kGgTileBytes + kGgXBytes;   // 40 KB
constexpr uint32_t kGgActBytes = kGgTileRows * 128;           // A^T: [128 j][64 tokens] bf16
constexpr uint32_t kGgTmemCols = 512;    // two (G^T, U^T) pairs at 0..127 and 128..255, Y tiles at 256..319 and 320..383
constexpr int kStatusGroupedTimeout = 4;

struct GgUnit {
    int32_t slot;      // global slot index (layer * slots + slot): 4th coordinate of the weight map
    int32_t jt;        // 128-row tile of the intermediate dimension
    int32_t row0;      // first row of this expert in the sorted token-row arrays
    int32_t ntok;      // tokens of this expert (1..64)
};

// One task of a CTA: phase 1 of `unit` (dt0 < 0), or phase 2 of `unit` for d-tiles dt0 .. dt1-1;
// unit < 0 ends the list.
struct GgTask {
    int32_t unit;
    int16_t dt0, dt1;
};
// Optional device-side wait of a unit: its expert's copy has landed once ready[watch] has reached `want`
// (the arrival counter of the slot that leads the batch of copies); watch < 0: nothing to wait for.
struct GgWait {
    int32_t watch;
    uint32_t want;
};
constexpr int kGgActReady = 4;           // arrivals (one per epilogue warp) that complete a unit's A^T
constexpr int kGgQueue = 4;              // tasks the producer warp may be ahead of the other warps

struct GgArgs {
    const GgUnit* units;
    int n_units;           // ... or, when n_units_dev is set, read from device memory (plan built on the device)
    const int* n_units_dev;
    const float* wrow;     // [rows] routing weight of each sorted token row
    float* partial;        // [I/128][rows_cap][D]
    int rows_cap;
    int D, I;
    int* status;
    unsigned long long wait_limit_ns;   // pipeline waits give up after this long (0: the 2 s default)
    // bf16 kernel only: the list of P2 chunks (null: one chunk per unit), the counter they are taken with,
    // the A^T slots and their arrival counters
    const GgTask* chunks;
    int n_chunks;              // (ignored without a list: the number of units)
    int* next_chunk;           // zeroed before the launch (by the gather kernel), like act_ready
    unsigned char* act_g;      // [units][16 KB] A^T of each unit, in the shared-memory operand layout
    int* act_ready;            // [units]
    unsigned long long* clock; // optional {earliest CTA past its dependency wait, latest CTA end} in ns (globaltimer)
    // optional device-side waiting: per unit, what its expert's copy is awaited by; the arrival counters of all slots
    const GgWait* unit_wait;
    const unsigned* ready;
};

// ---- tcgen05 / TMA wrappers ---------------------------------------------------
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]; bf16 inputs, fp32 accumulate; one thread issues.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// this thread's TMEM lane, 16 consecutive fp32 columns
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte offsets
// in 16-byte units, version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= uint64_t((addr >> 4) & 0x3fff);
    d |= uint64_t((lbo_bytes >> 4) & 0x3fff) << 16;
    d |= uint64_t((sbo_bytes >> 4) & 0x3fff) << 32;
    d |= uint64_t(1) << 46;      // descriptor version
    d |= uint64_t(2) << 61;      // SWIZZLE_128B
    return d;
}

// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 64, operand majors as given.
__host__ __device__ constexpr uint32_t gg_idesc(bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(a_mn_major) << 15) | (uint32_t(b_mn_major) << 16) |
           (uint32_t(kGgTokens >> 3) << 17) | (uint32_t(kGgTileRows >> 4) << 24);
}

// The same with N given at run time (a multiple of 16, at most kGgTokens): a unit with few tokens
// asks the tensor core for only that many columns.
__device__ __forceinline__ uint32_t gg_idesc_n(bool a_mn_major, bool b_mn_major, uint32_t n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(a_mn_major) << 15) | (uint32_t(b_mn_major) << 16) |
           ((n >> 3) << 17) | (uint32_t(kGgTileRows >> 4) << 24);
}
__device__ __forceinline__ uint32_t gg_pad_tokens(int ntok) { return uint32_t(max(16, (ntok + 15) & ~15)); }

// Token-row tensor maps with boxes of 16, 32 and 64 rows: a unit with few tokens brings only the
// rows its MMAs read. gg_token_box() picks the map, gg_token_rows() is the row count of its box.
struct GgTokenMaps {
    CUtensorMap m[3];
};
__device__ __forceinline__ int gg_token_box(int ntok) { return ntok <= 16 ? 0 : ntok <= 32 ? 1 : 2; }
__device__ __forceinline__ uint32_t gg_token_rows(int box) { return 16u << box; }

struct GgAbort {
    volatile int* flag;     // shared: set by the first wait that gives up
    int* status;
    unsigned long long limit_ns;
};

// bounded wait that also leaves when another role of the CTA has given up
__device__ __forceinline__ bool gg_wait(uint32_t bar, uint32_t parity, const GgAbort& ab) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*ab.flag) return false;
        if (global_timer_ns() - t0 > ab.limit_ns) {
            *ab.flag = 1;
            atomicOr(ab.status, kStatusGroupedTimeout);
            return false;
        }
    }
}

// bounded wait for the copy stream's arrival counter of a batch of expert copies (written from outside the GPU's
// kernels, hence system scope); the weights are then read through the async proxy
__device__ __forceinline__ bool gg_wait_arrival(const unsigned* p, unsigned want, const GgAbort& ab) {
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        unsigned v;
        asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
        if (int(v - want) >= 0) break;
        if (*ab.flag) return false;
        if (global_timer_ns() - t0 > ab.limit_ns) {
            *ab.flag = 1;
            atomicOr(ab.status, kStatusCopyTimeout);
            return false;
        }
        __nanosleep(200);
    }
    asm volatile("fence.proxy.async;" ::: "memory");
    return true;
}

// bounded wait for a counter in global memory (another CTA's arrivals) to reach `want`
__device__ __forceinline__ bool gg_wait_count(const int* p, int want, const GgAbort& ab) {
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
        if (v >= want) return true;
        if (*ab.flag) return false;
        if (global_timer_ns() - t0 > ab.limit_ns) {
            *ab.flag = 1;
            atomicOr(ab.status, kStatusGroupedTimeout);
            return false;
        }
        __nanosleep(100);
    }
}

__global__ void __launch_bounds__(kGgThreads, 1)
ffn_grouped_kernel(const __grid_constant__ CUtensorMap wmap, const __grid_constant__ GgTokenMaps xmaps, const GgArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // 1024-byte alignment is what the 128-byte swizzle atoms need
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* stages = smem;                                   // kGgStages x 40 KB
    unsigned char* act = smem + kGgStages * kGgStageBytes;          // 16 KB
    uint64_t* bars = reinterpret_cast<uint64_t*>(act + kGgActBytes);
    uint64_t* full = bars;                    // [stages]  TMA -> MMA
    uint64_t* empty = full + kGgStages;       // [stages]  MMA -> TMA
    uint64_t* acc1_full = empty + kGgStages;  // [2] MMA -> epilogue: G^T, U^T of a unit complete
    uint64_t* acc1_empty = acc1_full + 2;     // [2] epilogue -> MMA: that pair drained
    uint64_t* act_full = acc1_empty + 2;      // TMA -> MMA: A^T of the P2 task's unit has landed in shared memory
    uint64_t* act_empty = act_full + 1;       // MMA -> TMA: the P2 task has consumed A^T
    uint64_t* acc2_full = act_empty + 1;      // [2] MMA -> epilogue
    uint64_t* acc2_empty = acc2_full + 2;     // [2] epilogue -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc2_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* wrow_all = reinterpret_cast<float*>(tmem_slot + 4);      // [4 epilogue warps][64]
    uint64_t* q_full = reinterpret_cast<uint64_t*>(wrow_all + 4 * kGgTokens);   // [kGgQueue] producer -> MMA, epilogue warps
    uint64_t* q_empty = q_full + kGgQueue;                                      // [kGgQueue] they -> producer
    GgTask* queue = reinterpret_cast<GgTask*>(q_empty + kGgQueue);              // [kGgQueue]

    grid_dep_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = a.D;
    const int n_kb = D / kGgKBlock;            // phase-1 stages per unit
    const int n_dt = D / kGgTileRows;          // phase-2 stages per unit
    GgAbort ab{abort_flag, a.status, a.wait_limit_ns ? a.wait_limit_ns : kWaitLimitNs};

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGgStages; ++s) { mbar_init(smem_u32(full + s), 1); mbar_init(smem_u32(empty + s), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(acc1_full + b), 1);
            mbar_init(smem_u32(acc1_empty + b), 4);     // one arrival per epilogue warp
            mbar_init(smem_u32(acc2_full + b), 1);
            mbar_init(smem_u32(acc2_empty + b), 4);
        }
        mbar_init(smem_u32(act_full), 1);        // the producer's arrival + the bytes of the A^T bulk copy
        for (int i = 0; i < kGgQueue; ++i) { mbar_init(smem_u32(q_full + i), 1); mbar_init(smem_u32(q_empty + i), 5); }
        mbar_init(smem_u32(act_empty), 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kGgTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // barriers and TMEM are set up; everything below reads what the preceding kernels wrote
    grid_dep_wait();
    if (a.clock && threadIdx.x == 0) atomicMin(a.clock, global_timer_ns());
    const int n_units = a.n_units_dev ? __ldcg(a.n_units_dev) : a.n_units;
    // P1 tasks of this CTA: the units b, b + grid, ...; P2 chunks: taken from the common list.
    const int my_units = int(blockIdx.x) < n_units ? (n_units - 1 - int(blockIdx.x)) / int(gridDim.x) + 1 : 0;
    const int n_chunks = a.chunks ? a.n_chunks : n_units;
    // consumer side of the task queue (MMA warp and epilogue warps): next task, or unit < 0 at the end / after an abort
    uint32_t n_got = 0;
    auto next_task = [&]() -> GgTask {
        const uint32_t qs = n_got % kGgQueue;
        if (!__all_sync(0xffffffffu, gg_wait(smem_u32(q_full + qs), (n_got / kGgQueue) & 1, ab))) return GgTask{-1, 0, 0};
        const GgTask tk = queue[qs];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(q_empty + qs));
        ++n_got;
        return tk;
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        // The producer and the MMA issuer are walked by their whole warp in uniform control flow and
        // one elected lane issues: addresses and descriptors then stay in uniform registers (issued
        // from inside a one-lane branch, each tcgen05.mma cost the issuing thread about 90 cycles).
        uint32_t it = 0;      // ring position over all stages
        uint32_t n_p2 = 0;    // P2 tasks started
        uint32_t n_pub = 0;   // tasks published to the other warps
        bool ok = true;
        auto stage_free = [&](uint32_t s) {
            if (it >= kGgStages) ok = __all_sync(0xffffffffu, gg_wait(smem_u32(empty + s), ((it / kGgStages) - 1) & 1, ab));
        };
        auto publish = [&](GgTask tk) {
            const uint32_t qs = n_pub % kGgQueue;
            if (n_pub >= kGgQueue) ok = __all_sync(0xffffffffu, gg_wait(smem_u32(q_empty + qs), ((n_pub / kGgQueue) - 1) & 1, ab));
            if (ok && lane == 0) {
                queue[qs] = tk;
                mbar_arrive(smem_u32(q_full + qs));       // (release: the entry is visible to whoever sees the arrival)
            }
            __syncwarp();
            ++n_pub;
        };
        // ---- P1: gate / up rows of this CTA's own units
        for (int i = 0; i < my_units && ok; ++i) {
            const int32_t u = int32_t(blockIdx.x + i * gridDim.x);
            publish(GgTask{u, -1, -1});
            if (!ok) break;
            const GgUnit un = a.units[u];
            if (a.unit_wait) {       // the expert's copy may still be on its way: wait for it here, not on the host
                const GgWait uw = a.unit_wait[u];
                if (uw.watch >= 0) ok = __all_sync(0xffffffffu, gg_wait_arrival(a.ready + uw.watch, uw.want, ab));
                if (!ok) break;
            }
            const int xbox = gg_token_box(un.ntok);
            const CUtensorMap* xmap = &xmaps.m[xbox];
            const uint32_t x_bytes = gg_token_rows(xbox) * 128;
            for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
                const uint32_t s = it % kGgStages;
                stage_free(s);
                if (!ok) break;
                const uint32_t base = smem_u32(stages + s * kGgStageBytes);
                const uint32_t fb = smem_u32(full + s);
                if (elect_one()) {
                    mbar_arrive_expect_tx(fb, 2 * kGgTileBytes + x_bytes);
                    tma_load_4d(base, &wmap, kb * kGgKBlock, 0, un.jt * kGgTileRows, un.slot, fb);                 // gate rows
                    tma_load_4d(base + kGgTileBytes, &wmap, kb * kGgKBlock, 1, un.jt * kGgTileRows, un.slot, fb);  // up rows
                    tma_load_2d(base + 2 * kGgTileBytes, xmap, kb * kGgKBlock, un.row0, fb);                      // token rows
                }
                __syncwarp();
            }
        }
        // ---- P2: W_down tiles, chunk by chunk from the common list
        while (ok) {
            int idx = 0;
            if (lane == 0) idx = atomicAdd(a.next_chunk, 1);
            idx = __shfl_sync(0xffffffffu, idx, 0);
            if (idx >= n_chunks) break;
            const GgTask tk = a.chunks ? a.chunks[idx] : GgTask{idx, 0, int16_t(n_dt)};
            publish(tk);
            if (!ok) break;
            const GgUnit un = a.units[tk.unit];
            if (a.unit_wait) {       // the tiles below are requested before the unit's A^T (and with it its expert's arrival) is known
                const GgWait uw = a.unit_wait[tk.unit];
                if (uw.watch >= 0) ok = __all_sync(0xffffffffu, gg_wait_arrival(a.ready + uw.watch, uw.want, ab));
                if (!ok) break;
            }
            // The first ring-full of tiles is issued before A^T is fetched: those stage slots are freed by
            // MMAs of earlier tasks only, so the weight stream does not pause while this warp waits for the
            // preceding chunk's MMAs and for the unit's arrival counter.
            auto load_w = [&](int dt) {
                const uint32_t s = it % kGgStages;
                stage_free(s);
                if (!ok) return;
                const uint32_t base = smem_u32(stages + s * kGgStageBytes);
                const uint32_t fb = smem_u32(full + s);
                if (elect_one()) {
                    mbar_arrive_expect_tx(fb, 2 * kGgTileBytes);
                    tma_load_4d(base, &wmap, dt * kGgTileRows, 2, un.jt * kGgTileRows, un.slot, fb);                      // d 0..63
                    tma_load_4d(base + kGgTileBytes, &wmap, dt * kGgTileRows + 64, 2, un.jt * kGgTileRows, un.slot, fb); // d 64..127
                }
                __syncwarp();
                ++it;
            };
            int dt = tk.dt0;
            for (int pre = 0; pre < kGgStages && dt < tk.dt1 && ok; ++pre, ++dt) load_w(dt);
            if (ok && n_p2 > 0) ok = __all_sync(0xffffffffu, gg_wait(smem_u32(act_empty), (n_p2 - 1) & 1, ab));
            if (ok) ok = __all_sync(0xffffffffu, gg_wait_count(a.act_ready + tk.unit, kGgActReady, ab));
            if (!ok) break;
            if (elect_one()) {
                asm volatile("fence.proxy.async;" ::: "memory");     // A^T was written with ordinary stores, is read by a bulk copy
                mbar_arrive_expect_tx(smem_u32(act_full), kGgActBytes);
                bulk_g2s_plain(smem_u32(act), a.act_g + size_t(tk.unit) * kGgActBytes, kGgActBytes, smem_u32(act_full));
            }
            __syncwarp();
            ++n_p2;
            for (; dt < tk.dt1 && ok; ++dt) load_w(dt);
        }
        if (ok) publish(GgTask{-1, 0, 0});
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        uint32_t it = 0, nd = 0, n_p1 = 0, n_p2 = 0;     // stage, d-tile, P1 and P2 counters
        bool ok = true;
        auto wait_all = [&](uint64_t* bar, uint32_t parity) { ok = __all_sync(0xffffffffu, ok && gg_wait(smem_u32(bar), parity, ab)); };
        while (ok) {
            const GgTask tk = next_task();
            if (tk.unit < 0) break;
            const uint32_t n_pad = gg_pad_tokens(a.units[tk.unit].ntok);
            if (tk.dt0 < 0) {
                const uint32_t b = n_p1 & 1, m = n_p1 >> 1;
                // weights K-major, tokens K-major; N = the unit's tokens rounded up to 16
                const uint32_t idesc1 = gg_idesc_n(false, false, n_pad);
                if (n_p1 >= 2) wait_all(acc1_empty + b, (m - 1) & 1);   // pair drained two P1 tasks ago
                const uint32_t acc = tmem + 128 * b;
                for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
                    const uint32_t s = it % kGgStages;
                    wait_all(full + s, (it / kGgStages) & 1);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t base = smem_u32(stages + s * kGgStageBytes);
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {      // 4 x (K = 16) inside the 64-wide block
                            const uint64_t bx = smem_desc_sw128(base + 2 * kGgTileBytes + ks * 32, 16, 1024);
                            tc_mma_bf16(acc, smem_desc_sw128(base + ks * 32, 16, 1024), bx, idesc1, (kb | ks) != 0);
                            tc_mma_bf16(acc + 64, smem_desc_sw128(base + kGgTileBytes + ks * 32, 16, 1024), bx, idesc1, (kb | ks) != 0);
                        }
                        tc_commit(smem_u32(empty + s));
                    }
                    __syncwarp();
                }
                if (ok && elect_one()) tc_commit(smem_u32(acc1_full + b));
                __syncwarp();
                ++n_p1;
                continue;
            }
            // W_down column tile M-major, A^T N-major
            const uint32_t idesc2 = gg_idesc_n(true, true, n_pad);
            wait_all(act_full, n_p2 & 1);
            if (!ok) break;
            tc_fence_after();
            const uint32_t act_addr = smem_u32(act);
            for (int dt = tk.dt0; dt < tk.dt1 && ok; ++dt, ++it, ++nd) {
                const uint32_t s = it % kGgStages, b = nd & 1;
                wait_all(full + s, (it / kGgStages) & 1);
                if (nd >= 2) wait_all(acc2_empty + b, ((nd >> 1) - 1) & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t base = smem_u32(stages + s * kGgStageBytes);
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {      // K = 16 rows j per step, 2048 bytes of each operand
                        const uint64_t da = smem_desc_sw128(base + ks * 2048, kGgTileBytes, 1024);
                        const uint64_t db = smem_desc_sw128(act_addr + ks * 2048, kGgActBytes, 1024);
                        tc_mma_bf16(tmem + 256 + 64 * b, da, db, idesc2, ks != 0);
                    }
                    tc_commit(smem_u32(empty + s));
                    tc_commit(smem_u32(acc2_full + b));
                }
                __syncwarp();
            }
            if (ok && elect_one()) tc_commit(smem_u32(act_empty));
            __syncwarp();
            ++n_p2;
        }
    } else {
        // ---------------- epilogue warps (TMEM lane quarter = warp % 4) ----------------
        const int q = warp & 3;
        const int row = q * 32 + lane;                  // accumulator row handled by this thread
        const uint32_t lane_addr = uint32_t(q * 32) << 16;
        float* wrow_s = wrow_all + q * kGgTokens;       // this warp's copy: no cross-warp barrier needed
        uint32_t nd = 0, n_p1 = 0;
        bool ok = true;
        while (ok) {
            const GgTask tk = next_task();
            if (tk.unit < 0) break;
            const GgUnit un = a.units[tk.unit];
            if (tk.dt0 < 0) {
                const uint32_t b1 = n_p1 & 1;
                // routing weights of this expert's token rows (0 beyond the real tokens)
                __syncwarp();
#pragma unroll
                for (int t = lane; t < kGgTokens; t += 32) wrow_s[t] = t < un.ntok ? a.wrow[un.row0 + t] : 0.f;
                __syncwarp();
                ok = __all_sync(0xffffffffu, gg_wait(smem_u32(acc1_full + b1), (n_p1 >> 1) & 1, ab));
                if (!ok) break;
                tc_fence_after();
                // A^T[j = row][t] = silu(G) * U * w_t, bf16, 16-byte chunks swizzled by (row % 8): the layout
                // the second GEMM's B operand has in shared memory, stored to the unit's slot in global memory
                const int n_pad = int(gg_pad_tokens(un.ntok));      // columns the MMAs of this unit wrote
                unsigned char* rowp = a.act_g + size_t(tk.unit) * kGgActBytes + row * 128;
#pragma unroll
                for (int c = 0; c < kGgTokens / 16; ++c) {
                    if (c * 16 >= n_pad) break;
                    float g[16], up[16];
                    tmem_ld16(tmem + lane_addr + 128 * b1 + c * 16, g);
                    tmem_ld16(tmem + lane_addr + 128 * b1 + 64 + c * 16, up);
                    uint32_t packed[8];
#pragma unroll
                    for (int k2 = 0; k2 < 8; ++k2) {
                        const float a0 = g[2 * k2] / (1.f + expf(-g[2 * k2])) * up[2 * k2] * wrow_s[c * 16 + 2 * k2];
                        const float a1 = g[2 * k2 + 1] / (1.f + expf(-g[2 * k2 + 1])) * up[2 * k2 + 1] * wrow_s[c * 16 + 2 * k2 + 1];
                        const __nv_bfloat162 p = __floats2bfloat162_rn(a0, a1);
                        packed[k2] = *reinterpret_cast<const uint32_t*>(&p);
                    }
                    *reinterpret_cast<uint4*>(rowp + (((2 * c) ^ (row & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    *reinterpret_cast<uint4*>(rowp + (((2 * c + 1) ^ (row & 7)) << 4)) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
                }
                tc_fence_before();
                __syncwarp();                   // the warp's 32 rows are written ...
                if (lane == 0) {
                    mbar_arrive(smem_u32(acc1_empty + b1));
                    __threadfence();            // ... and made visible device-wide before the arrival is counted
                    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.act_ready + tk.unit) : "memory");
                }
                ++n_p1;
                continue;
            }
            // phase 2: one [128 d x tokens] accumulator per d-tile; store the real tokens' rows
            float* prow = a.partial + (size_t(un.jt) * a.rows_cap + un.row0) * D;
            for (int dt = tk.dt0; dt < tk.dt1 && ok; ++dt, ++nd) {
                const uint32_t b = nd & 1;
                ok = __all_sync(0xffffffffu, gg_wait(smem_u32(acc2_full + b), (nd >> 1) & 1, ab));
                if (!ok) break;
                tc_fence_after();
                for (int c = 0; c * 16 < un.ntok; ++c) {
                    float y[16];
                    tmem_ld16(tmem + lane_addr + 256 + 64 * b + c * 16, y);
#pragma unroll
                    for (int k2 = 0; k2 < 16; ++k2)
                        if (c * 16 + k2 < un.ntok) prow[size_t(c * 16 + k2) * D + dt * kGgTileRows + row] = y[k2];
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(acc2_empty + b));
            }
        }
    }

    // everyone meets here (also after an abort); the allocating warp returns the TMEM columns
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kGgTmemCols);
    if (a.clock && threadIdx.x == 0) atomicMax(a.clock + 1, global_timer_ns());
}

inline size_t ffn_grouped_smem() {
    return 1024 + size_t(kGgStages) * kGgStageBytes + kGgActBytes + 256 + 4 * kGgTokens * sizeof(float) + 64 +
           2 * kGgQueue * sizeof(uint64_t) + kGgQueue * sizeof(GgTask);
}

// Sorted token rows of one wave: Xs[row][:] = bf16(x[token][:]), wrow[row] = w[token][k].
struct GgRow { int32_t token, k; };

static __global__ void gg_gather_kernel(const float* __restrict__ x, const float* __restrict__ w, const GgRow* __restrict__ rows,
                                        int n_rows, const int* n_rows_dev, int D, int K, __nv_bfloat16* __restrict__ xs,
                                        float* __restrict__ wrow, int perm8, int* act_ready = nullptr, int n_ready = 0) {
    grid_dep_launch();
    grid_dep_wait();
    // the grouped kernel that follows counts arrivals per unit from zero
    if (blockIdx.x == 0) for (int i = threadIdx.x; i < n_ready; i += blockDim.x) act_ready[i] = 0;
    if (n_rows_dev) n_rows = __ldcg(n_rows_dev);
    const int r = blockIdx.x;
    if (r >= n_rows) return;
    const GgRow ri = rows[r];
    const float* src = x + size_t(ri.token) * D;
    __nv_bfloat16* dst = xs + size_t(r) * D;
    if (perm8) {
        // columns 8g .. 8g+7 are stored in the order 0 4 1 5 2 6 3 7: the order in which the 4-bit
        // kernel unpacks a word of eight weights, so that its operand needs no re-ordering
        for (int i = threadIdx.x * 8; i < D; i += blockDim.x * 8) {
            const float4 v0 = *reinterpret_cast<const float4*>(src + i), v1 = *reinterpret_cast<const float4*>(src + i + 4);
            const __nv_bfloat162 p0 = __floats2bfloat162_rn(v0.x, v1.x), p1 = __floats2bfloat162_rn(v0.y, v1.y);
            const __nv_bfloat162 p2 = __floats2bfloat162_rn(v0.z, v1.z), p3 = __floats2bfloat162_rn(v0.w, v1.w);
            uint4 o;
            o.x = *reinterpret_cast<const uint32_t*>(&p0);
            o.y = *reinterpret_cast<const uint32_t*>(&p1);
            o.z = *reinterpret_cast<const uint32_t*>(&p2);
            o.w = *reinterpret_cast<const uint32_t*>(&p3);
            *reinterpret_cast<uint4*>(dst + i) = o;
        }
    } else {
        for (int i = threadIdx.x * 4; i < D; i += blockDim.x * 4) {
            const float4 v = *reinterpret_cast<const float4*>(src + i);
            const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
            uint2 o;
            o.x = *reinterpret_cast<const uint32_t*>(&lo);
            o.y = *reinterpret_cast<const uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(dst + i) = o;
        }
    }
    if (threadIdx.x == 0) wrow[r] = w[size_t(ri.token) * K + ri.k];
}

// h[t][d] += sum over the token's experts of this wave (in k order) of the sum over j-tiles (ascending) of
// P[jt][rowmap[t][k]][d]; rowmap < 0 marks experts that belong to another wave.
// Block = (32 groups of four columns) x (K experts): thread (c, k) has all j-tiles of its expert in flight at
// once and adds them in j order; the K sums meet in shared memory and are added in k order, so the result does
// not depend on the launch geometry beyond this fixed tree.
constexpr int kCombineCols = 32;          // float4 column groups per block
constexpr int kCombineMaxJt = 16;         // j-tiles a thread keeps in flight (intermediate size <= 2048)
static __global__ void gg_combine_kernel(const float* __restrict__ partial, const int32_t* __restrict__ rowmap, int K, int n_jt,
                                         int rows_cap, int D, float* h) {
    __shared__ float4 part[SPM_MAX_TOPK][kCombineCols];
    grid_dep_launch();
    grid_dep_wait();
    const int t = blockIdx.y;
    const int c = threadIdx.x % kCombineCols, k = threadIdx.x / kCombineCols;
    const int d = (blockIdx.x * kCombineCols + c) * 4;
    const int r = (k < K && d < D) ? rowmap[t * SPM_MAX_TOPK + k] : -1;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r >= 0) {
        for (int j0 = 0; j0 < n_jt; j0 += kCombineMaxJt) {
            float4 v[kCombineMaxJt];
#pragma unroll
            for (int j = 0; j < kCombineMaxJt; ++j)
                v[j] = j0 + j < n_jt ? __ldcg(reinterpret_cast<const float4*>(partial + (size_t(j0 + j) * rows_cap + r) * D + d))
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < kCombineMaxJt; ++j)
                if (j0 + j < n_jt) { acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w; }
        }
    }
    if (k < K) part[k][c] = acc;
    __syncthreads();
    if (k == 0 && d < D) {
        float4 tot = *reinterpret_cast<const float4*>(h + size_t(t) * D + d);
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int kk = 0; kk < K; ++kk) {
            if (rowmap[t * SPM_MAX_TOPK + kk] < 0) continue;
            const float4 p = part[kk][c];
            sum.x += p.x; sum.y += p.y; sum.z += p.z; sum.w += p.w;
        }
        tot.x += sum.x; tot.y += sum.y; tot.z += sum.z; tot.w += sum.w;
        *reinterpret_cast<float4*>(h + size_t(t) * D + d) = tot;
    }
}
// launch geometry of gg_combine_kernel for hidden size D and top-K
inline dim3 gg_combine_grid(int D, int nb) { return dim3((D / 4 + kCombineCols - 1) / kCombineCols, nb); }
inline dim3 gg_combine_block(int K) { return dim3(kCombineCols * K); }

// Wave plan built on the device (all experts resident, one wave): the (token, k) pairs sorted by
// expert id, then token, then k — the order the host-side planner produces — the units of every
// routed expert, and the row of each pair for the combine step. One CTA, one thread per pair:
// a pair's row is (pairs of lower experts) + (same-expert pairs in lower warps) + (same-expert
// pairs in lower lanes of its warp), the last from a warp match, the others from small prefix sums.
constexpr int kGgPlanThreads = 1024;     // >= SPM_MAX_BATCH * SPM_MAX_TOPK pairs
static_assert(kGgPlanThreads >= SPM_MAX_BATCH * SPM_MAX_TOPK, "one thread per (token, k) pair");

inline size_t gg_plan_smem(int n) { return (size_t(kGgPlanThreads / 32) * n + 3 * size_t(n)) * sizeof(int32_t); }

static __global__ void __launch_bounds__(kGgPlanThreads)
gg_plan_kernel(const int32_t* __restrict__ ids, const short* __restrict__ slot_map, int slot_base, int nb, int K, int n,
               int n_jt, GgUnit* __restrict__ units, GgRow* __restrict__ rows, int32_t* __restrict__ rowmap,
               int* __restrict__ counts /* {n_units, n_rows} */, int* status) {
    extern __shared__ int32_t plan_sm[];
    constexpr int NW = kGgPlanThreads / 32;
    int32_t* tab = plan_sm;                    // [NW][n] same-expert pairs per warp -> exclusive prefix over warps
    int32_t* cnt = tab + NW * n;               // [n] pairs per expert
    int32_t* start = cnt + n;                  // [n] first row of the expert
    int32_t* rank = start + n;                 // [n] routed experts before e, -1 if not routed
    grid_dep_launch();
    const int tid = threadIdx.x, lane = tid & 31, wi = tid >> 5, total = nb * K;
    for (int i = tid; i < NW * n; i += kGgPlanThreads) tab[i] = 0;      // independent of the preceding kernel
    grid_dep_wait();
    const int e = tid < total ? __ldcg(ids + tid) : -1;
    for (int i = tid; i < nb * SPM_MAX_TOPK; i += kGgPlanThreads) rowmap[i] = -1;
    __syncthreads();
    const unsigned same = __match_any_sync(0xffffffffu, e);
    const int before = __popc(same & ((1u << lane) - 1u));
    if (e >= 0 && before == 0) tab[wi * n + e] = __popc(same);
    __syncthreads();
    for (int x = tid; x < n; x += kGgPlanThreads) {
        int run = 0;
        for (int w2 = 0; w2 < NW; ++w2) { const int c = tab[w2 * n + x]; tab[w2 * n + x] = run; run += c; }
        cnt[x] = run;
    }
    __syncthreads();
    if (wi == 0) {           // exclusive scans over the experts: rows and routed-expert ranks
        int row = 0, routed = 0;
        for (int x0 = 0; x0 < n; x0 += 32) {
            const int x = x0 + lane;
            const int c = x < n ? cnt[x] : 0, r = c > 0;
            int pc = c, pr = r;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int tc = __shfl_up_sync(0xffffffffu, pc, o), tr = __shfl_up_sync(0xffffffffu, pr, o);
                if (lane >= o) { pc += tc; pr += tr; }
            }
            if (x < n) { start[x] = row + pc - c; rank[x] = r ? routed + pr - r : -1; }
            row += __shfl_sync(0xffffffffu, pc, 31);
            routed += __shfl_sync(0xffffffffu, pr, 31);
        }
        if (lane == 0) { counts[0] = routed * n_jt; counts[1] = row; }
    }
    __syncthreads();
    if (e >= 0) {
        const int r = start[e] + tab[wi * n + e] + before;
        const int t = tid / K, k = tid - t * K;
        rows[r] = GgRow{t, k};
        rowmap[t * SPM_MAX_TOPK + k] = r;
    }
    for (int x = tid; x < n * n_jt; x += kGgPlanThreads) {
        const int ex = x / n_jt, jt = x - ex * n_jt;
        if (rank[ex] < 0) continue;
        const int slot = slot_map[ex];
        if (slot < 0 && jt == 0) atomicOr(status, kStatusBadSlot);
        units[rank[ex] * n_jt + jt] = GgUnit{slot_base + (slot < 0 ? 0 : slot), jt, start[ex], cnt[ex]};
    }
}

}  // namespace spm
