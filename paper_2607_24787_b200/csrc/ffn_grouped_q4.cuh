// Batched decode with 4-bit experts: the grouped SwiGLU expert FFN of ffn_grouped.cuh fed from
// packed 4-bit blobs (groups of 32 weights + one fp16 scale, see ffn_gemv_q4.cuh).
//
// The tensor cores take bf16 operands, so a fourth role is added between the TMA producer and the
// MMA issuer: eight de-quantisation warps in two groups of four (one warp per TMEM lane quarter);
// a group expands every second item, so two items are in flight and one group's waits overlap the
// other's arithmetic. The conversion stays in packed bf16 arithmetic: a nibble q is OR-ed into the
// mantissa of 128.0 (exact 128 + q), 136 is subtracted (exact q - 8) and the result is multiplied
// by the group's scale rounded to bf16: weight = bf16_rn(bf16_rn(scale) * (q - 8)), two
// instructions per pair of weights.
//   First GEMM (gate and up tiles, K-major): the expanded weights never touch shared memory. Row
// r of a 128-row tile is TMEM lane r; a thread writes its row's 64 weights of both tiles as 2 x 32
// columns with tcgen05.st, and tcgen05.mma takes the A operand from tensor memory (two stages of
// 64 columns behind the accumulators). Second GEMM (W_down's column tile, consumed M-major: the
// rows of the packed tile run along the contraction): the tile is written to a shared-memory
// stage with the 128-byte swizzle a TMA load of bf16 data would have produced.
//
// Rings. Packed stages (TMA -> de-quantisation) hold 64 bytes of nibbles per row, i.e. two
// K-blocks of gate and up rows (phase 1) or one d-tile of the W_down column tile (phase 2), and
// every second one also the 16 bytes of scales per row that cover it and its successor; a group
// copies the nibbles of its item to registers and hands the stage back at once, so the producer
// (warp 0) runs ahead as far as the ring allows. Token-row stages (TMA -> MMA) hold the bf16
// token rows of one K-block and have their own producer (warp 14), so that a wait for a token
// stage never holds back the weight stream. Every wait is bounded and shares the abort flag of
// the CTA; no multicast.
#pragma once

#include "ffn_gemv_q4.cuh"
#include "ffn_grouped.cuh"

namespace spm {

constexpr int kQgThreads = 480;          // warp 0 TMA (packed weights), 1 MMA + TMEM, 2-5 epilogue, 6-13 de-quantisation, 14 TMA (token rows)
constexpr int kQgDequantWarps = 8;
constexpr int kQgGroups = 2;             // de-quantisation groups of four warps (one per TMEM lane quarter); group g expands every second item
constexpr int kQgGroupWarps = kQgDequantWarps / kQgGroups;
constexpr int kQgOperandStages = 2;      // shared-memory operand stages of the second GEMM, 2 x 16 KB bf16 tiles each
constexpr int kQgTmemStages = 2;         // tensor-memory operand stages of the first GEMM, 2 x 32 columns each
constexpr uint32_t kQgTmemA = 384;       // first column of those stages (the accumulators end at 383)
constexpr int kQgPackedStages = 6;
constexpr int kQgTokenStages = 2;        // 8 KB each
constexpr uint32_t kQgOperandBytes = 2 * kGgTileBytes;
constexpr uint32_t kQgHalfBytes = 8192;  // [128 rows][64 B] of nibbles
constexpr uint32_t kQgNibBytes = 2 * kQgHalfBytes;   // phase 1: gate + up; phase 2: one such tile
constexpr uint32_t kQgScaleBytes = 2048; // [128 rows][16 B] = 8 fp16 scales per row
constexpr uint32_t kQgPackedBytes = kQgNibBytes + 2 * kQgScaleBytes;

// 8 nibbles of one word -> 8 bf16 (scale * (q - 8)) as one 16-byte chunk. Nibbles p and p + 4 sit at
// the same position of the two 16-bit halves, so four packed operations give the pairs (e0,e4)
// (e1,e5) (e2,e6) (e3,e7), and the chunk is stored in that order: element positions 0..7 of a group of
// eight hold weights 0 4 1 5 2 6 3 7. Where the group runs along the contraction (first GEMM) the
// token rows are gathered in the same order; where it runs along the output rows (second GEMM) the
// epilogue maps the accumulator row back (qg_unpermute).
__device__ __forceinline__ uint4 dequant_chunk(uint32_t w, __nv_bfloat162 scale2) {
    const uint32_t off_bits = 0x43084308u;                       // bf16x2 {136, 136}
    const __nv_bfloat162 off = *reinterpret_cast<const __nv_bfloat162*>(&off_bits);
    uint32_t r[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const uint32_t bits = ((w >> (4 * p)) & 0x000f000fu) | 0x43004300u;     // bf16x2 {128 + q_p, 128 + q_{p+4}}
        const __nv_bfloat162 v = __hmul2(__hsub2(*reinterpret_cast<const __nv_bfloat162*>(&bits), off), scale2);
        r[p] = *reinterpret_cast<const uint32_t*>(&v);
    }
    return make_uint4(r[0], r[1], r[2], r[3]);
}

// 32 consecutive 32-bit columns of this thread's TMEM lane (the mirror of tmem_ld16)
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
          "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
          "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem desc]: the A operand (128 rows = lanes, 16 bf16 = 8 columns) comes from tensor memory
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t"
        "}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ int qg_unpermute(int m) { return (m & ~7) | ((m & 7) >> 1) | ((m & 1) << 2); }

__device__ __forceinline__ __nv_bfloat162 scale_at(const uint4& v, int i) {      // i-th fp16 of a 16-byte vector, as bf16x2
    const uint32_t w = i < 2 ? v.x : i < 4 ? v.y : i < 6 ? v.z : v.w;
    return __float2bfloat162_rn(__half2float(__ushort_as_half((unsigned short)((i & 1) ? (w >> 16) : (w & 0xffffu)))));
}

// The super-items (one packed stage each) of a CTA in work order: phase1(0), then for i = 0, 1, ...:
// phase1(i + 1) if it exists, phase2(i). A phase-1 super-item is two K-blocks, a phase-2 one a d-tile.
struct QgSeq {
    int my_units, p1, p2;          // units of this CTA, super-items per phase
    int u1 = 0, i = 0, idx = 0;    // unit whose phase 1 / phase 2 is being walked, position inside the phase
    bool phase1 = true, done = false;
    __device__ QgSeq(int units, int n1, int n2) : my_units(units), p1(n1), p2(n2) { done = units == 0; }
    __device__ int unit() const { return phase1 ? u1 : i; }
    __device__ void next() {
        if (++idx < (phase1 ? p1 : p2)) return;
        idx = 0;
        if (phase1) {
            if (u1 == 0 && my_units > 1) { u1 = 1; return; }     // after phase1(0): phase1(1), then phase2(0)
            phase1 = false;                                       // after phase1(i + 1): phase2(i)
        } else {
            if (++i >= my_units) { done = true; return; }
            if (i + 1 < my_units) { u1 = i + 1; phase1 = true; }
        }
    }
};

__global__ void __launch_bounds__(kQgThreads, 1)
ffn_grouped_q4_kernel(const __grid_constant__ CUtensorMap nib64, const __grid_constant__ CUtensorMap sc16,
                      const __grid_constant__ GgTokenMaps xmaps, const GgArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* mst = smem;                                               // operand stages
    unsigned char* act = mst + kQgOperandStages * kQgOperandBytes;           // A^T, 16 KB
    unsigned char* xst = act + kGgActBytes;                                  // token-row stages
    unsigned char* qst = xst + kQgTokenStages * kGgXBytes;                   // packed stages
    uint64_t* bars = reinterpret_cast<uint64_t*>(qst + kQgPackedStages * kQgPackedBytes);
    uint64_t* qfull = bars;                          // [packed]   TMA -> de-quantisation
    uint64_t* qempty = qfull + kQgPackedStages;      // [packed]   de-quantisation -> TMA
    uint64_t* xfull = qempty + kQgPackedStages;      // [token]    TMA -> MMA
    uint64_t* xempty = xfull + kQgTokenStages;       // [token]    MMA -> TMA
    uint64_t* mfull = xempty + kQgTokenStages;       // [operand]  de-quantisation -> MMA
    uint64_t* mempty = mfull + kQgOperandStages;     // [operand]  MMA -> de-quantisation
    uint64_t* tfull = mempty + kQgOperandStages;     // [tmem]     de-quantisation -> MMA (first GEMM)
    uint64_t* tempty = tfull + kQgTmemStages;        // [tmem]     MMA -> de-quantisation
    uint64_t* acc1_full = tempty + kQgTmemStages;    // [2]
    uint64_t* acc1_empty = acc1_full + 2;            // [2]
    uint64_t* act_full = acc1_empty + 2;
    uint64_t* act_empty = act_full + 1;
    uint64_t* acc2_full = act_empty + 1;             // [2]
    uint64_t* acc2_empty = acc2_full + 2;            // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc2_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* wrow_all = reinterpret_cast<float*>(tmem_slot + 4);               // [4 epilogue warps][64]

    grid_dep_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = a.D;
    const int n_kb = D / kGgKBlock;
    const int n_dt = D / kGgTileRows;
    GgAbort ab{abort_flag, a.status, a.wait_limit_ns ? a.wait_limit_ns : kWaitLimitNs};

    if (threadIdx.x == 0) {
        for (int s = 0; s < kQgPackedStages; ++s) { mbar_init(smem_u32(qfull + s), 1); mbar_init(smem_u32(qempty + s), kQgDequantWarps); }
        for (int s = 0; s < kQgTokenStages; ++s) { mbar_init(smem_u32(xfull + s), 1); mbar_init(smem_u32(xempty + s), 1); }
        for (int s = 0; s < kQgOperandStages; ++s) { mbar_init(smem_u32(mfull + s), kQgGroupWarps); mbar_init(smem_u32(mempty + s), 1); }
        for (int s = 0; s < kQgTmemStages; ++s) { mbar_init(smem_u32(tfull + s), kQgGroupWarps); mbar_init(smem_u32(tempty + s), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(acc1_full + b), 1);
            mbar_init(smem_u32(acc1_empty + b), 4);
            mbar_init(smem_u32(acc2_full + b), 1);
            mbar_init(smem_u32(acc2_empty + b), 4);
        }
        mbar_init(smem_u32(act_full), 4);
        mbar_init(smem_u32(act_empty), 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kGgTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_dep_wait();
    if (a.clock && threadIdx.x == 0) atomicMin(a.clock, global_timer_ns());
    const int n_units = a.n_units_dev ? __ldcg(a.n_units_dev) : a.n_units;
    const int my_units = int(blockIdx.x) < n_units ? (n_units - 1 - int(blockIdx.x)) / int(gridDim.x) + 1 : 0;
    const int sc_x0 = D / 2;                         // byte offset of the scales inside a packed row
    const int p1_supers = n_kb / 2, p2_supers = n_dt;

    if (warp == 0) {
        // ---------------- TMA producer of the packed weights: runs ahead as far as the packed ring allows ----------------
        // The whole warp walks the loop in uniform control flow and one elected lane issues.
        {
            uint32_t np = 0;              // packed stages issued so far
            bool ok = true;
            auto load_packed = [&](const QgSeq& q) {
                const int32_t u = int32_t(blockIdx.x + q.unit() * gridDim.x);
                const GgUnit un = a.units[u];
                if (a.unit_wait && q.phase1 && q.idx == 0) {     // first item of a unit: its expert's copy may still be on its way
                    const GgWait uw = a.unit_wait[u];
                    if (uw.watch >= 0) ok = __all_sync(0xffffffffu, gg_wait_arrival(a.ready + uw.watch, uw.want, ab));
                    if (!ok) return;
                }
                const uint32_t ps = np % kQgPackedStages;
                if (np >= uint32_t(kQgPackedStages))
                    ok = __all_sync(0xffffffffu, gg_wait(smem_u32(qempty + ps), ((np / kQgPackedStages) - 1) & 1, ab));
                if (!ok) return;
                const uint32_t qb = smem_u32(qst + ps * kQgPackedBytes), fq = smem_u32(qfull + ps);
                const int r0 = un.jt * kGgTileRows;
                const bool with_scales = (q.idx & 1) == 0;        // 16 bytes of scales cover two super-items
                if (elect_one()) {
                    if (q.phase1) {
                        mbar_arrive_expect_tx(fq, 2 * kQgHalfBytes + (with_scales ? 2 * kQgScaleBytes : 0));
                        tma_load_4d(qb, &nib64, q.idx * 64, 0, r0, un.slot, fq);
                        tma_load_4d(qb + kQgHalfBytes, &nib64, q.idx * 64, 1, r0, un.slot, fq);
                        if (with_scales) {
                            tma_load_4d(qb + kQgNibBytes, &sc16, sc_x0 + (q.idx >> 1) * 16, 0, r0, un.slot, fq);
                            tma_load_4d(qb + kQgNibBytes + kQgScaleBytes, &sc16, sc_x0 + (q.idx >> 1) * 16, 1, r0, un.slot, fq);
                        }
                    } else {
                        mbar_arrive_expect_tx(fq, kQgHalfBytes + (with_scales ? kQgScaleBytes : 0));
                        tma_load_4d(qb, &nib64, q.idx * 64, 2, r0, un.slot, fq);
                        if (with_scales) tma_load_4d(qb + kQgNibBytes, &sc16, sc_x0 + (q.idx >> 1) * 16, 2, r0, un.slot, fq);
                    }
                }
                __syncwarp();
                ++np;
            };
            for (QgSeq q(my_units, p1_supers, p2_supers); !q.done && ok; q.next()) load_packed(q);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (as in the bf16 kernel; operands and token rows on separate rings) ----------------
        // The whole warp walks the loop in uniform control flow and one elected lane issues.
        {
            uint32_t t1 = 0, t2 = 0, nx = 0, nd = 0;     // items of the first / second GEMM, token-row stages, d-tiles consumed so far
            bool ok = true;
            auto wait_all = [&](uint64_t* bar, uint32_t parity) { ok = __all_sync(0xffffffffu, ok && gg_wait(smem_u32(bar), parity, ab)); };
            auto mma_phase1 = [&](int i) {
                const uint32_t b = i & 1, m = uint32_t(i) >> 1;
                const uint32_t idesc1 = gg_idesc_n(false, false, gg_pad_tokens(a.units[blockIdx.x + i * gridDim.x].ntok));
                if (i >= 2) wait_all(acc1_empty + b, (m - 1) & 1);
                const uint32_t acc = tmem + 128 * b;
                for (int kb = 0; kb < n_kb && ok; ++kb, ++t1, ++nx) {
                    const uint32_t s = t1 % kQgTmemStages, xs = nx % kQgTokenStages;
                    wait_all(tfull + s, (t1 / kQgTmemStages) & 1);
                    wait_all(xfull + xs, (nx / kQgTokenStages) & 1);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t at = tmem + kQgTmemA + 64 * s, xb = smem_u32(xst + xs * kGgXBytes);
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t bx = smem_desc_sw128(xb + ks * 32, 16, 1024);
                            tc_mma_bf16_ts(acc, at + ks * 8, bx, idesc1, (kb | ks) != 0);
                            tc_mma_bf16_ts(acc + 64, at + 32 + ks * 8, bx, idesc1, (kb | ks) != 0);
                        }
                        tc_commit(smem_u32(tempty + s));
                        tc_commit(smem_u32(xempty + xs));
                    }
                    __syncwarp();
                }
                if (ok && elect_one()) tc_commit(smem_u32(acc1_full + b));
                __syncwarp();
            };
            auto mma_phase2 = [&](int i) {
                const uint32_t idesc2 = gg_idesc_n(true, true, gg_pad_tokens(a.units[blockIdx.x + i * gridDim.x].ntok));
                wait_all(act_full, i & 1);
                if (!ok) return;
                tc_fence_after();
                const uint32_t act_addr = smem_u32(act);
                for (int dt = 0; dt < n_dt && ok; ++dt, ++t2, ++nd) {
                    const uint32_t s = t2 % kQgOperandStages, b = nd & 1;
                    wait_all(mfull + s, (t2 / kQgOperandStages) & 1);
                    if (nd >= 2) wait_all(acc2_empty + b, ((nd >> 1) - 1) & 1);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t base = smem_u32(mst + s * kQgOperandBytes);
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint64_t da = smem_desc_sw128(base + ks * 2048, kGgTileBytes, 1024);
                            const uint64_t db = smem_desc_sw128(act_addr + ks * 2048, kGgActBytes, 1024);
                            tc_mma_bf16(tmem + 256 + 64 * b, da, db, idesc2, ks != 0);
                        }
                        tc_commit(smem_u32(mempty + s));
                        tc_commit(smem_u32(acc2_full + b));
                    }
                    __syncwarp();
                }
                if (ok && elect_one()) tc_commit(smem_u32(act_empty));
                __syncwarp();
            };
            if (my_units > 0) mma_phase1(0);
            for (int i = 0; i < my_units && ok; ++i) {
                if (i + 1 < my_units) mma_phase1(i + 1);
                if (ok) mma_phase2(i);
            }
        }
    } else if (warp == 14) {
        // ---------------- TMA producer of the token rows: the two K-blocks of every phase-1 super-item ----------------
        // (its own warp, so that a wait for a token-row stage never holds back the weight stream)
        uint32_t nx = 0;
        bool ok = true;
        for (QgSeq q(my_units, p1_supers, p2_supers); !q.done && ok; q.next()) {
            if (!q.phase1) continue;
            const GgUnit un = a.units[blockIdx.x + q.unit() * gridDim.x];
            const int xbox = gg_token_box(un.ntok);
            for (int j = 0; j < 2 && ok; ++j, ++nx) {
                const uint32_t xs = nx % kQgTokenStages;
                if (nx >= uint32_t(kQgTokenStages))
                    ok = __all_sync(0xffffffffu, gg_wait(smem_u32(xempty + xs), ((nx / kQgTokenStages) - 1) & 1, ab));
                if (!ok) break;
                const uint32_t fx = smem_u32(xfull + xs);
                if (elect_one()) {
                    mbar_arrive_expect_tx(fx, gg_token_rows(xbox) * 128);
                    tma_load_2d(smem_u32(xst + xs * kGgXBytes), &xmaps.m[xbox], (q.idx * 2 + j) * kGgKBlock, un.row0, fx);
                }
                __syncwarp();
            }
        }
    } else if (warp >= 6) {
        // ---------------- de-quantisation warps: two groups of four warps, each expanding every second item ----------------
        // First GEMM: the expanded weights go straight to tensor memory (tcgen05.st) and the MMA
        // takes its A operand from there: row r of the tile is TMEM lane r, so the four warps of a
        // group are those whose warp number mod 4 covers the four lane quarters, and a thread
        // expands its row of both tiles (gate, up): 2 x 64 weights = 2 x 32 columns. Second GEMM:
        // W_down's tile is consumed M-major (rows of the packed tile run along the contraction),
        // so it goes to a swizzled shared-memory stage as a TMA load of bf16 data would have put it.
        const int dq = warp - 6;
        const int grp = dq / kQgGroupWarps;
        const int r = (warp & 3) * 32 + lane;                // row of the 128-row tile = TMEM lane
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        const uint32_t sw = uint32_t(r & 7);                 // 128-byte swizzle of the bf16 operand rows
        const uint32_t sq = uint32_t((r >> 1) & 3);          // 64-byte swizzle of the packed rows
        uint32_t t1 = 0, t2 = 0, np = 0;                     // items seen of the first / second GEMM, packed stages consumed
        bool ok = true;
        uint4 sc[2];                                         // [tile]: 8 scales of row r for the current pair of super-items
        sc[0] = sc[1] = make_uint4(0, 0, 0, 0);
        for (QgSeq q(my_units, p1_supers, p2_supers); !q.done && ok; q.next(), ++np) {
            const uint32_t ps = np % kQgPackedStages;
            ok = __all_sync(0xffffffffu, gg_wait(smem_u32(qfull + ps), (np / kQgPackedStages) & 1, ab));
            if (!ok) break;
            const unsigned char* qb = qst + ps * kQgPackedBytes;
            if ((q.idx & 1) == 0) {
                sc[0] = *reinterpret_cast<const uint4*>(qb + kQgNibBytes + r * 16);
                if (q.phase1) sc[1] = *reinterpret_cast<const uint4*>(qb + kQgNibBytes + kQgScaleBytes + r * 16);
            }
            // A packed chunk (16 bytes, 32 weights) has one scale: number 4 * (idx & 1) + chunk of the row's vector.
            const int g0 = 4 * (q.idx & 1);
            if (q.phase1) {
                // two items (K-blocks 2*idx and 2*idx + 1), one per group; t1 is even here, so item j has stage j
                const int j = grp;
                const uint32_t tm = t1 + uint32_t(j);
                t1 += 2;
                uint4 nib[2][2];                              // [tile][chunk]: packed chunks 2j, 2j+1 of the row
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {
                    const unsigned char* nrow = qb + tile * kQgHalfBytes + r * 64;
                    nib[tile][0] = *reinterpret_cast<const uint4*>(nrow + ((uint32_t(2 * j) ^ sq) << 4));
                    nib[tile][1] = *reinterpret_cast<const uint4*>(nrow + ((uint32_t(2 * j + 1) ^ sq) << 4));
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(qempty + ps));       // nibbles are in registers: hand the stage back
                const uint32_t s = tm % kQgTmemStages;
                if (tm >= uint32_t(kQgTmemStages))
                    ok = __all_sync(0xffffffffu, gg_wait(smem_u32(tempty + s), ((tm / kQgTmemStages) - 1) & 1, ab));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {
                    const __nv_bfloat162 s0 = scale_at(sc[tile], g0 + 2 * j), s1 = scale_at(sc[tile], g0 + 2 * j + 1);
                    const uint4 n0 = nib[tile][0], n1 = nib[tile][1];
                    const uint32_t w0[4] = {n0.x, n0.y, n0.z, n0.w}, w1[4] = {n1.x, n1.y, n1.z, n1.w};
                    uint32_t cols[32];                        // 64 weights of the row, two per column
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint4 v0 = dequant_chunk(w0[c], s0), v1 = dequant_chunk(w1[c], s1);
                        cols[4 * c] = v0.x; cols[4 * c + 1] = v0.y; cols[4 * c + 2] = v0.z; cols[4 * c + 3] = v0.w;
                        cols[16 + 4 * c] = v1.x; cols[16 + 4 * c + 1] = v1.y; cols[16 + 4 * c + 2] = v1.z; cols[16 + 4 * c + 3] = v1.w;
                    }
                    tmem_st32(tmem + lane_addr + kQgTmemA + 64 * s + 32 * tile, cols);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(tfull + s));
            } else {
                // one item (a d-tile of the W_down column tile), groups alternate
                const uint32_t tm = t2;
                t2 += 1;
                const bool mine = int(tm % kQgGroups) == grp;
                uint4 nib[4];                                 // the row's four packed chunks = 128 d-values
                if (mine) {
                    const unsigned char* nrow = qb + r * 64;
#pragma unroll
                    for (int c = 0; c < 4; ++c) nib[c] = *reinterpret_cast<const uint4*>(nrow + ((uint32_t(c) ^ sq) << 4));
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(qempty + ps));
                if (!mine) continue;
                const uint32_t ms = tm % kQgOperandStages;
                if (tm >= uint32_t(kQgOperandStages))
                    ok = __all_sync(0xffffffffu, gg_wait(smem_u32(mempty + ms), ((tm / kQgOperandStages) - 1) & 1, ab));
                if (!ok) break;
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {        // d 0..63 and d 64..127 of the d-tile
                    const __nv_bfloat162 s0 = scale_at(sc[0], g0 + 2 * tile), s1 = scale_at(sc[0], g0 + 2 * tile + 1);
                    unsigned char* row = mst + ms * kQgOperandBytes + tile * kGgTileBytes + r * 128;
                    const uint4 n0 = nib[2 * tile], n1 = nib[2 * tile + 1];
                    const uint32_t w0[4] = {n0.x, n0.y, n0.z, n0.w}, w1[4] = {n1.x, n1.y, n1.z, n1.w};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        *reinterpret_cast<uint4*>(row + ((uint32_t(c) ^ sw) << 4)) = dequant_chunk(w0[c], s0);
                        *reinterpret_cast<uint4*>(row + ((uint32_t(c + 4) ^ sw) << 4)) = dequant_chunk(w1[c], s1);
                    }
                }
                fence_proxy_async();          // generic-proxy writes -> visible to the MMA's async reads
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(mfull + ms));
            }
        }
    } else {
        // ---------------- epilogue warps (as in the bf16 kernel) ----------------
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t lane_addr = uint32_t(q * 32) << 16;
        float* wrow_s = wrow_all + q * kGgTokens;
        uint32_t nd = 0;
        bool ok = true;
        for (int i = 0; i < my_units && ok; ++i) {
            const GgUnit un = a.units[blockIdx.x + i * gridDim.x];
            const uint32_t b1 = i & 1;
            __syncwarp();
#pragma unroll
            for (int tk = lane; tk < kGgTokens; tk += 32) wrow_s[tk] = tk < un.ntok ? a.wrow[un.row0 + tk] : 0.f;
            __syncwarp();
            ok = gg_wait(smem_u32(acc1_full + b1), (uint32_t(i) >> 1) & 1, ab);
            if (ok && i > 0) ok = gg_wait(smem_u32(act_empty), (i - 1) & 1, ab);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int n_pad = int(gg_pad_tokens(un.ntok));      // columns the MMAs of this unit wrote
#pragma unroll
            for (int c = 0; c < kGgTokens / 16; ++c) {
                if (c * 16 >= n_pad) break;
                float g[16], up[16];
                tmem_ld16(tmem + lane_addr + 128 * b1 + c * 16, g);
                tmem_ld16(tmem + lane_addr + 128 * b1 + 64 + c * 16, up);
                uint32_t packed[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float a0 = g[2 * e] / (1.f + expf(-g[2 * e])) * up[2 * e] * wrow_s[c * 16 + 2 * e];
                    const float a1 = g[2 * e + 1] / (1.f + expf(-g[2 * e + 1])) * up[2 * e + 1] * wrow_s[c * 16 + 2 * e + 1];
                    const __nv_bfloat162 p = __floats2bfloat162_rn(a0, a1);
                    packed[e] = *reinterpret_cast<const uint32_t*>(&p);
                }
                unsigned char* rowp = act + row * 128;
                *reinterpret_cast<uint4*>(rowp + (((2 * c) ^ (row & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                *reinterpret_cast<uint4*>(rowp + (((2 * c + 1) ^ (row & 7)) << 4)) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
            }
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(smem_u32(acc1_empty + b1)); mbar_arrive(smem_u32(act_full)); }

            float* prow = a.partial + (size_t(un.jt) * a.rows_cap + un.row0) * D;
            for (int dt = 0; dt < n_dt && ok; ++dt, ++nd) {
                const uint32_t b = nd & 1;
                ok = __all_sync(0xffffffffu, gg_wait(smem_u32(acc2_full + b), (nd >> 1) & 1, ab));
                if (!ok) break;
                tc_fence_after();
                const int d = dt * kGgTileRows + qg_unpermute(row);       // accumulator row -> output column
                for (int c = 0; c * 16 < un.ntok; ++c) {
                    float y[16];
                    tmem_ld16(tmem + lane_addr + 256 + 64 * b + c * 16, y);
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        if (c * 16 + e < un.ntok) prow[size_t(c * 16 + e) * D + d] = y[e];
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(acc2_empty + b));
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kGgTmemCols);
    if (a.clock && threadIdx.x == 0) atomicMax(a.clock + 1, global_timer_ns());
}

inline size_t ffn_grouped_q4_smem() {
    return 1024 + size_t(kQgOperandStages) * kQgOperandBytes + kGgActBytes + size_t(kQgTokenStages) * kGgXBytes +
           size_t(kQgPackedStages) * kQgPackedBytes + 512 + 4 * kGgTokens * sizeof(float) + 64;
}
static_assert(1024 + kQgOperandStages * kQgOperandBytes + kGgActBytes + kQgTokenStages * kGgXBytes +
              kQgPackedStages * kQgPackedBytes + 512 + 4 * kGgTokens * 4 + 64 <= 232448, "shared memory of the 4-bit grouped kernel");

}  // namespace spm
