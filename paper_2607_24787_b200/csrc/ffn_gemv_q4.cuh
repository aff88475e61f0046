// Slot-indexed SwiGLU expert FFN for decode with 4-bit experts (the paper's on-device setting:
// 4-bit weights, 1.94 MB per DeepSeek-VL2-Tiny expert).
//
// Quantisation: groups of 32 weights along a row share one fp16 scale, value = scale * (q - 8),
// q in 0..15. A packed row of D weights is D/2 bytes of nibbles (element 2b in the low half of
// byte b, 2b+1 in the high half) followed by D/32 fp16 scales; a blob row j holds the packed
// gate[j][:], up[j][:] and column j of W_down back to back, so the kernel keeps the structure of
// ffn_gemv_kernel: per-warp rings of row triples filled by 1-D bulk async copies, the two dot
// products and the rank-1 update of y from one row, deterministic partial rows per CTA.
// A lane owns whole groups: 16 bytes of nibbles = 32 weights = one scale, so de-quantisation needs
// no cross-lane traffic: nibbles become exact (q - 8) halves with one lop3 + one half2 subtract
// per pair, are widened to fp32 and multiplied with fp32 activations; the scale is applied once
// per group. Transfers and HBM traffic shrink 3.56x against bf16.
#pragma once

#include <cuda_fp16.h>

#include "ffn_gemv.cuh"

namespace spm {

// 8 nibbles of one 32-bit word -> fp32 (q - 8), in element order 0..7
__device__ __forceinline__ void unpack_q4_word(uint32_t w, float (&f)[8]) {
    const __half2 bias = __floats2half2_rn(1032.f, 1032.f);      // 1024 + 8
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        // nibbles p and p + 4 sit at the same position of the two 16-bit halves
        uint32_t h = ((w >> (4 * p)) & 0x000f000fu) | 0x64006400u;          // half2 {1024 + q_p, 1024 + q_{p+4}}
        const __half2 v = __hsub2(*reinterpret_cast<__half2*>(&h), bias);   // exact q - 8
        const float2 t = __half22float2(v);
        f[p] = t.x;
        f[p + 4] = t.y;
    }
}

constexpr int kQ4MaxWarps = 16;    // activations live in shared memory here, so registers allow 16 warps
constexpr int kQ4Pad = 36;         // floats per 32-wide group in shared memory: lanes then start 4 banks apart

template <int NCH, int MAXNB>     // NCH = 16-byte nibble chunks (groups of 32 weights) per lane
__global__ void __launch_bounds__(kQ4MaxWarps * 32, 1)
ffn_gemv_q4_kernel(const __grid_constant__ FfnArgs<MAXNB> a, const int depth, const int D) {
    extern __shared__ __align__(128) unsigned char smem[];
    grid_dep_launch();
    const unsigned long long t_entry = (a.clock && threadIdx.x == 0) ? global_timer_ns() : 0ull;
    const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nw = blockDim.x >> 5;
    const int tok = blockIdx.y;
    const int G = gridDim.x, c = blockIdx.x;
    const int I = a.I;
    const int n_grp = D / 32;                         // groups per row
    const uint32_t RB = uint32_t(D / 2 + D / 16);     // bytes of one packed row
    const uint32_t ROWB = 3u * RB;
    const int R = a.entries(tok) * I;
    // even split: CTA c takes q rows, the first R % G CTAs one more (one 32-bit division)
    const int q_rows = R / G, rem_rows = R - q_rows * G;
    const int r_begin = q_rows * c + min(c, rem_rows);
    const int r_end = r_begin + q_rows + (c < rem_rows ? 1 : 0);
    const int span = r_end - r_begin - wi;
    const int my_n = span > 0 ? (span + nw - 1) / nw : 0;

    unsigned char* ring = smem + size_t(wi) * depth * ROWB;
    // layout: [ring, reused for the cross-warp reduction][barriers][activations, padded per group]
    const size_t ring_bytes = size_t(nw) * depth * ROWB, red_bytes = size_t(nw) * n_grp * kQ4Pad * sizeof(float);
    const size_t area = ((ring_bytes > red_bytes ? ring_bytes : red_bytes) + 15) & ~size_t(15);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + area);
    float* xs = reinterpret_cast<float*>(smem + area + ((size_t(nw) * depth * 8 + 15) & ~size_t(15)));
    const uint32_t bar0 = smem_u32(bars + wi * depth);
    const uint32_t ring0 = smem_u32(ring);
    if (lane == 0) {
        for (int d = 0; d < depth; ++d) mbar_init(bar0 + 8u * d, 1);
        fence_barrier_init();
    }
    __syncwarp();
    grid_dep_wait();          // routing results (slot codes, activations, weights) are read from here on
    // window start: kernel entry, or the end of the dependency wait when launched ahead of its predecessor's end
    if (a.clock && threadIdx.x == 0) atomicMin(a.clock, a.dev_code ? global_timer_ns() : t_entry);

    const uint64_t pol = policy_evict_first();
    bool ok = true;
    int src_ent = -1;                          // lane 0: entry being streamed and where its blob starts
    const unsigned char* src_base = nullptr;   //         (null: the entry cannot be served)
    auto resolve = [&](int ent) -> const unsigned char* {
        const int code = a.code_of(tok, ent);
        if (code < 0) {
            if (-1 - code >= a.n_shared) { atomicOr(a.status, kStatusBadSlot); return nullptr; }
            return a.shared + size_t(-1 - code) * a.blob_bytes;
        }
        if (code >= a.n_slots) { atomicOr(a.status, kStatusBadSlot); return nullptr; }
        // device-side wait for the batch of copies that fills this slot (see ffn_gemv_kernel)
        if (a.ready && !ffn_wait_arrival(a.ready + a.watch[ent], a.want[ent], a.limit())) {
            atomicOr(a.status, kStatusCopyTimeout);
            return nullptr;
        }
        return a.pool + size_t(code) * a.blob_bytes;
    };
    auto issue = [&](int i) {
        const int r = r_begin + wi + i * nw;
        const int ent = r / I;
        const int j = r - ent * I;
        if (ent != src_ent) { src_ent = ent; src_base = resolve(ent); }
        const unsigned char* base = src_base;
        if (!base) return false;
        const int st = i % depth;
        mbar_arrive_expect_tx(bar0 + 8u * st, ROWB);
        bulk_g2s(ring0 + uint32_t(st) * ROWB, base + size_t(j) * ROWB, ROWB, bar0 + 8u * st, pol);
        return true;
    };
    int n_issued = 0;
    if (lane == 0) {
        for (; n_issued < depth && n_issued < my_n; ++n_issued)
            if (!issue(n_issued)) { ok = false; break; }
    }

    // activations go to shared memory once (group g at xs[g * kQ4Pad ..]); the partial y of this
    // lane's groups (g = ch * 32 + lane) stays in registers
    for (int i = threadIdx.x; i < D; i += blockDim.x) xs[(i >> 5) * kQ4Pad + (i & 31)] = a.x[size_t(tok) * D + i];
    float ya[NCH][32];
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
        for (int v = 0; v < 32; ++v) ya[ch][v] = 0.f;
    __syncthreads();
    ok = __shfl_sync(0xffffffffu, ok, 0);

    int cur_ent = -1;
    float wk = 0.f;
    int done = 0;
    bool halt = false;
    if (ok) {
        for (int i = 0; i < my_n; ++i) {
            if (i >= __shfl_sync(0xffffffffu, n_issued, 0)) break;
            const int st = i % depth;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8u * st, (i / depth) & 1, a.limit()))) {
                if (lane == 0) atomicOr(a.status, kStatusCopyTimeout);
                ok = false;
                break;
            }
            done = i + 1;
            const int r = r_begin + wi + i * nw;
            const int ent = r / I;
            if (ent != cur_ent) {
                cur_ent = ent;
                const int kk = a.kidx_of(tok, ent);
                wk = kk == 255 ? 1.f : a.w[size_t(tok) * a.K + kk];
            }
            const unsigned char* buf = ring + size_t(st) * ROWB;
            float pg = 0.f, pu = 0.f;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                const int g = ch * 32 + lane;
                if (g < n_grp) {
                    const uint4 vg = *reinterpret_cast<const uint4*>(buf + g * 16);
                    const uint4 vu = *reinterpret_cast<const uint4*>(buf + RB + g * 16);
                    const float sg = __half2float(*reinterpret_cast<const __half*>(buf + D / 2 + g * 2));
                    const float su = __half2float(*reinterpret_cast<const __half*>(buf + RB + D / 2 + g * 2));
                    const uint32_t wg[4] = {vg.x, vg.y, vg.z, vg.w}, wu[4] = {vu.x, vu.y, vu.z, vu.w};
                    const float* xg = xs + g * kQ4Pad;
                    float dg = 0.f, du = 0.f;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float fg[8], fu[8];
                        unpack_q4_word(wg[q], fg);
                        unpack_q4_word(wu[q], fu);
                        const float4 x0 = *reinterpret_cast<const float4*>(xg + q * 8);
                        const float4 x1 = *reinterpret_cast<const float4*>(xg + q * 8 + 4);
                        const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            dg = fmaf(fg[v], xv[v], dg);
                            du = fmaf(fu[v], xv[v], du);
                        }
                    }
                    pg = fmaf(sg, dg, pg);
                    pu = fmaf(su, du, pu);
                }
            }
            pg = warp_sum(pg);
            pu = warp_sum(pu);
            const float act = pg / (1.f + expf(-pg)) * pu * wk;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                const int g = ch * 32 + lane;
                if (g < n_grp) {
                    const uint4 vd = *reinterpret_cast<const uint4*>(buf + 2 * RB + g * 16);
                    const float sd = act * __half2float(*reinterpret_cast<const __half*>(buf + 2 * RB + D / 2 + g * 2));
                    const uint32_t wd[4] = {vd.x, vd.y, vd.z, vd.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float fd[8];
                        unpack_q4_word(wd[q], fd);
#pragma unroll
                        for (int v = 0; v < 8; ++v) ya[ch][q * 8 + v] = fmaf(sd, fd[v], ya[ch][q * 8 + v]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0 && n_issued < my_n && !halt) {
                if (issue(n_issued)) ++n_issued;
                else halt = true;
            }
        }
    }
    if (!ok) {
        n_issued = __shfl_sync(0xffffffffu, n_issued, 0);
        for (int i = done; i < n_issued; ++i)
            if (!mbar_wait_bounded(bar0 + 8u * (i % depth), (i / depth) & 1, a.limit())) break;
    }

    // sum the warps' partial y in warp order, one partial row per CTA
    __syncthreads();
    float* red = reinterpret_cast<float*>(smem);
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
        const int g = ch * 32 + lane;
        if (g < n_grp) {
#pragma unroll
            for (int v = 0; v < 32; v += 4)
                *reinterpret_cast<float4*>(red + (size_t(wi) * n_grp + g) * kQ4Pad + v) = make_float4(ya[ch][v], ya[ch][v + 1], ya[ch][v + 2], ya[ch][v + 3]);
        }
    }
    __syncthreads();
    float* out = a.partial + (size_t(tok) * G + c) * D;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        const int o = (d >> 5) * kQ4Pad + (d & 31);
        float acc = red[o];
        for (int w2 = 1; w2 < nw; ++w2) acc += red[size_t(w2) * n_grp * kQ4Pad + o];
        out[d] = acc;
    }
    if (a.clock) {
        __syncthreads();
        if (threadIdx.x == 0) atomicMax(a.clock + 1, global_timer_ns());
    }
}

// Launch shape for 4-bit rows: the warp count that leaves the fewest rows on the busiest warp, a
// ring deep enough to hold a warp's whole share when it fits, and room for the cross-warp reduction.
inline void ffn_gemv_q4_shape(size_t row_bytes, int D, int rows_per_cta, int* warps, int* depth, size_t* smem) {
    int best_w = 8, best_cost = 1 << 30;
    for (int w = 4; w <= kQ4MaxWarps; ++w) {
        const int cost = (rows_per_cta + w - 1) / w;
        if (cost < best_cost || (cost == best_cost && w < best_w)) { best_w = w; best_cost = cost; }
    }
    int d = best_cost < 2 ? 2 : (best_cost > 6 ? 6 : best_cost);
    while (d > 2 && size_t(best_w) * d * row_bytes > 150 * 1024) --d;
    size_t area = size_t(best_w) * d * row_bytes;
    const size_t red = size_t(best_w) * (D / 32) * kQ4Pad * sizeof(float);
    if (area < red) area = red;
    *warps = best_w;
    *depth = d;
    *smem = ((area + 15) & ~size_t(15)) + ((size_t(best_w) * d * 8 + 15) & ~size_t(15)) + size_t(D / 32) * kQ4Pad * sizeof(float) + 16;
}

}  // namespace spm
