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

template <int NCH, int MAXNB>     // NCH = 16-byte nibble chunks (groups of 32 weights) per lane
__global__ void __launch_bounds__(kFfnMaxThreads, 1)
ffn_gemv_q4_kernel(const __grid_constant__ FfnArgs<MAXNB> a, const int depth, const int D) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nw = blockDim.x >> 5;
    if (a.clock && threadIdx.x == 0) atomicMin(a.clock, global_timer_ns());
    const int tok = blockIdx.y;
    const int G = gridDim.x, c = blockIdx.x;
    const int I = a.I;
    const int n_grp = D / 32;                         // groups per row
    const uint32_t RB = uint32_t(D / 2 + D / 16);     // bytes of one packed row
    const uint32_t ROWB = 3u * RB;
    const int R = int(a.count[tok]) * I;
    const int r_begin = int((long long)R * c / G);
    const int r_end = int((long long)R * (c + 1) / G);
    const int span = r_end - r_begin - wi;
    const int my_n = span > 0 ? (span + nw - 1) / nw : 0;

    unsigned char* ring = smem + size_t(wi) * depth * ROWB;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ((size_t(nw) * depth * ROWB + 15) & ~size_t(15)));
    const uint32_t bar0 = smem_u32(bars + wi * depth);
    const uint32_t ring0 = smem_u32(ring);
    if (lane == 0) {
        for (int d = 0; d < depth; ++d) mbar_init(bar0 + 8u * d, 1);
        fence_barrier_init();
    }
    __syncwarp();

    const uint64_t pol = policy_evict_first();
    bool ok = true;
    auto issue = [&](int i) {
        const int r = r_begin + wi + i * nw;
        const int ent = r / I;
        const int j = r - ent * I;
        const int code = a.code[tok * SPM_MAX_TOPK + ent];
        const unsigned char* base;
        if (code >= 0) {
            if (code >= a.n_slots) { atomicOr(a.status, kStatusBadSlot); return false; }
            base = a.pool + size_t(code) * a.blob_bytes;
        } else {
            if (-1 - code >= a.n_shared) { atomicOr(a.status, kStatusBadSlot); return false; }
            base = a.shared + size_t(-1 - code) * a.blob_bytes;
        }
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

    // activations of this lane's groups (group g = ch * 32 + lane), their sums, and the partial y
    float xr[NCH][32], ya[NCH][32];
    {
        const float* xt = a.x + size_t(tok) * D;
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            const int g = ch * 32 + lane;
#pragma unroll
            for (int v = 0; v < 32; v += 4) {
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (g < n_grp) t = *reinterpret_cast<const float4*>(xt + g * 32 + v);
                xr[ch][v] = t.x; xr[ch][v + 1] = t.y; xr[ch][v + 2] = t.z; xr[ch][v + 3] = t.w;
            }
#pragma unroll
            for (int v = 0; v < 32; ++v) ya[ch][v] = 0.f;
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);

    int cur_ent = -1;
    float wk = 0.f;
    int done = 0;
    bool halt = false;
    if (ok) {
        for (int i = 0; i < my_n; ++i) {
            if (i >= __shfl_sync(0xffffffffu, n_issued, 0)) break;
            const int st = i % depth;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8u * st, (i / depth) & 1, kWaitLimitNs))) {
                if (lane == 0) atomicOr(a.status, kStatusCopyTimeout);
                ok = false;
                break;
            }
            done = i + 1;
            const int r = r_begin + wi + i * nw;
            const int ent = r / I;
            if (ent != cur_ent) {
                cur_ent = ent;
                const int kk = a.kidx[tok * SPM_MAX_TOPK + ent];
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
                    float dg = 0.f, du = 0.f;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float fg[8], fu[8];
                        unpack_q4_word(wg[q], fg);
                        unpack_q4_word(wu[q], fu);
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            dg = fmaf(fg[v], xr[ch][q * 8 + v], dg);
                            du = fmaf(fu[v], xr[ch][q * 8 + v], du);
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
            if (!mbar_wait_bounded(bar0 + 8u * (i % depth), (i / depth) & 1, kWaitLimitNs)) break;
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
                *reinterpret_cast<float4*>(red + wi * D + g * 32 + v) = make_float4(ya[ch][v], ya[ch][v + 1], ya[ch][v + 2], ya[ch][v + 3]);
        }
    }
    __syncthreads();
    float* out = a.partial + (size_t(tok) * G + c) * D;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        float acc = red[d];
        for (int w2 = 1; w2 < nw; ++w2) acc += red[w2 * D + d];
        out[d] = acc;
    }
    if (a.clock) {
        __syncthreads();
        if (threadIdx.x == 0) atomicMax(a.clock + 1, global_timer_ns());
    }
}

// Launch shape for 4-bit rows. The cross-warp reduction needs warps * D floats of shared memory,
// which for these short rows is more than a shallow ring would take, so the ring depth is raised
// until it covers it.
inline void ffn_gemv_q4_shape(size_t row_bytes, int D, int rows_per_cta, int* warps, int* depth, size_t* smem) {
    int best_w = 8, best_cost = 1 << 30;
    for (int w = 4; w <= kFfnMaxWarps; ++w) {
        const int cost = (rows_per_cta + w - 1) / w;
        if (cost < best_cost || (cost == best_cost && w > best_w)) { best_w = w; best_cost = cost; }
    }
    int d = 8;
    while (d > 2 && size_t(best_w) * d * row_bytes > 160 * 1024) --d;
    size_t ring = size_t(best_w) * d * row_bytes;
    const size_t red = size_t(best_w) * D * sizeof(float);
    if (ring < red) ring = red;
    *warps = best_w;
    *depth = d;
    *smem = ((ring + 15) & ~size_t(15)) + size_t(best_w) * d * 8 + 16;
}

}  // namespace spm
