// Slot-indexed SwiGLU expert FFN for decode (one activation row per token): a weight-streaming
// GEMV bound by HBM bandwidth.
//
//   y = sum_k w_k * W_down,k ( silu(W_gate,k x) * (W_up,k x) )         (+ shared experts, weight 1)
//
// Weights are read in place from the cache slots (the kernel receives slot numbers, nothing is
// gathered). In the packed expert blob, row j holds gate[j][:], up[j][:] and column j of W_down
// back to back, so one contiguous 3*D-element read yields everything intermediate unit j
// contributes: its two dot products and its rank-1 update of y.
//
// Work decomposition: the (expert, j) rows of a token are split evenly over gridDim.x CTAs; in
// a CTA each warp owns a private ring of row buffers in shared memory that lane 0 keeps full
// with 1-D bulk async copies (cp.async.bulk + mbarrier byte counting, no multicast), so about
// 190 KB per SM are in flight without costing registers. Per-warp partial y vectors live in
// registers, are summed across warps in a fixed order through shared memory, and each CTA
// writes one partial row; ffn_reduce_kernel adds the partials in CTA order (deterministic, so
// outputs are bitwise reproducible for a given launch geometry).
#pragma once

#include "ptx.cuh"
#include "../../include/spm.h"

namespace spm {

constexpr int kFfnWarps = 8;
constexpr int kFfnThreads = kFfnWarps * 32;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s: give up, set status, return

// kernel status bits (device int, read by the host)
constexpr int kStatusCopyTimeout = 1;
constexpr int kStatusBadSlot = 2;

template <int MAXNB>
struct FfnArgs {
    const unsigned char* pool;      // slot pool of this layer
    const unsigned char* shared;    // shared-expert blobs of this layer (may be null)
    const float* x;                 // [nb][D] router input
    const float* w;                 // [nb][K] routing weights
    float* partial;                 // [nb][gridDim.x][D]
    int* status;
    unsigned long long blob_bytes;
    int I, K, n_slots, n_shared;
    unsigned char count[MAXNB];                     // expert entries of token t in this launch
    short code[MAXNB * SPM_MAX_TOPK];               // >= 0: slot number; < 0: shared expert -1-s
    unsigned char kidx[MAXNB * SPM_MAX_TOPK];       // column of w[t][.]; 255: weight 1
};

template <typename WT, int NSEG, int MAXNB>
__global__ void __launch_bounds__(kFfnThreads, 1)
ffn_gemv_kernel(const __grid_constant__ FfnArgs<MAXNB> a, const int depth) {
    constexpr int VEC = 16 / int(sizeof(WT));
    constexpr int D = NSEG * 32 * VEC;
    constexpr uint32_t ROWB = 3u * D * sizeof(WT);

    extern __shared__ __align__(128) unsigned char smem[];
    const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tok = blockIdx.y;
    const int G = gridDim.x, c = blockIdx.x;
    const int I = a.I;
    const int R = int(a.count[tok]) * I;
    const int r_begin = int((long long)R * c / G);
    const int r_end = int((long long)R * (c + 1) / G);
    const int span = r_end - r_begin - wi;
    const int my_n = span > 0 ? (span + kFfnWarps - 1) / kFfnWarps : 0;

    unsigned char* ring = smem + size_t(wi) * depth * ROWB;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + size_t(kFfnWarps) * depth * ROWB);
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
        const int r = r_begin + wi + i * kFfnWarps;
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

    // router input of this token, laid out like one 16-byte weight vector per lane and segment
    float xr[NSEG][VEC];
    float ya[NSEG][VEC];
    {
        const float* xt = a.x + size_t(tok) * D;
#pragma unroll
        for (int s = 0; s < NSEG; ++s) {
#pragma unroll
            for (int v = 0; v < VEC; v += 4) {
                const float4 t = *reinterpret_cast<const float4*>(xt + s * 32 * VEC + lane * VEC + v);
                xr[s][v] = t.x; xr[s][v + 1] = t.y; xr[s][v + 2] = t.z; xr[s][v + 3] = t.w;
            }
#pragma unroll
            for (int v = 0; v < VEC; ++v) ya[s][v] = 0.f;
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);

    int cur_ent = -1;
    float wk = 0.f;
    int done = 0;
    bool halt = false;   // lane 0: a bad slot number was seen, issue nothing more
    if (ok) {
        for (int i = 0; i < my_n; ++i) {
            // rows past the last issued copy exist only after a bad slot: stop there
            if (i >= __shfl_sync(0xffffffffu, n_issued, 0)) break;
            const int st = i % depth;
            // warp-uniform outcome: a lane that gave up makes the whole warp give up
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8u * st, (i / depth) & 1, kWaitLimitNs))) {
                if (lane == 0) atomicOr(a.status, kStatusCopyTimeout);
                ok = false;
                break;
            }
            done = i + 1;
            const int r = r_begin + wi + i * kFfnWarps;
            const int ent = r / I;
            if (ent != cur_ent) {
                cur_ent = ent;
                const int kk = a.kidx[tok * SPM_MAX_TOPK + ent];
                wk = kk == 255 ? 1.f : a.w[size_t(tok) * a.K + kk];
            }
            const unsigned char* buf = ring + size_t(st) * ROWB;
            float pg = 0.f, pu = 0.f;
#pragma unroll
            for (int s = 0; s < NSEG; ++s) {
                const uint4 vg = *reinterpret_cast<const uint4*>(buf + (s * 32 + lane) * 16);
                const uint4 vu = *reinterpret_cast<const uint4*>(buf + D * sizeof(WT) + (s * 32 + lane) * 16);
                float fg[VEC], fu[VEC];
                unpack16(vg, fg);
                unpack16(vu, fu);
#pragma unroll
                for (int v = 0; v < VEC; ++v) {
                    pg = fmaf(fg[v], xr[s][v], pg);
                    pu = fmaf(fu[v], xr[s][v], pu);
                }
            }
            pg = warp_sum(pg);
            pu = warp_sum(pu);
            const float act = pg / (1.f + expf(-pg)) * pu * wk;
#pragma unroll
            for (int s = 0; s < NSEG; ++s) {
                const uint4 vd = *reinterpret_cast<const uint4*>(buf + 2 * D * sizeof(WT) + (s * 32 + lane) * 16);
                float fd[VEC];
                unpack16(vd, fd);
#pragma unroll
                for (int v = 0; v < VEC; ++v) ya[s][v] = fmaf(act, fd[v], ya[s][v]);
            }
            __syncwarp();   // every lane is done with this buffer before it is refilled
            if (lane == 0 && n_issued < my_n && !halt) {
                if (issue(n_issued)) ++n_issued;
                else halt = true;
            }
        }
    }
    if (!ok) {
        // leave no copy in flight into shared memory that is about to be released
        n_issued = __shfl_sync(0xffffffffu, n_issued, 0);
        for (int i = done; i < n_issued; ++i)
            if (!mbar_wait_bounded(bar0 + 8u * (i % depth), (i / depth) & 1, kWaitLimitNs)) break;
    }

    // sum the warps' partial y in warp order, one partial row per CTA
    __syncthreads();
    float* red = reinterpret_cast<float*>(smem);
#pragma unroll
    for (int s = 0; s < NSEG; ++s)
#pragma unroll
        for (int v = 0; v < VEC; v += 4)
            *reinterpret_cast<float4*>(red + wi * D + s * 32 * VEC + lane * VEC + v) =
                make_float4(ya[s][v], ya[s][v + 1], ya[s][v + 2], ya[s][v + 3]);
    __syncthreads();
    float* out = a.partial + (size_t(tok) * G + c) * D;
    for (int d = threadIdx.x; d < D; d += kFfnThreads) {
        float acc = red[d];
#pragma unroll
        for (int w2 = 1; w2 < kFfnWarps; ++w2) acc += red[w2 * D + d];
        out[d] = acc;
    }
}

// h_out[t][d] = h_in[t][d] + sum over CTAs (in CTA order) of partial[t][c][d]
__global__ void ffn_reduce_kernel(const float* __restrict__ partial, const float* h_in, float* h_out,
                                  int G, int D) {
    const int tok = blockIdx.y;
    const int d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= D) return;
    const float* p = partial + size_t(tok) * G * D + d;
    float acc = 0.f;
    int c = 0;
    for (; c + 4 <= G; c += 4) {
        const float p0 = p[size_t(c) * D], p1 = p[size_t(c + 1) * D];
        const float p2 = p[size_t(c + 2) * D], p3 = p[size_t(c + 3) * D];
        acc += p0; acc += p1; acc += p2; acc += p3;
    }
    for (; c < G; ++c) acc += p[size_t(c) * D];
    h_out[size_t(tok) * D + d] = h_in[size_t(tok) * D + d] + acc;
}

// Shared-memory bytes of the GEMV kernel for a row of `row_bytes` and ring depth `depth`.
inline size_t ffn_gemv_smem(size_t row_bytes, int depth) {
    return size_t(kFfnWarps) * depth * row_bytes + size_t(kFfnWarps) * depth * 8;
}

}  // namespace spm
