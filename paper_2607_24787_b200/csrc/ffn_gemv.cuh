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
// 170-220 KB per SM are in flight without costing registers. The host picks the number of warps
// per CTA so that rows divide evenly: the kernel ends when its busiest warp does. Per-warp partial y vectors live in
// registers, are summed across warps in a fixed order through shared memory, and each CTA
// writes one partial row; ffn_reduce_kernel adds the partials in CTA order (deterministic, so
// outputs are bitwise reproducible for a given launch geometry).
#pragma once

#include "ptx.cuh"
#include "../../include/spm.h"

namespace spm {

constexpr int kFfnMaxWarps = 9;                    // 9 * 32 threads * 216 registers fit one SM
constexpr int kFfnMaxThreads = kFfnMaxWarps * 32;
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
    unsigned long long* clock;      // optional {earliest CTA start, latest CTA end} in ns (globaltimer)
    const unsigned* ready;          // optional per-slot arrival counters of this pool (device-side wait)
    const short* dev_code;          // optional [nb][K] slot numbers left in device memory by the routing kernel:
                                    // the launch then needs no host knowledge of the routing (count/code/kidx unused;
                                    // token t has K routed entries followed by the n_shared shared experts)
    unsigned want[SPM_MAX_TOPK];    // token 0 only: entry k's expert has landed once ready[watch[k]] >= want[k]
    short watch[SPM_MAX_TOPK];      //   (the counter of the slot that leads the batch of copies entry k's slot was filled by)
    unsigned long long blob_bytes;
    int I, K, n_slots, n_shared;
    unsigned char count[MAXNB];                     // expert entries of token t in this launch
    short code[MAXNB * SPM_MAX_TOPK];               // >= 0: slot number; < 0: shared expert -1-s
    unsigned char kidx[MAXNB * SPM_MAX_TOPK];       // column of w[t][.]; 255: weight 1

    __device__ __forceinline__ int entries(int tok) const { return dev_code ? K + n_shared : int(count[tok]); }
    // slot code of entry `ent`; kBadCode when the device-side table names no slot
    __device__ __forceinline__ int code_of(int tok, int ent) const {
        if (!dev_code) return code[tok * SPM_MAX_TOPK + ent];
        if (ent >= K) return -1 - (ent - K);
        const int s = __ldcg(dev_code + tok * K + ent);
        return s >= 0 ? s : (1 << 20);                  // no slot: fails the range check below
    }
    __device__ __forceinline__ int kidx_of(int tok, int ent) const {
        if (!dev_code) return kidx[tok * SPM_MAX_TOPK + ent];
        return ent < K ? ent : 255;
    }
};

template <typename WT, int NSEG, int MAXNB>
__global__ void __launch_bounds__(kFfnMaxThreads, 1)
ffn_gemv_kernel(const __grid_constant__ FfnArgs<MAXNB> a, const int depth) {
    constexpr int VEC = 16 / int(sizeof(WT));
    constexpr int D = NSEG * 32 * VEC;
    constexpr uint32_t ROWB = 3u * D * sizeof(WT);

    extern __shared__ __align__(128) unsigned char smem[];
#ifdef SPM_FFN_TIMESTAMPS
    const unsigned long long ts_start = global_timer_ns();
    unsigned long long ts_first = 0, ts_loop = 0;
#endif
    grid_dep_launch();
    const unsigned long long t_entry = (a.clock && threadIdx.x == 0) ? global_timer_ns() : 0ull;
    const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nw = blockDim.x >> 5;      // warps per CTA, chosen by the host to balance rows per warp
    const int tok = blockIdx.y;
    const int G = gridDim.x, c = blockIdx.x;
    const int I = a.I;
    const int R = a.entries(tok) * I;
    const int r_begin = int((long long)R * c / G);
    const int r_end = int((long long)R * (c + 1) / G);
    const int span = r_end - r_begin - wi;
    const int my_n = span > 0 ? (span + nw - 1) / nw : 0;

    unsigned char* ring = smem + size_t(wi) * depth * ROWB;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + size_t(nw) * depth * ROWB);
    const uint32_t bar0 = smem_u32(bars + wi * depth);
    const uint32_t ring0 = smem_u32(ring);

    if (lane == 0) {
        for (int d = 0; d < depth; ++d) mbar_init(bar0 + 8u * d, 1);
        fence_barrier_init();
    }
    __syncwarp();
    // everything above is independent of the preceding kernel; routing results are read below
    grid_dep_wait();
    // window start: kernel entry, or the end of the dependency wait when launched ahead of its predecessor's end
    if (a.clock && threadIdx.x == 0) atomicMin(a.clock, a.dev_code ? global_timer_ns() : t_entry);

    const uint64_t pol = policy_evict_first();
    bool ok = true;
    int src_ent = -1;                          // lane 0: entry being streamed and where its blob starts
    const unsigned char* src_base = nullptr;   //         (null: the entry cannot be served)

    // Blob of entry `ent`, resolved once per entry: slot number (launch arguments, or the routing
    // kernel's device-side codes), range check, and with device-side waiting the arrival of its copy.
    auto resolve = [&](int ent) -> const unsigned char* {
        const int code = a.code_of(tok, ent);
        if (code < 0) {
            if (-1 - code >= a.n_shared) { atomicOr(a.status, kStatusBadSlot); return nullptr; }
            return a.shared + size_t(-1 - code) * a.blob_bytes;
        }
        if (code >= a.n_slots) { atomicOr(a.status, kStatusBadSlot); return nullptr; }
        if (a.ready) {
            // Device-side wait: the copy stream bumps the slot's counter after the expert's bytes
            // have landed. Bounded; on timeout the status word is set and the launch winds down.
            const unsigned* f = a.ready + a.watch[ent];
            const unsigned want = a.want[ent];
            const unsigned long long t0 = global_timer_ns();
            for (;;) {
                unsigned v;
                asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(f) : "memory");
                if (int(v - want) >= 0) break;
                __nanosleep(200);
                if (global_timer_ns() - t0 > kWaitLimitNs) { atomicOr(a.status, kStatusCopyTimeout); return nullptr; }
            }
            asm volatile("fence.proxy.async;" ::: "memory");   // the weights are read through the async proxy
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
#ifdef SPM_FFN_TIMESTAMPS
            if (i == 0) ts_first = global_timer_ns();
#endif
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

#ifdef SPM_FFN_TIMESTAMPS
    ts_loop = global_timer_ns();
#endif
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
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        float acc = red[d];
        for (int w2 = 1; w2 < nw; ++w2) acc += red[w2 * D + d];
        out[d] = acc;
    }
    if (a.clock) {
        __syncthreads();
        if (threadIdx.x == 0) atomicMax(a.clock + 1, global_timer_ns());
    }
#ifdef SPM_FFN_TIMESTAMPS
    // profiling aid: per-warp phase times and the SM id, appended behind the partial rows
    if (lane == 0) {
        unsigned long long* ts = reinterpret_cast<unsigned long long*>(a.partial + size_t(gridDim.y) * G * D) + (size_t(c) * nw + wi) * 5;
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        ts[0] = ts_start; ts[1] = ts_first; ts[2] = ts_loop; ts[3] = global_timer_ns(); ts[4] = smid;
    }
#endif
}

// h_out[t][d] = h_in[t][d] + sum over CTAs (in CTA order) of partial[t][c][d].
// A block owns kReduceCols columns; its kReduceGroups thread groups each sum a contiguous run of
// partial rows (all loads of a thread are independent, so they are in flight together), and the
// group sums are combined in group order: the summation order is fixed by (G, launch geometry).
constexpr int kReduceCols = 32;
constexpr int kReduceGroups = 8;
constexpr int kReduceMaxRows = 40;     // rows per group: kReduceGroups * kReduceMaxRows >= max G

static __global__ void __launch_bounds__(kReduceCols * kReduceGroups)
ffn_reduce_kernel(const float* __restrict__ partial, const float* h_in, float* h_out, int G, int D,
                  unsigned long long* clock = nullptr) {
    __shared__ float part[kReduceGroups][kReduceCols];
    grid_dep_launch();
    grid_dep_wait();
    if (clock && threadIdx.x == 0) atomicMin(clock, global_timer_ns());
    const int tok = blockIdx.y;
    const int col = threadIdx.x % kReduceCols, grp = threadIdx.x / kReduceCols;
    const int d = blockIdx.x * kReduceCols + col;
    const int per = (G + kReduceGroups - 1) / kReduceGroups;
    const int c0 = grp * per, c1 = min(G, c0 + per);
    const float* p = partial + size_t(tok) * G * D + d;
    float v[kReduceMaxRows];
#pragma unroll
    for (int i = 0; i < kReduceMaxRows; ++i) v[i] = (d < D && c0 + i < c1) ? __ldcg(p + size_t(c0 + i) * D) : 0.f;
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kReduceMaxRows; ++i) acc += v[i];
    part[grp][col] = acc;
    __syncthreads();
    if (grp == 0 && d < D) {
        float tot = part[0][col];
#pragma unroll
        for (int g = 1; g < kReduceGroups; ++g) tot += part[g][col];
        h_out[size_t(tok) * D + d] = h_in[size_t(tok) * D + d] + tot;
    }
    if (clock) {
        __syncthreads();
        if (threadIdx.x == 0) atomicMax(clock + 1, global_timer_ns());
    }
}

constexpr size_t kFfnSmemLimit = 232448;   // 227 KB per CTA

// Shared-memory bytes of the GEMV kernel: `warps` private rings of `depth` rows + their barriers.
inline size_t ffn_gemv_smem(size_t row_bytes, int warps, int depth) {
    return size_t(warps) * depth * row_bytes + size_t(warps) * depth * 8;
}

// Launch shape for `rows_per_cta` rows of `row_bytes`: the warp count that leaves the fewest rows
// on the busiest warp (the kernel ends when that warp does), then the most bytes in flight.
inline void ffn_gemv_shape(size_t row_bytes, int rows_per_cta, int* warps, int* depth) {
    int best_w = 0, best_d = 0, best_cost = 1 << 30;
    size_t best_flight = 0;
    for (int w = 4; w <= kFfnMaxWarps; ++w) {
        int d = int((kFfnSmemLimit - 1024) / (size_t(w) * row_bytes));
        if (d > 4) d = 4;
        if (d < 2 && !(w == 4 && d == 1)) continue;      // want double buffering; 4 warps x 1 is the last resort
        const int cost = (rows_per_cta + w - 1) / w;
        const size_t flight = size_t(w) * d * row_bytes;
        if (cost < best_cost || (cost == best_cost && flight > best_flight)) {
            best_w = w; best_d = d; best_cost = cost; best_flight = flight;
        }
    }
    *warps = best_w;
    *depth = best_d;
}

}  // namespace spm
