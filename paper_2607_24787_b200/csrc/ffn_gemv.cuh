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
//
// Arithmetic of a row: the 24 shared-memory reads of a lane are issued ahead of the math that
// consumes them; products run as packed fp32 pairs (fma.rn.f32x2: even / odd elements of a 16-byte
// vector accumulate side by side, two pair accumulators per dot product), silu uses the fast
// exponential and division (relative error about 1e-6, far inside the parity tolerance).
//
// Launched with the programmatic-serialisation attribute and `early` set (slot numbers known to
// the host), a CTA starts its first weight copies before griddepcontrol.wait, i.e. while the
// preceding kernel of the stream is still running: weights never depend on that kernel, only the
// router input and the routing weights do, and those are read after the wait.
#pragma once

#include "ptx.cuh"
#include "../../include/spm.h"

namespace spm {

constexpr int kFfnMaxWarps = 9;                    // 9 * 32 threads * 216 registers fit one SM
constexpr int kFfnMaxThreads = kFfnMaxWarps * 32;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // default limit of every device-side wait (2 s): give up, set status, return

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
    unsigned long long wait_limit_ns;   // every wait in the kernel gives up after this long (0: the 2 s default)
    int early;                      // 1: start the first weight copies before the launch dependency resolves (needs slot numbers in `code`)
    unsigned char count[MAXNB];                     // expert entries of token t in this launch
    short code[MAXNB * SPM_MAX_TOPK];               // >= 0: slot number; < 0: shared expert -1-s
    unsigned char kidx[MAXNB * SPM_MAX_TOPK];       // column of w[t][.]; 255: weight 1

    __device__ __forceinline__ unsigned long long limit() const { return wait_limit_ns ? wait_limit_ns : kWaitLimitNs; }
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

// Device-side wait for a batch of expert copies: the copy stream bumps the batch leader's counter
// after the batch's bytes have landed. Bounded: false when the limit ran out (the caller records
// the status and winds the launch down).
__device__ __forceinline__ bool ffn_wait_arrival(const unsigned* counter, unsigned want, unsigned long long limit_ns) {
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        unsigned v;
        asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if (int(v - want) >= 0) break;
        __nanosleep(200);
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
    asm volatile("fence.proxy.async;" ::: "memory");   // the weights are read through the async proxy
    return true;
}

// packed fp32 pairs (one 64-bit register pair) for fma.rn.f32x2
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t pack2u(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// 16 bytes of weights -> fp32 pairs {element 2i, element 2i + 1}
__device__ __forceinline__ void unpack16p(const uint4& v, uint64_t (&f)[4]) {   // bf16: 8 values
    f[0] = pack2u(v.x << 16, v.x & 0xffff0000u); f[1] = pack2u(v.y << 16, v.y & 0xffff0000u);
    f[2] = pack2u(v.z << 16, v.z & 0xffff0000u); f[3] = pack2u(v.w << 16, v.w & 0xffff0000u);
}
__device__ __forceinline__ void unpack16p(const uint4& v, uint64_t (&f)[2]) {   // fp32: 4 values
    f[0] = pack2u(v.x, v.y); f[1] = pack2u(v.z, v.w);
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

template <typename WT, int NSEG, int MAXNB>
__global__ void __launch_bounds__(kFfnMaxThreads, 1)
ffn_gemv_kernel(const __grid_constant__ FfnArgs<MAXNB> a, const int depth) {
    constexpr int VEC = 16 / int(sizeof(WT));
    constexpr int D = NSEG * 32 * VEC;
    constexpr uint32_t ROWB = 3u * D * sizeof(WT);
    constexpr uint32_t PART = D * sizeof(WT);      // bytes of one matrix's part of a blob row

    extern __shared__ __align__(128) unsigned char smem[];
    grid_dep_launch();
    const unsigned long long t_entry = (a.clock && threadIdx.x == 0) ? global_timer_ns() : 0ull;
    const int wi = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned long long wait_limit = a.limit();
    const int nw = blockDim.x >> 5;      // warps per CTA, chosen by the host to balance rows per warp
    const int tok = blockIdx.y;
    const int G = gridDim.x, c = blockIdx.x;
    const int I = a.I;
    const int R = a.entries(tok) * I;
    // even split: CTA c takes q rows, the first R % G CTAs one more (one 32-bit division)
    const int q_rows = R / G, rem_rows = R - q_rows * G;
    const int r_begin = q_rows * c + min(c, rem_rows);
    const int r_end = r_begin + q_rows + (c < rem_rows ? 1 : 0);
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
    // Everything above is independent of the preceding kernel. Routing results are read below; with
    // `early` the first weight copies go out before the dependency wait (weights never depend on it).
    const bool early = a.early && !a.dev_code;
    if (!early) grid_dep_wait();
    // window start: kernel entry, or the end of the dependency wait when launched ahead of its predecessor's end
    if (a.clock && threadIdx.x == 0 && !early) atomicMin(a.clock, a.dev_code ? global_timer_ns() : t_entry);

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
        if (a.ready && !ffn_wait_arrival(a.ready + a.watch[ent], a.want[ent], wait_limit)) {
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

    // router input of this token, laid out like one 16-byte weight vector per lane and segment; its
    // loads go out ahead of the weight copies so that they do not queue behind them
    float xr[NSEG][VEC];
    uint64_t ya[NSEG][VEC / 2];        // partial y, packed pairs
    auto load_x = [&]() {
        const float* xt = a.x + size_t(tok) * D;
#pragma unroll
        for (int s = 0; s < NSEG; ++s)
#pragma unroll
            for (int v = 0; v < VEC; v += 4) {
                const float4 t = *reinterpret_cast<const float4*>(xt + s * 32 * VEC + lane * VEC + v);
                xr[s][v] = t.x; xr[s][v + 1] = t.y; xr[s][v + 2] = t.z; xr[s][v + 3] = t.w;
            }
    };
    if (!early) load_x();
    int n_issued = 0;
    if (lane == 0) {
        for (; n_issued < depth && n_issued < my_n; ++n_issued)
            if (!issue(n_issued)) { ok = false; break; }
    }
    if (early) {
        grid_dep_wait();
        if (a.clock && threadIdx.x == 0) atomicMin(a.clock, global_timer_ns());
        load_x();
    }
#pragma unroll
    for (int s = 0; s < NSEG; ++s)
#pragma unroll
        for (int v = 0; v < VEC / 2; ++v) ya[s][v] = 0ull;

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
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8u * st, (i / depth) & 1, wait_limit))) {
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
            // gate / up rows first (16 reads), then the down row's reads go out ahead of the reductions
            const uint32_t b32 = ring0 + uint32_t(st) * ROWB + lane * 16;
            uint4 vg[NSEG], vu[NSEG];
#pragma unroll
            for (int s = 0; s < NSEG; ++s) { vg[s] = lds128(b32 + s * 512); vu[s] = lds128(b32 + PART + s * 512); }
            uint64_t ag[2] = {0ull, 0ull}, au[2] = {0ull, 0ull};
#pragma unroll
            for (int s = 0; s < NSEG; ++s) {
                uint64_t fg[VEC / 2], fu[VEC / 2];
                unpack16p(vg[s], fg);
                unpack16p(vu[s], fu);
#pragma unroll
                for (int v = 0; v < VEC / 2; ++v) {
                    const uint64_t xp = pack2(xr[s][2 * v], xr[s][2 * v + 1]);
                    ag[v & 1] = fma2(fg[v], xp, ag[v & 1]);
                    au[v & 1] = fma2(fu[v], xp, au[v & 1]);
                }
            }
            uint4 vd[NSEG];
#pragma unroll
            for (int s = 0; s < NSEG; ++s) vd[s] = lds128(b32 + 2 * PART + s * 512);
            float a0, a1, a2, a3;
            unpack2(ag[0], a0, a1); unpack2(ag[1], a2, a3);
            float pg = (a0 + a1) + (a2 + a3);
            unpack2(au[0], a0, a1); unpack2(au[1], a2, a3);
            float pu = (a0 + a1) + (a2 + a3);
            pg = warp_sum(pg);
            pu = warp_sum(pu);
            const float act = __fdividef(pg, 1.f + __expf(-pg)) * pu * wk;
            const uint64_t ap = pack2(act, act);
#pragma unroll
            for (int s = 0; s < NSEG; ++s) {
                uint64_t fd[VEC / 2];
                unpack16p(vd[s], fd);
#pragma unroll
                for (int v = 0; v < VEC / 2; ++v) ya[s][v] = fma2(ap, fd[v], ya[s][v]);
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
            if (!mbar_wait_bounded(bar0 + 8u * (i % depth), (i / depth) & 1, wait_limit)) break;
    }

    // Sum the warps' partial y in warp order, one partial row per CTA. A warp stages its values in
    // its own ring (all its copies have landed and been read), so it need not wait for the others
    // first: as float4s, one per (segment, quad, lane), so that stores and loads of a warp are
    // contiguous; a thread has the values of all warps in flight at once and adds them in warp order.
    constexpr int Q = VEC / 4;                  // float4s per lane and segment
    constexpr int NP = D / 4;                   // float4 positions of a row
    static_assert(ROWB >= NP * sizeof(float4), "a ring row holds a warp's partial y");
    {
        float4* mine = reinterpret_cast<float4*>(ring);
#pragma unroll
        for (int s = 0; s < NSEG; ++s)
#pragma unroll
            for (int h = 0; h < Q; ++h) {
                float4 t;
                unpack2(ya[s][2 * h], t.x, t.y);
                unpack2(ya[s][2 * h + 1], t.z, t.w);
                mine[s * (32 * Q) + h * 32 + lane] = t;
            }
    }
    __syncthreads();
    const size_t ring_stride = size_t(depth) * ROWB;
    float* out = a.partial + (size_t(tok) * G + c) * D;
    for (int p = threadIdx.x; p < NP; p += blockDim.x) {
        float4 v[kFfnMaxWarps];
#pragma unroll
        for (int w2 = 0; w2 < kFfnMaxWarps; ++w2)
            if (w2 < nw) v[w2] = reinterpret_cast<const float4*>(smem + w2 * ring_stride)[p];
        float4 acc = v[0];
#pragma unroll
        for (int w2 = 1; w2 < kFfnMaxWarps; ++w2)
            if (w2 < nw) { acc.x += v[w2].x; acc.y += v[w2].y; acc.z += v[w2].z; acc.w += v[w2].w; }
        const int s = p / (32 * Q), h = (p / 32) % Q, ln = p % 32;
        *reinterpret_cast<float4*>(out + s * 32 * VEC + ln * VEC + 4 * h) = acc;
    }
    if (a.clock) {
        __syncthreads();
        if (threadIdx.x == 0) atomicMax(a.clock + 1, global_timer_ns());
    }
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

// Launch shape for `rows_per_cta` rows of `row_bytes`. A ring of at least three rows per warp comes first:
// with two, the slot of a row is blocked while that row is being computed, and the first row of a launch
// is slow to compute (cold instruction fetch), so the copy stream ran dry once per launch (Qwen3 shape,
// plain launches: 9 warps x 2 rows 17.5 us, 6 warps x 3 rows 16.5 us; same bytes in flight). Among such
// shapes the most warps win. Rows too large for that fall back to the warp count that leaves the fewest
// rows on the busiest warp (the kernel ends when that warp does), then the most bytes in flight.
inline void ffn_gemv_shape(size_t row_bytes, int rows_per_cta, int* warps, int* depth) {
    int best_w = 0, best_d = 0;
    for (int w = 4; w <= kFfnMaxWarps; ++w) {
        int d = int((kFfnSmemLimit - 1024) / (size_t(w) * row_bytes));
        if (d > 4) d = 4;
        if (d >= 3 && (w > best_w || (w == best_w && d > best_d))) { best_w = w; best_d = d; }
    }
    if (best_w == 0) {
        int best_cost = 1 << 30;
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
    }
    *warps = best_w;
    *depth = best_d;
}

}  // namespace spm
