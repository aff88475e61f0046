// spm_ffn_noalloc: the slot-indexed SwiGLU expert FFN for one token, for callers that are not
// allowed to allocate. It launches the same two kernels as spm_moe_ffn (ffn_gemv_kernel writes
// one partial output row per CTA, ffn_reduce_kernel adds them and the residual), but the partial
// rows live in a fixed array that is part of the library image instead of a caller arena.
//
// Who needs this: code running where cudaMalloc (or any allocating call) is off limits -- inside
// a latency-critical serving loop that has frozen its memory map, in a process whose whole device
// memory is already handed to another allocator, or in a callback that may not block on the
// driver's allocation lock. Such callers cannot create an spm_ctx either (that creates events and
// pinned memory), so this entry point takes plain pointers and keeps no state but the array.
#include <cstdint>
#include <mutex>
#include <string>

#include <cuda_runtime.h>

#include "../../include/spm.h"
#include "ffn_gemv.cuh"

namespace spm {
void set_thread_error(const std::string& msg);   // defined next to spm_last_error
}

using namespace spm;

namespace {

struct bf16_t { uint16_t v; };

constexpr int kNoAllocMaxCtas = SPM_NOALLOC_MAX_CTAS;
constexpr int kNoAllocMaxHidden = SPM_NOALLOC_MAX_HIDDEN;
constexpr size_t kHeaderBytes = 256;   // status word, kept apart from the partial rows
constexpr size_t kScratchBytes = kHeaderBytes + size_t(kNoAllocMaxCtas) * kNoAllocMaxHidden * sizeof(float);
static_assert(kScratchBytes == SPM_NOALLOC_SCRATCH_BYTES, "header and implementation agree on the size");

// Every GPU that loads the library holds one copy of this array until the process exits.
// In host code the name below is only a handle for cudaGetSymbolAddress: it is not a device
// address and must never be passed to a kernel directly.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {};
int g_num_sms[kMaxDevices] = {};

int fail(int code, const std::string& msg) {
    set_thread_error(msg);
    return code;
}

template <typename WT, int NSEG>
cudaError_t launch(const FfnArgs<1>& a, int G, int warps, int depth, size_t smem, cudaStream_t st) {
    ffn_gemv_kernel<WT, NSEG, 1><<<dim3(G, 1), warps * 32, smem, st>>>(a, depth);
    return cudaGetLastError();
}

template <typename WT>
cudaError_t launch_seg(int nseg, const FfnArgs<1>& a, int G, int w, int d, size_t smem, cudaStream_t st) {
    switch (nseg) {
        case 1: return launch<WT, 1>(a, G, w, d, smem, st);
        case 2: return launch<WT, 2>(a, G, w, d, smem, st);
        case 3: return launch<WT, 3>(a, G, w, d, smem, st);
        case 4: return launch<WT, 4>(a, G, w, d, smem, st);
        case 5: return launch<WT, 5>(a, G, w, d, smem, st);
        case 6: return launch<WT, 6>(a, G, w, d, smem, st);
        case 7: return launch<WT, 7>(a, G, w, d, smem, st);
        case 8: return launch<WT, 8>(a, G, w, d, smem, st);
    }
    return cudaErrorInvalidValue;
}

// The kernel's shared-memory ring needs the opt-in limit; set for every variant during a device's
// one-time set-up, so that no later call (perhaps inside a stream capture) has to.
template <typename WT, int NSEG>
cudaError_t allow_smem() {
    return cudaFuncSetAttribute(ffn_gemv_kernel<WT, NSEG, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kFfnSmemLimit));
}
template <typename WT>
cudaError_t allow_smem_all() {
    cudaError_t e = allow_smem<WT, 1>();
    if (e == cudaSuccess) e = allow_smem<WT, 2>();
    if (e == cudaSuccess) e = allow_smem<WT, 3>();
    if (e == cudaSuccess) e = allow_smem<WT, 4>();
    if (e == cudaSuccess) e = allow_smem<WT, 5>();
    if (e == cudaSuccess) e = allow_smem<WT, 6>();
    if (e == cudaSuccess) e = allow_smem<WT, 7>();
    if (e == cudaSuccess) e = allow_smem<WT, 8>();
    return e;
}

bool aligned(const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; }

}  // namespace

extern "C" int spm_ffn_noalloc(const spm_model_cfg* cfg, const void* blobs, int n_blobs, const int32_t* which,
                               const float* w, int count, const float* x_norm, float* h_inout, void* stream,
                               int wait_and_check) {
    if (!cfg || !blobs || !which || !w || !x_norm || !h_inout) return fail(SPM_ERR_INVALID_ARG, "spm_ffn_noalloc: null argument");
    if (cfg->dtype != SPM_DTYPE_FP32 && cfg->dtype != SPM_DTYPE_BF16)
        return fail(SPM_ERR_CONFIG, "spm_ffn_noalloc: only fp32 and bf16 experts are supported");
    const int seg = cfg->dtype == SPM_DTYPE_BF16 ? 256 : 128;
    if (cfg->hidden < seg || cfg->hidden % seg || cfg->hidden / seg > 8 || cfg->hidden > kNoAllocMaxHidden)
        return fail(SPM_ERR_CONFIG, "spm_ffn_noalloc: hidden " + std::to_string(cfg->hidden) + " not supported: a multiple of " +
                                        std::to_string(seg) + ", at most " + std::to_string(std::min(8 * seg, kNoAllocMaxHidden)) +
                                        " (the built-in scratch array holds " + std::to_string(kNoAllocMaxCtas) + " rows of " +
                                        std::to_string(kNoAllocMaxHidden) + " floats)");
    if (cfg->inter < 1) return fail(SPM_ERR_CONFIG, "spm_ffn_noalloc: inter must be positive");
    if (count < 1 || count > SPM_MAX_TOPK)
        return fail(SPM_ERR_INVALID_ARG, "spm_ffn_noalloc: count " + std::to_string(count) + " outside 1.." + std::to_string(SPM_MAX_TOPK));
    if (n_blobs < 1 || n_blobs > 32767) return fail(SPM_ERR_INVALID_ARG, "spm_ffn_noalloc: n_blobs outside 1..32767");
    for (int i = 0; i < count; ++i)
        if (which[i] < 0 || which[i] >= n_blobs)
            return fail(SPM_ERR_INVALID_ARG, "spm_ffn_noalloc: blob index " + std::to_string(which[i]) + " outside the " + std::to_string(n_blobs) + " blobs given");

    // The kernel reads weight rows with 16-byte bulk copies and the activation row with 16-byte loads,
    // and the combine kernel walks h in place: a misaligned view (an offset slice, say) would fault on
    // the GPU, so it is refused here, before anything is enqueued.
    if (!aligned(blobs, 16) || !aligned(x_norm, 16) || !aligned(h_inout, 16) || !aligned(w, 4))
        return fail(SPM_ERR_INVALID_ARG, "spm_ffn_noalloc: blobs, x_norm and h_inout must be 16-byte aligned, w 4-byte aligned");

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: cudaGetDevice: ") + cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(SPM_ERR_CONFIG, "spm_ffn_noalloc: device ordinal out of range");

    unsigned char* scratch = nullptr;
    int sms = 0;
    {
        // The lock covers only the one-time set-up of this device (it is the current one): the array's
        // device address, the SM count, the kernels' shared-memory attribute. Launches run outside it.
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_ptr[dev]) {
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (e != cudaSuccess || !p) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess || sms < 1) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: cudaDeviceGetAttribute: ") + cudaGetErrorString(e));
            e = allow_smem_all<float>();
            if (e == cudaSuccess) e = allow_smem_all<bf16_t>();
            if (e != cudaSuccess) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: cudaFuncSetAttribute: ") + cudaGetErrorString(e));
            g_num_sms[dev] = sms;
            g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
        }
        scratch = g_scratch_ptr[dev];
        sms = g_num_sms[dev];
    }
    const int G = std::min(sms, kNoAllocMaxCtas);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t elem = cfg->dtype == SPM_DTYPE_BF16 ? 2 : 4;
    const size_t row_bytes = size_t(3) * cfg->hidden * elem;

    // The array keeps whatever the previous call left. The partial rows are overwritten in full by
    // every launch (each CTA stores its whole row); the status word must start at zero.
    e = cudaMemsetAsync(scratch, 0, kHeaderBytes, st);
    if (e != cudaSuccess) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: cudaMemsetAsync: ") + cudaGetErrorString(e));

    FfnArgs<1> a{};
    a.pool = static_cast<const unsigned char*>(blobs);
    a.shared = nullptr;
    a.x = x_norm;
    a.w = w;
    a.partial = reinterpret_cast<float*>(scratch + kHeaderBytes);
    a.status = reinterpret_cast<int*>(scratch);
    a.clock = nullptr;
    a.blob_bytes = row_bytes * size_t(cfg->inter);
    a.I = cfg->inter; a.K = count; a.n_slots = n_blobs; a.n_shared = 0;
    a.count[0] = (unsigned char)count;
    for (int i = 0; i < count; ++i) { a.code[i] = short(which[i]); a.kidx[i] = (unsigned char)i; }
    int warps = 8, depth = 2;
    ffn_gemv_shape(row_bytes, (count * cfg->inter + G - 1) / G, &warps, &depth);
    const size_t smem = ffn_gemv_smem(row_bytes, warps, depth);
    const int nseg = cfg->hidden / seg;
    const int dt = cfg->dtype == SPM_DTYPE_BF16 ? 1 : 0;
    e = dt ? launch_seg<bf16_t>(nseg, a, G, warps, depth, smem, st) : launch_seg<float>(nseg, a, G, warps, depth, smem, st);
    if (e != cudaSuccess) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: expert kernel launch: ") + cudaGetErrorString(e));
    ffn_reduce_kernel<<<dim3((cfg->hidden + kReduceCols - 1) / kReduceCols, 1), kReduceCols * kReduceGroups, 0, st>>>(
        a.partial, h_inout, h_inout, G, cfg->hidden);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: combine kernel launch: ") + cudaGetErrorString(e));
    if (wait_and_check) {
        int status = 0;
        e = cudaStreamSynchronize(st);
        if (e == cudaSuccess) e = cudaMemcpy(&status, scratch, sizeof status, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return fail(SPM_ERR_CUDA, std::string("spm_ffn_noalloc: wait: ") + cudaGetErrorString(e));
        if (status & kStatusCopyTimeout) return fail(SPM_ERR_TIMEOUT, "spm_ffn_noalloc: the expert kernel gave up waiting for a weight copy");
        if (status & kStatusBadSlot) return fail(SPM_ERR_NOT_RESIDENT, "spm_ffn_noalloc: the expert kernel saw a blob index outside the range");
    }
    return SPM_OK;
}
