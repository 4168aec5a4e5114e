// Decode step that allocates nothing and needs no caller scratch: the per-head weight hand-off between the two
// decode kernels (see decode_split.cu) lives in a device array owned by the library instead of in the caller's
// `work` buffer.  Some callers cannot obtain device scratch at call time -- code running inside a memory pool that
// has been sized and frozen up front, a plug-in that is handed its tensors and has no allocator of its own, a
// stream-ordered region where cudaMalloc would synchronise the device -- and for them a fixed array that every
// GPU loading the library carries until exit is the only place such scratch can come from.
#include <atomic>

#include "internal.cuh"

namespace sketchssm {

namespace {

constexpr size_t kStaticWorkFloats = SKETCHSSM_STATIC_WORK_BYTES / sizeof(float);
constexpr int kMaxDevices = 64;

// File-scope device array: 4 MiB per GPU that loads the library, alive until the process exits.  In host code
// this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) float g_static_work[kStaticWorkFloats];

// Device address of g_static_work per device ordinal, resolved on the first call made with that device current.
// Atomic because any calling thread may be the first on a device; two threads that race both store the same address.
std::atomic<float*> g_static_work_ptr[kMaxDevices];

}  // namespace

int launch_decode_static(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    const size_t need = (size_t)c.batch * c.heads * (size_t)(c.dk + c.buf_len);
    if (need > kStaticWorkFloats) return SKETCHSSM_UNSUPPORTED_SHAPE;
    int dev = -1;
    if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    if (dev < 0 || dev >= kMaxDevices) return SKETCHSSM_UNSUPPORTED_SHAPE;
    float* work = g_static_work_ptr[dev].load(std::memory_order_acquire);
    if (work == nullptr) {
        // one-time set-up for this device (it is the current one): ask the runtime where the array lives here
        float* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_work);
        if (e != cudaSuccess || ptr == nullptr) {
            ctx->last_cuda_error = e;
            return SKETCHSSM_CUDA_ERROR;
        }
        g_static_work_ptr[dev].store(ptr, std::memory_order_release);
        work = ptr;
    }
    Params p = p_in;
    p.work = work;
    p.wstride = c.dk + c.buf_len;
    const bool bf = c.io_dtype == SKETCHSSM_BF16;
    switch (c.kind) {
        case SKETCHSSM_MAMBA2:
            return bf ? launch_decode_split_mamba2_bf16(ctx, p, stream) : launch_decode_split_mamba2_f32(ctx, p, stream);
        case SKETCHSSM_GDN:
            return bf ? launch_decode_split_gdn_bf16(ctx, p, stream) : launch_decode_split_gdn_f32(ctx, p, stream);
        default:
            return bf ? launch_decode_split_kda_bf16(ctx, p, stream) : launch_decode_split_kda_f32(ctx, p, stream);
    }
}

}  // namespace sketchssm
