// Internal declarations shared by the SketchSSM CUDA translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sketchssm.h"

namespace sketchssm {

constexpr int kMaxBufLen = 64;
constexpr int kMaxRank = 64;
constexpr int kStatusInts = 4;
// device fault codes written to the status word
constexpr int kFaultDecodeWait = 1;
constexpr int kFaultFullReadWait = 2;
constexpr int kFaultUpdateWait = 3;
constexpr int kFaultProbeWait = 4;     // the self-test kernel's wait (sketchssm_selftest_wait_timeout)

struct RingLayout {
    size_t head_bytes, v_off, beta_off, decay_off;
};

struct Ctx {
    sketchssm_config cfg;
    sketchssm_buffers bufs;
    RingLayout ring;
    bool bound;
    int io_size;
    int sm_count;       // filled lazily on first launch
    int max_smem_optin; // ditto
    int last_launches;
    bool sketch_fresh;  // the last hot-path call on this context was a state update that wrote the sketch (or none was made yet)
    cudaError_t last_cuda_error;  // of the most recent failing runtime call
};

// Arguments common to the three kernels.
struct Params {
    // token inputs
    const void* q;
    const void* k;
    const void* v;
    const float* beta;
    const void* decay;
    void* out;
    // caller buffers
    float* state;
    float* sketch;
    unsigned char* ring;
    const float* omega;
    const float* coef;
    int* status;
    float* work;        // [B][H][wstride]: per-head weights handed from the decode weights kernel to the output kernel
    int wstride;        // dk + buf_len floats: [0, dk) coefficients c (or q~), [dk + s] buffer weight a_s
    RingLayout rl;
    int B, H, R, L;
    int dk, dv;
    int n_before;    // tokens already in the ring
    int has_token;   // current token given
    int append;      // store the token in the ring
    int out_bf16;
    int write_sketch;
    int write_state;
    int full_read;   // decode: read S instead of U, C
    int batches_per_cta;
    int stages;
    int warps_per_cta;   // decode: 0 = library default
    int max_warps_per_sm; // decode weights kernel: cap on resident warps per SM (0 = default)
    int update_impl;      // 0: warp-specialised tensor-core kernels where their shape limits allow, CUDA cores otherwise;
                          // 1: CUDA cores only; 3: single-group tensor-core kernel for Mamba-2, CUDA cores otherwise
    int pdl;              // launch the default decode and the tensor-core update with programmatic dependent launch
    int early_sketch;     // decode: the first head's sketch rows may be requested before the predecessor in the stream is
                          // waited for (no kernel that may still be running writes the sketch)
    int coef_per_seq;     // the coefficient map is per (batch, head) [B][H][r][K] and rebuilt by every state update
    int pivots;           // coefficient-map construction: pivot count P of the approximated state metric; 0 = exact ridge form
    float ridge_lambda;   // ridge of the state-dependent coefficient map
    const int* head_rank; // optional [H]: sketch rank per head index (0: the head reads the full state); nullptr: R for every head
    const int* n_dev;     // optional [B]: per-sequence phase of a mixed step (>= 0: decode step at that ring fill; < 0: flush with
                          // -v - 1 buffered tokens); nullptr: n_before for every sequence
    int n_cap;            // update (CUDA cores) with per-sequence phases: ring rows the shared-memory layout has room for
    int sketch_bf16;      // U (and the fixed C) are stored as bfloat16
    float* erase;         // projected erase vectors f_s [B][H][L][R] (Eq. 44-45), or nullptr: c_t = C q~_t from the swept query
    int tok_base;         // update (GDN tensor-core kernel): first ring row of this pass when a flush is replayed in blocks of 16 tokens
};

int launch_decode(Ctx* ctx, const Params& p, cudaStream_t stream);        // one warp per head
// two-kernel decode with the weight hand-off in the library's static device array
int launch_decode_static(Ctx* ctx, const Params& p, cudaStream_t stream);
// decode as two kernels (weights, then output rows), one entry per (kind, I/O type)
int launch_decode_split_mamba2_f32(Ctx* ctx, const Params& p, cudaStream_t stream);
int launch_decode_split_mamba2_bf16(Ctx* ctx, const Params& p, cudaStream_t stream);
int launch_decode_split_gdn_f32(Ctx* ctx, const Params& p, cudaStream_t stream);
int launch_decode_split_gdn_bf16(Ctx* ctx, const Params& p, cudaStream_t stream);
int launch_decode_split_kda_f32(Ctx* ctx, const Params& p, cudaStream_t stream);
int launch_decode_split_kda_bf16(Ctx* ctx, const Params& p, cudaStream_t stream);
int launch_update(Ctx* ctx, const Params& p, cudaStream_t stream);       // CUDA cores, every configuration
int launch_coef_map(Ctx* ctx, const Params& p, cudaStream_t stream);     // state-dependent coefficient maps from S_new and U (after a flush)
int launch_wait_probe(Ctx* ctx, int poll_limit, int where, cudaStream_t stream);   // self-test: a bounded wait that runs out
int launch_update_tc(Ctx* ctx, const Params& p, cudaStream_t stream);    // tcgen05 tensor cores, Mamba-2; UNSUPPORTED_SHAPE outside its domain
int launch_update_tc_ws(Ctx* ctx, const Params& p, cudaStream_t stream); // same, two warp groups per CTA (operand building overlaps the state stream)
int launch_update_tc_ws_gdn(Ctx* ctx, const Params& p, cudaStream_t stream); // gated delta rule, warp-specialised, the state read once
int launch_update_tc_ws_kda(Ctx* ctx, const Params& p, cudaStream_t stream); // delta rule with per-channel decay, warp-specialised, up to 32 tokens per pass

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__

// Launch with (or without) the programmatic-stream-serialization attribute.
template <typename Kern>
inline cudaError_t launch_kernel(Kern kern, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, const Params& p,
                                 bool pdl) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

// One potentially blocking poll of the barrier phase.  (An explicit suspend-time hint was measured: waiting warps
// then woke only when the hint ran out, which cost the kernels with few warps up to 2x, so none is given.)
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Non-blocking test of a barrier phase (for a thread that polls two barriers in turn).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Bounded wait: returns false if the barrier phase did not complete within the iteration limit.  (Sleeping between
// polls was measured too: neutral for the kernels with many warps, up to 1.7x slower for those with few.)
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit = (1u << 22)) {
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}

// 1-D bulk asynchronous copy global -> shared of this CTA (no multicast), completion on an mbarrier.
// src, dst 16-byte aligned; bytes a positive multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start while its
// predecessor in the stream is still draining; everything it does before grid_dep_wait() must not touch memory the
// predecessor may write.  Both instructions are no-ops for a normally launched kernel.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void record_fault(int* status, int code, int where) {
    if (status != nullptr) {
        if (atomicCAS(status, 0, code) == 0) status[1] = where;
    }
}

// One element of the sketch, in the configured storage type (index in elements).
__device__ __forceinline__ void store_sketch(const Params& p, size_t idx, float u) {
    if (p.sketch_bf16) reinterpret_cast<__nv_bfloat16*>(p.sketch)[idx] = __float2bfloat16_rn(u);
    else p.sketch[idx] = u;
}

// The same with the storage type fixed at compile time (for loops that branch once on p.sketch_bf16 outside).
template <bool BF>
__device__ __forceinline__ void store_sketch_as(const Params& p, size_t idx, float u) {
    if (BF) reinterpret_cast<__nv_bfloat16*>(p.sketch)[idx] = __float2bfloat16_rn(u);
    else p.sketch[idx] = u;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Load N consecutive io elements (float or bf16) starting at element index `idx` as floats.
template <int N>
__device__ __forceinline__ void load_io(const float* base, int idx, float (&dst)[N]) {
    if constexpr (N == 4) {
        float4 t = *reinterpret_cast<const float4*>(base + idx);
        dst[0] = t.x; dst[1] = t.y; dst[2] = t.z; dst[3] = t.w;
    } else if constexpr (N == 2) {
        float2 t = *reinterpret_cast<const float2*>(base + idx);
        dst[0] = t.x; dst[1] = t.y;
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) dst[i] = base[idx + i];
    }
}

template <int N>
__device__ __forceinline__ void load_io(const __nv_bfloat16* base, int idx, float (&dst)[N]) {
    if constexpr (N == 4) {
        uint2 t = *reinterpret_cast<const uint2*>(base + idx);
        __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&t.x);
        __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&t.y);
        float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
        dst[0] = fa.x; dst[1] = fa.y; dst[2] = fb.x; dst[3] = fb.y;
    } else if constexpr (N == 2) {
        __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(base + idx);
        float2 fa = __bfloat1622float2(a);
        dst[0] = fa.x; dst[1] = fa.y;
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) dst[i] = __bfloat162float(base[idx + i]);
    }
}

template <int N>
__device__ __forceinline__ void store_io(float* base, int idx, const float (&src)[N]) {
    if constexpr (N == 4) {
        *reinterpret_cast<float4*>(base + idx) = make_float4(src[0], src[1], src[2], src[3]);
    } else if constexpr (N == 2) {
        *reinterpret_cast<float2*>(base + idx) = make_float2(src[0], src[1]);
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) base[idx + i] = src[i];
    }
}

template <int N>
__device__ __forceinline__ void store_io(__nv_bfloat16* base, int idx, const float (&src)[N]) {
    if constexpr (N == 4) {
        __nv_bfloat162 a = __floats2bfloat162_rn(src[0], src[1]);
        __nv_bfloat162 b = __floats2bfloat162_rn(src[2], src[3]);
        uint2 t;
        t.x = *reinterpret_cast<uint32_t*>(&a);
        t.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(base + idx) = t;
    } else if constexpr (N == 2) {
        *reinterpret_cast<__nv_bfloat162*>(base + idx) = __floats2bfloat162_rn(src[0], src[1]);
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) base[idx + i] = __float2bfloat16_rn(src[i]);
    }
}

#endif  // __CUDACC__

}  // namespace sketchssm
