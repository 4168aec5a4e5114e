// Decode step for the Mamba-2 transition with the dot products on the tensor cores (sm_100a).
//
// Mamba-2 has no erase, so the effective query is a scalar multiple of the query, q~_t = (prod_j a_j) q_t, and
// every buffer weight is an independent dot product (Eq. 4 with M_s = a_s I):
//     a_s = beta_s (prod_{s<j<=t} a_j) <k_s, q_t>,      c = (prod_j a_j) C q_t,
//     o   = sum_g c_g U[g,:] + sum_s a_s v_s.
// A warp serving one head on CUDA cores spends ~1000 instructions on this, most of them shuffles, bf16->fp32
// unpacking and shared-memory loads for matrix-vector products, and the kernel is bound by instruction issue at
// half the HBM rate.  Here the matrix-vector products [k_1 .. k_t; C] q_t run as mma.sync.m16n8k16 (bf16 inputs,
// fp32 accumulation) with the query as the only used column of the B operand: keys and queries are bf16, so the
// products are exact; the fp32 coefficient map is split once per CTA into bf16 hi + lo (two MMAs, ~16 mantissa
// bits).  That is eight times more arithmetic than needed on a pipe that is otherwise idle, and four times fewer
// instructions.  The weighted sum of rows stays on the FMA pipe (it is one FMA per loaded element).
//
// One warp per (batch, head); a CTA serves one head index for a chunk of the batch.  Each warp's operands arrive
// in its private shared-memory stage by bulk asynchronous copies (TMA, no multicast) on an mbarrier; key rows
// are copied one by one into rows padded to 272 bytes so that ldmatrix reads them without bank conflicts.
#include "internal.cuh"

namespace sketchssm {

namespace {

constexpr int kMK = 128;             // key/query channels handled by this kernel
constexpr int kRowB = 272;           // padded shared-memory row of 128 bf16 (256 B + 16 B)

struct MStage {
    uint32_t u_off, u_bytes, k_off, k_bytes, v_off, v_bytes, gate_off, gate_bytes, tq_off, tv_off, total;
};

__host__ __device__ inline MStage make_mstage(int V, int R, int L, int n) {
    MStage s;
    const uint32_t tiles = (uint32_t)(n + 1 + 15) / 16;
    uint32_t off = 0;
    s.u_off = off; s.u_bytes = (uint32_t)(R * V * 4); off += s.u_bytes;
    s.k_off = off; s.k_bytes = tiles * 16u * kRowB; off += s.k_bytes;
    s.v_off = off; s.v_bytes = (uint32_t)(n * V * 2); off += s.v_bytes;
    s.gate_off = off; s.gate_bytes = n > 0 ? (uint32_t)(2 * L * 4) : 0u; off += s.gate_bytes;
    s.tq_off = off; off += 256u;
    s.tv_off = off; off += (uint32_t)(V * 2);
    s.total = (off + 127u) & ~127u;
    return s;
}

struct MSmem {
    uint32_t coef_bytes, bar_off, scratch_off, stage_off, total;
};

__host__ __device__ inline MSmem make_msmem(int R, int nwarps, uint32_t stage_bytes) {
    MSmem d;
    const uint32_t rtiles = (uint32_t)(R + 15) / 16;
    d.coef_bytes = 2u * rtiles * 16u * kRowB;                   // C hi, C lo, padded rows
    d.bar_off = d.coef_bytes;
    uint32_t off = d.bar_off + 128u;
    d.scratch_off = off; off += (uint32_t)nwarps * 192u * 4u;   // per warp: weights a_s (64+1), coefficients c (64)
    d.stage_off = off;
    d.total = off + (uint32_t)nwarps * stage_bytes;
    return d;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

}  // namespace

template <int V>
__global__ void __launch_bounds__(256) decode_mamba2_mma_kernel(const Params p) {
    constexpr int K = kMK;
    constexpr int EV = V / 32;
    constexpr int MAXT = 4;        // up to 64 slots
    extern __shared__ __align__(128) unsigned char smem[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int R = p.R, L = p.L, H = p.H, n = p.n_before;
    const int rtiles = (R + 15) / 16;
    const int stiles = (n + 1 + 15) / 16;

    const int chunks = (p.B + p.batches_per_cta - 1) / p.batches_per_cta;
    const int h = blockIdx.x / chunks;
    const int b0 = (blockIdx.x % chunks) * p.batches_per_cta;
    const int b1 = min(p.B, b0 + p.batches_per_cta);

    const MStage sl = make_mstage(V, R, L, n);
    const MSmem ds = make_msmem(R, nwarps, sl.total);
    unsigned char* sChi = smem;
    unsigned char* sClo = smem + ds.coef_bytes / 2;
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + ds.bar_off) + warp;
    float* sWt = reinterpret_cast<float*>(smem + ds.scratch_off) + warp * 192;     // a_s at [0, 65), c_g at [128, 192)
    unsigned char* stage = smem + ds.stage_off + (size_t)warp * sl.total;

    if (threadIdx.x == 0) {
        for (int i = 0; i < nwarps; ++i) mbar_init(reinterpret_cast<uint64_t*>(smem + ds.bar_off) + i, 1);
        mbar_fence_init();
    }
    // coefficient map of this head index: fp32 -> bf16 hi + lo, rows padded to 272 bytes, unused rows zero
    {
        const float* cg = p.coef + (size_t)h * R * K;
        for (int idx = threadIdx.x; idx < rtiles * 16 * (K / 2); idx += blockDim.x) {
            const int g = idx / (K / 2), i2 = (idx % (K / 2)) * 2;
            float x0 = 0.f, x1 = 0.f;
            if (g < R) { x0 = cg[(size_t)g * K + i2]; x1 = cg[(size_t)g * K + i2 + 1]; }
            __nv_bfloat162 hi = __floats2bfloat162_rn(x0, x1);
            const uint32_t hu = *reinterpret_cast<uint32_t*>(&hi);
            __nv_bfloat162 lo = __floats2bfloat162_rn(x0 - __uint_as_float(hu << 16), x1 - __uint_as_float(hu & 0xffff0000u));
            *reinterpret_cast<uint32_t*>(sChi + (size_t)g * kRowB + i2 * 2) = hu;
            *reinterpret_cast<uint32_t*>(sClo + (size_t)g * kRowB + i2 * 2) = *reinterpret_cast<uint32_t*>(&lo);
        }
    }
    __syncthreads();

    const uint32_t tx_bytes = sl.u_bytes + (uint32_t)(n + 1) * 256u + sl.v_bytes + sl.gate_bytes + 256u + (uint32_t)(V * 2);

    auto issue = [&](int b) {   // whole warp
        const size_t bh = (size_t)b * H + h;
        const unsigned char* rh = p.ring + bh * p.rl.head_bytes;
        if (lane == 0) mbar_expect_tx(bar, tx_bytes);
        __syncwarp();
        // key rows: lane s copies ring row s (and s + 32), each into its padded row
        for (int s = lane; s < n; s += 32) bulk_g2s(stage + sl.k_off + (size_t)s * kRowB, rh + (size_t)s * 256, 256u, bar);
        if (lane == 0) {
            bulk_g2s(stage + sl.k_off + (size_t)n * kRowB, reinterpret_cast<const __nv_bfloat16*>(p.k) + bh * K, 256u, bar);
            bulk_g2s(stage + sl.u_off, p.sketch + bh * (size_t)R * V, sl.u_bytes, bar);
        } else if (lane == 1) {
            bulk_g2s(stage + sl.tq_off, reinterpret_cast<const __nv_bfloat16*>(p.q) + bh * K, 256u, bar);
            bulk_g2s(stage + sl.tv_off, reinterpret_cast<const __nv_bfloat16*>(p.v) + bh * V, (uint32_t)(V * 2), bar);
        } else if (lane == 2 && n > 0) {
            bulk_g2s(stage + sl.v_off, rh + p.rl.v_off, sl.v_bytes, bar);
            bulk_g2s(stage + sl.gate_off, rh + p.rl.beta_off, sl.gate_bytes, bar);
        }
    };

    const int first_b = b0 + warp;
    const int count = first_b < b1 ? (b1 - first_b + nwarps - 1) / nwarps : 0;
    if (count > 0) issue(first_b);

    for (int it = 0; it < count; ++it) {
        const int b = first_b + it * nwarps;
        const size_t bh = (size_t)b * H + h;
        const float bt = p.beta[bh];
        const float dct = reinterpret_cast<const float*>(p.decay)[bh];

        if (!mbar_wait_bounded(bar, (uint32_t)(it & 1))) {
            record_fault(p.status, kFaultDecodeWait, (int)blockIdx.x);
            break;
        }

        // ---- [k_1 .. k_t ; C_hi ; C_lo] q_t on the tensor cores ----
        float accS[MAXT][4], accC[MAXT][4];
#pragma unroll
        for (int t = 0; t < MAXT; ++t) {
#pragma unroll
            for (int e = 0; e < 4; ++e) { accS[t][e] = 0.f; accC[t][e] = 0.f; }
        }
        const uint32_t row_off = (uint32_t)(lane & 15) * kRowB + (uint32_t)(lane >> 4) * 16u;   // ldmatrix row address of this lane
        const uint32_t kbase = smem_u32(stage + sl.k_off) + row_off;
        const uint32_t chi = smem_u32(sChi) + row_off, clo = smem_u32(sClo) + row_off;
        const unsigned char* sq = stage + sl.tq_off;
#pragma unroll
        for (int ks = 0; ks < K / 16; ++ks) {
            // B operand: the query in column 0 (lanes 0..3 hold it), zero elsewhere
            uint32_t bq0 = 0u, bq1 = 0u;
            if (lane < 4) {
                bq0 = *reinterpret_cast<const uint32_t*>(sq + (ks * 16 + lane * 2) * 2);
                bq1 = *reinterpret_cast<const uint32_t*>(sq + (ks * 16 + 8 + lane * 2) * 2);
            }
#pragma unroll
            for (int t = 0; t < MAXT; ++t) {
                if (t < stiles) {
                    uint32_t a[4];
                    ldmatrix_x4(kbase + (uint32_t)t * 16u * kRowB + (uint32_t)ks * 32u, a);
                    mma_bf16_16816(accS[t], a, bq0, bq1);
                }
                if (t < rtiles) {
                    uint32_t a[4];
                    ldmatrix_x4(chi + (uint32_t)t * 16u * kRowB + (uint32_t)ks * 32u, a);
                    mma_bf16_16816(accC[t], a, bq0, bq1);
                    ldmatrix_x4(clo + (uint32_t)t * 16u * kRowB + (uint32_t)ks * 32u, a);
                    mma_bf16_16816(accC[t], a, bq0, bq1);
                }
            }
        }
        // column 0 of the accumulators: lanes 0, 4, .., 28 hold rows lane/4 and lane/4 + 8 of every tile
        __syncwarp();
        if ((lane & 3) == 0) {
            const int r0 = lane >> 2;
#pragma unroll
            for (int t = 0; t < MAXT; ++t) {
                if (t < stiles) { sWt[t * 16 + r0] = accS[t][0]; sWt[t * 16 + r0 + 8] = accS[t][2]; }
                if (t < rtiles) { sWt[128 + t * 16 + r0] = accC[t][0]; sWt[128 + t * 16 + r0 + 8] = accC[t][2]; }
            }
        }
        __syncwarp();

        // ---- weights: a_s = beta_s (a_t prod_{s<j<n} a_j) p_s for buffered slots, a_n = beta_t p_n ----
        const float* sBeta = reinterpret_cast<const float*>(stage + sl.gate_off);
        const float* sDec = sBeta + L;
        float dtot;
        {
            // lane l owns ring slots l and l + 32 (n <= 64).  inc = product of the decays of slots >= own slot
            // within its half (inclusive suffix scan); the exclusive suffix over (s, n) follows by one more shift.
            float inc_lo = lane < n ? sDec[lane] : 1.f;
            float inc_hi = 1.f;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float t = __shfl_down_sync(0xffffffffu, inc_lo, o);
                if (lane + o < 32) inc_lo *= t;
            }
            if (n > 32) {
                inc_hi = lane + 32 < n ? sDec[lane + 32] : 1.f;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float t = __shfl_down_sync(0xffffffffu, inc_hi, o);
                    if (lane + o < 32) inc_hi *= t;
                }
            }
            const float all_hi = __shfl_sync(0xffffffffu, inc_hi, 0);
            const float all_lo = __shfl_sync(0xffffffffu, inc_lo, 0);
            float ex_lo = __shfl_down_sync(0xffffffffu, inc_lo, 1);
            float ex_hi = __shfl_down_sync(0xffffffffu, inc_hi, 1);
            if (lane == 31) { ex_lo = 1.f; ex_hi = 1.f; }
            ex_lo *= all_hi;
            dtot = dct * all_lo * all_hi;                 // a_t times the decays of all ring slots
            if (lane < n) sWt[lane] = sBeta[lane] * (dct * ex_lo) * sWt[lane];
            if (lane + 32 < n) sWt[lane + 32] = sBeta[lane + 32] * (dct * ex_hi) * sWt[lane + 32];
            if (lane == 0) sWt[n] = bt * sWt[n];
            for (int g = lane; g < R; g += 32) sWt[128 + g] *= dtot;
        }
        __syncwarp();

        // ---- append the token to the ring (rows come from the stage) ----
        if (p.append) {
            unsigned char* rhw = p.ring + bh * p.rl.head_bytes;
            const uint2 kq = *reinterpret_cast<const uint2*>(stage + sl.k_off + (size_t)n * kRowB + lane * 8);
            *reinterpret_cast<uint2*>(rhw + (size_t)n * 256 + lane * 8) = kq;
            if (V == 128) {
                *reinterpret_cast<uint2*>(rhw + p.rl.v_off + (size_t)n * 256 + lane * 8) =
                    *reinterpret_cast<const uint2*>(stage + sl.tv_off + lane * 8);
            } else {
                *reinterpret_cast<uint32_t*>(rhw + p.rl.v_off + (size_t)n * 128 + lane * 4) =
                    *reinterpret_cast<const uint32_t*>(stage + sl.tv_off + lane * 4);
            }
            if (lane == 0) {
                reinterpret_cast<float*>(rhw + p.rl.beta_off)[n] = bt;
                reinterpret_cast<float*>(rhw + p.rl.decay_off)[n] = dct;
            }
        }

        // ---- o = sum_g c_g U[g,:] + sum_s a_s v_s + a_n v_t ----
        float o[EV];
#pragma unroll
        for (int e = 0; e < EV; ++e) o[e] = 0.f;
        const float* sU = reinterpret_cast<const float*>(stage + sl.u_off);
        const __nv_bfloat16* sV = reinterpret_cast<const __nv_bfloat16*>(stage + sl.v_off);
#pragma unroll 8
        for (int g = 0; g < R; ++g) {
            const float cg = sWt[128 + g];
            float u[EV];
            load_io<EV>(sU, g * V + lane * EV, u);
#pragma unroll
            for (int e = 0; e < EV; ++e) o[e] = fmaf(cg, u[e], o[e]);
        }
#pragma unroll 4
        for (int s = 0; s < n; ++s) {
            const float a = sWt[s];
            float vr[EV];
            load_io<EV>(sV, s * V + lane * EV, vr);
#pragma unroll
            for (int e = 0; e < EV; ++e) o[e] = fmaf(a, vr[e], o[e]);
        }
        {
            const float a = sWt[n];
            float vr[EV];
            load_io<EV>(reinterpret_cast<const __nv_bfloat16*>(stage + sl.tv_off), lane * EV, vr);
#pragma unroll
            for (int e = 0; e < EV; ++e) o[e] = fmaf(a, vr[e], o[e]);
        }
        if (p.out_bf16) store_io<EV>(reinterpret_cast<__nv_bfloat16*>(p.out) + bh * V, lane * EV, o);
        else store_io<EV>(reinterpret_cast<float*>(p.out) + bh * V, lane * EV, o);

        __syncwarp();   // every lane is done with the stage and the scratch before they are refilled
        if (it + 1 < count) issue(b + nwarps);
    }
}

// Returns SKETCHSSM_UNSUPPORTED_SHAPE outside this kernel's domain (the caller then uses the generic kernel).
int launch_decode_mma(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    if (c.kind != SKETCHSSM_MAMBA2 || c.io_dtype != SKETCHSSM_BF16 || c.dk != kMK || p_in.full_read) return SKETCHSSM_UNSUPPORTED_SHAPE;
    Params p = p_in;
    const MStage sl = make_mstage(c.dv, p.R, p.L, p.n_before);
    const uint32_t smem_budget = 227u * 1024u;
    int best_nw = 0, best_warps = 0;
    for (int nw = 8; nw >= 1; --nw) {
        if (p.warps_per_cta && nw != p.warps_per_cta) continue;
        const MSmem d = make_msmem(p.R, nw, sl.total);
        if (d.total > smem_budget) continue;
        int ctas = (int)((228u * 1024u) / (d.total + 1024u));
        if (ctas * nw > 40) ctas = 40 / nw;
        if (ctas < 1) ctas = 1;
        if (ctas * nw > best_warps) { best_warps = ctas * nw; best_nw = nw; }
    }
    if (best_nw == 0) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (p.batches_per_cta <= 0) p.batches_per_cta = best_nw * 2;
    const MSmem d = make_msmem(p.R, best_nw, sl.total);
    auto kern = c.dv == 128 ? decode_mamba2_mma_kernel<128> : decode_mamba2_mma_kernel<64>;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)d.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    const int chunks = (p.B + p.batches_per_cta - 1) / p.batches_per_cta;
    kern<<<dim3((unsigned)(p.H * chunks)), best_nw * 32, d.total, stream>>>(p);
    if ((ctx->last_cuda_error = cudaGetLastError()) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

}  // namespace sketchssm
