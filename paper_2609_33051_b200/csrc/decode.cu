// Decode-step kernels of the SketchSSM hot path (sm_100a).
//
// One warp owns one (batch, head) at a time.  Its per-head operands -- the sketch U and the
// buffered keys / values / gates of the ring -- are brought from HBM into a private shared-memory
// stage by 1-D bulk asynchronous copies (TMA, no multicast) that complete on an mbarrier, so the
// copies of the next head overlap the arithmetic of the current one and no register is spent on
// data in flight.  The per-head coefficient map C is shared by the whole batch: a CTA serves one
// head index h for a chunk of batch entries and stages C in shared memory once.
//
// Arithmetic per head (Algorithm 1, non-flush step; Eq. 4):
//   x <- q_t;  for s = t .. 1:  a_s = beta_s <k_s, x>;  x <- D_s (x - a_s k_s)   [Mamba-2: x <- a_s-decay * x]
//   sketch mode:    o = sum_g (C x)_g U[g,:] + sum_s a_s v_s
//   full-read mode: o = S_0^T x            + sum_s a_s v_s
#include "internal.cuh"

namespace sketchssm {

struct StageLayout {
    uint32_t u_off, u_bytes;      // sketch U (sketch mode only)
    uint32_t k_off, k_bytes;      // n buffered keys
    uint32_t v_off, v_bytes;      // n buffered values
    uint32_t gate_off, gate_bytes;  // beta[L] (+ decay[L] for scalar kinds)
    uint32_t g_off, g_bytes;      // KDA: n per-channel decays
    uint32_t total;               // stage stride, multiple of 128
};

__host__ __device__ inline StageLayout make_stage_layout(int kind, int io, int K, int V, int R, int L, int n,
                                                         int full_read) {
    StageLayout s;
    uint32_t off = 0;
    s.u_off = off; s.u_bytes = full_read ? 0u : (uint32_t)(R * V * 4); off += s.u_bytes;
    s.k_off = off; s.k_bytes = (uint32_t)(n * K * io); off += s.k_bytes;
    s.v_off = off; s.v_bytes = (uint32_t)(n * V * io); off += s.v_bytes;
    s.gate_off = off;
    s.gate_bytes = n > 0 ? (uint32_t)((kind == SKETCHSSM_KDA ? 1 : 2) * L * 4) : 0u;
    off += s.gate_bytes;
    s.g_off = off; s.g_bytes = kind == SKETCHSSM_KDA ? (uint32_t)(n * K * io) : 0u; off += s.g_bytes;
    s.total = (off + 127u) & ~127u;
    return s;
}

struct DecodeSmem {
    uint32_t coef_bytes, bar_off, x_off, stage_off, total;
};

__host__ __device__ inline DecodeSmem make_decode_smem(int K, int R, int nwarps, int stages, int full_read,
                                                       uint32_t stage_bytes) {
    DecodeSmem d;
    d.coef_bytes = full_read ? 0u : (uint32_t)(R * K * 4);
    d.bar_off = d.coef_bytes;
    uint32_t off = d.bar_off + (((uint32_t)(nwarps * stages * 8) + 127u) & ~127u);
    d.x_off = off;
    off += full_read ? (uint32_t)(nwarps * K * 4) : 0u;
    d.stage_off = off;
    d.total = off + (uint32_t)(nwarps * stages) * stage_bytes;
    return d;
}

template <int KIND, typename IO, int K, int V>
__global__ void __launch_bounds__(256) decode_kernel(const Params p) {
    constexpr int EK = K / 32;
    constexpr int EV = V / 32;
    extern __shared__ __align__(128) unsigned char smem[];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int R = p.R, L = p.L, H = p.H, n = p.n_before;
    const int stages = p.stages;

    const int chunks = (p.B + p.batches_per_cta - 1) / p.batches_per_cta;
    const int h = blockIdx.x / chunks;
    const int b0 = (blockIdx.x % chunks) * p.batches_per_cta;
    const int b1 = min(p.B, b0 + p.batches_per_cta);

    const StageLayout sl = make_stage_layout(KIND, (int)sizeof(IO), K, V, R, L, n, p.full_read);
    const DecodeSmem ds = make_decode_smem(K, R, nwarps, stages, p.full_read, sl.total);
    float* sC = reinterpret_cast<float*>(smem);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ds.bar_off) + warp * stages;
    float* sX = reinterpret_cast<float*>(smem + ds.x_off) + warp * K;
    unsigned char* my_stage = smem + ds.stage_off + (size_t)warp * stages * sl.total;

    if (threadIdx.x == 0) {
        for (int i = 0; i < nwarps * stages; ++i) mbar_init(reinterpret_cast<uint64_t*>(smem + ds.bar_off) + i, 1);
        mbar_fence_init();
    }
    if (!p.full_read) {
        const float4* src = reinterpret_cast<const float4*>(p.coef + (size_t)h * R * K);
        float4* dst = reinterpret_cast<float4*>(sC);
        for (int i = threadIdx.x; i < R * K / 4; i += blockDim.x) dst[i] = src[i];
    }
    __syncthreads();

    const uint32_t tx_bytes = sl.u_bytes + sl.k_bytes + sl.v_bytes + sl.gate_bytes + sl.g_bytes;
    const bool has_copies = tx_bytes > 0;

    auto issue = [&](int b, int st) {
        // lane 0 only
        uint64_t* bar = &bars[st];
        unsigned char* sb = my_stage + (size_t)st * sl.total;
        const size_t bh = (size_t)b * H + h;
        const unsigned char* rh = p.ring + bh * p.rl.head_bytes;
        mbar_expect_tx(bar, tx_bytes);
        if (sl.u_bytes) bulk_g2s(sb + sl.u_off, p.sketch + bh * (size_t)R * V, sl.u_bytes, bar);
        if (sl.k_bytes) {
            bulk_g2s(sb + sl.k_off, rh, sl.k_bytes, bar);
            bulk_g2s(sb + sl.v_off, rh + p.rl.v_off, sl.v_bytes, bar);
            bulk_g2s(sb + sl.gate_off, rh + p.rl.beta_off, sl.gate_bytes, bar);
            if (sl.g_bytes) bulk_g2s(sb + sl.g_off, rh + p.rl.decay_off, sl.g_bytes, bar);
        }
    };

    const int first_b = b0 + warp;
    const int count = first_b < b1 ? (b1 - first_b + nwarps - 1) / nwarps : 0;
    bool dead = false;

    if (has_copies && count > 0 && lane == 0) issue(first_b, 0);

    for (int it = 0; it < count; ++it) {
        const int b = first_b + it * nwarps;
        const int st = stages == 2 ? (it & 1) : 0;
        const uint32_t parity = stages == 2 ? ((it >> 1) & 1) : (it & 1);
        if (stages == 2 && has_copies && it + 1 < count && lane == 0) issue(b + nwarps, st ^ 1);

        const size_t bh = (size_t)b * H + h;
        const IO* qg = reinterpret_cast<const IO*>(p.q) + bh * K;
        const IO* kg = reinterpret_cast<const IO*>(p.k) + bh * K;
        const IO* vg = reinterpret_cast<const IO*>(p.v) + bh * V;

        float q0[EK], x[EK], kk[EK], gg[EK], vv[EV], o[EV];
        load_io<EK>(qg, lane * EK, q0);
        load_io<EK>(kg, lane * EK, kk);
        load_io<EV>(vg, lane * EV, vv);
        float bt = p.beta[bh];
        float dsc = 1.f;
        if constexpr (KIND == SKETCHSSM_KDA) {
            load_io<EK>(reinterpret_cast<const IO*>(p.decay) + bh * K, lane * EK, gg);
        } else {
            dsc = reinterpret_cast<const float*>(p.decay)[bh];
        }
#pragma unroll
        for (int e = 0; e < EK; ++e) x[e] = q0[e];
#pragma unroll
        for (int e = 0; e < EV; ++e) o[e] = 0.f;

        if (p.append) {
            unsigned char* rh = p.ring + bh * p.rl.head_bytes;
            store_io<EK>(reinterpret_cast<IO*>(rh) + (size_t)n * K, lane * EK, kk);
            store_io<EV>(reinterpret_cast<IO*>(rh + p.rl.v_off) + (size_t)n * V, lane * EV, vv);
            if constexpr (KIND == SKETCHSSM_KDA) {
                store_io<EK>(reinterpret_cast<IO*>(rh + p.rl.decay_off) + (size_t)n * K, lane * EK, gg);
                if (lane == 0) reinterpret_cast<float*>(rh + p.rl.beta_off)[n] = bt;
            } else {
                if (lane == 0) {
                    reinterpret_cast<float*>(rh + p.rl.beta_off)[n] = bt;
                    reinterpret_cast<float*>(rh + p.rl.decay_off)[n] = dsc;
                }
            }
        }

        // One step of the backward sweep (M_s^T applied to the running vector) for the token held in
        // (kk, vv, bt, dsc / gg).  Mamba-2 has no erase, so its running vector is dsuf * q_t.
        float dsuf = 1.f;
        auto sweep = [&]() {
            float part = 0.f;
#pragma unroll
            for (int e = 0; e < EK; ++e) part = fmaf(kk[e], x[e], part);
            const float dot = warp_sum(part);
            float a;
            if constexpr (KIND == SKETCHSSM_MAMBA2) {
                a = bt * dsuf * dot;
                dsuf *= dsc;
            } else if constexpr (KIND == SKETCHSSM_GDN) {
                a = bt * dot;
#pragma unroll
                for (int e = 0; e < EK; ++e) x[e] = dsc * fmaf(-a, kk[e], x[e]);
            } else {
                a = bt * dot;
#pragma unroll
                for (int e = 0; e < EK; ++e) x[e] = gg[e] * fmaf(-a, kk[e], x[e]);
            }
#pragma unroll
            for (int e = 0; e < EV; ++e) o[e] = fmaf(a, vv[e], o[e]);
        };
        sweep();  // the current token, s = t

        if (has_copies) {
            if (!mbar_wait_bounded(&bars[st], parity)) {
                record_fault(p.status, p.full_read ? kFaultFullReadWait : kFaultDecodeWait, (int)blockIdx.x);
                dead = true;
                break;
            }
        }
        const unsigned char* sb = my_stage + (size_t)st * sl.total;
        const IO* sK = reinterpret_cast<const IO*>(sb + sl.k_off);
        const IO* sV = reinterpret_cast<const IO*>(sb + sl.v_off);
        const float* sBeta = reinterpret_cast<const float*>(sb + sl.gate_off);
        const float* sDec = sBeta + L;
        const IO* sG = reinterpret_cast<const IO*>(sb + sl.g_off);

        for (int s = n - 1; s >= 0; --s) {
            load_io<EK>(sK, s * K + lane * EK, kk);
            load_io<EV>(sV, s * V + lane * EV, vv);
            bt = sBeta[s];
            if constexpr (KIND == SKETCHSSM_KDA) {
                load_io<EK>(sG, s * K + lane * EK, gg);
            } else {
                dsc = sDec[s];
            }
            sweep();
        }
        if constexpr (KIND == SKETCHSSM_MAMBA2) {
#pragma unroll
            for (int e = 0; e < EK; ++e) x[e] = dsuf * q0[e];
        }

        if (!p.full_read) {
            const float* sU = reinterpret_cast<const float*>(sb + sl.u_off);
#pragma unroll 4
            for (int g = 0; g < R; ++g) {
                float cw[EK], uu[EV];
                load_io<EK>(sC, g * K + lane * EK, cw);
                load_io<EV>(sU, g * V + lane * EV, uu);
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < EK; ++e) part = fmaf(cw[e], x[e], part);
                const float cg = warp_sum(part);
#pragma unroll
                for (int e = 0; e < EV; ++e) o[e] = fmaf(cg, uu[e], o[e]);
            }
        } else {
            store_io<EK>(sX, lane * EK, x);
            __syncwarp();
            const float* Sg = p.state + bh * (size_t)K * V + lane * EV;
            constexpr int RB = 8;
            for (int i0 = 0; i0 < K; i0 += RB) {
                float rows[RB][EV];
#pragma unroll
                for (int r = 0; r < RB; ++r) load_io<EV>(Sg, (i0 + r) * V, rows[r]);
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const float xi = sX[i0 + r];
#pragma unroll
                    for (int e = 0; e < EV; ++e) o[e] = fmaf(rows[r][e], xi, o[e]);
                }
            }
            __syncwarp();
        }

        if (p.out_bf16) {
            store_io<EV>(reinterpret_cast<__nv_bfloat16*>(p.out) + bh * V, lane * EV, o);
        } else {
            store_io<EV>(reinterpret_cast<float*>(p.out) + bh * V, lane * EV, o);
        }

        __syncwarp();  // every lane is done reading this stage before it is refilled
        if (stages == 1 && has_copies && it + 1 < count && lane == 0) issue(b + nwarps, 0);
    }

    if (dead && stages == 2 && has_copies) {
        // give the other stage's copies a bounded chance to land before the CTA retires
        mbar_wait_bounded(&bars[0], 0, 1u << 16);
        mbar_wait_bounded(&bars[1], 0, 1u << 16);
    }
}

template <int KIND, typename IO, int K, int V>
static int launch_decode_t(Ctx* ctx, Params p, cudaStream_t stream) {
    const int io = (int)sizeof(IO);
    const StageLayout sl = make_stage_layout(KIND, io, K, V, p.R, p.L, p.n_before, p.full_read);
    const size_t smem_budget = 227u * 1024u;
    // choose warps per CTA and stage count: as many resident warps per SM as shared memory allows
    int best_nw = 1, best_stages = 1, best_warps = 0;
    const int stage_opts[2] = {1, 2};
    for (int si = 0; si < 2; ++si) {
        for (int nw = 8; nw >= 1; --nw) {
            const DecodeSmem d = make_decode_smem(K, p.R, nw, stage_opts[si], p.full_read, sl.total);
            if (d.total > smem_budget) continue;
            int ctas = (int)(smem_budget / (d.total + 1024u));
            if (ctas < 1) ctas = 1;
            if (ctas * nw > 48) ctas = 48 / nw;   // 48 warps is plenty; keeps register pressure irrelevant
            if (ctas > 32) ctas = 32;
            const int warps = ctas * nw;
            // prefer more resident warps; at equal warps prefer a single stage with more CTAs
            if (warps > best_warps) { best_warps = warps; best_nw = nw; best_stages = stage_opts[si]; }
        }
    }
    if (p.stages == 1 || p.stages == 2) {
        // explicit request: re-pick the warp count for that stage count
        best_warps = 0;
        for (int nw = 8; nw >= 1; --nw) {
            const DecodeSmem d = make_decode_smem(K, p.R, nw, p.stages, p.full_read, sl.total);
            if (d.total > smem_budget) continue;
            int ctas = (int)(smem_budget / (d.total + 1024u));
            if (ctas < 1) ctas = 1;
            if (ctas * nw > 48) ctas = 48 / nw;
            const int warps = ctas * nw;
            if (warps > best_warps) { best_warps = warps; best_nw = nw; }
        }
        best_stages = p.stages;
    }
    if (best_warps == 0) return SKETCHSSM_UNSUPPORTED_SHAPE;
    p.stages = best_stages;
    if (p.batches_per_cta <= 0) p.batches_per_cta = best_nw * 2;
    const DecodeSmem d = make_decode_smem(K, p.R, best_nw, best_stages, p.full_read, sl.total);
    auto kern = decode_kernel<KIND, IO, K, V>;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)d.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    const int chunks = (p.B + p.batches_per_cta - 1) / p.batches_per_cta;
    const dim3 grid((unsigned)(p.H * chunks));
    kern<<<grid, best_nw * 32, d.total, stream>>>(p);
    if ((ctx->last_cuda_error = cudaGetLastError()) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

template <int KIND, typename IO>
static int launch_decode_shape(Ctx* ctx, const Params& p, cudaStream_t stream) {
    const int K = ctx->cfg.dk, V = ctx->cfg.dv;
    if (K == 128 && V == 128) return launch_decode_t<KIND, IO, 128, 128>(ctx, p, stream);
    if (K == 128 && V == 64) return launch_decode_t<KIND, IO, 128, 64>(ctx, p, stream);
    if (K == 64 && V == 64) return launch_decode_t<KIND, IO, 64, 64>(ctx, p, stream);
    if (K == 64 && V == 128) return launch_decode_t<KIND, IO, 64, 128>(ctx, p, stream);
    return SKETCHSSM_UNSUPPORTED_SHAPE;
}

template <int KIND>
static int launch_decode_io(Ctx* ctx, const Params& p, cudaStream_t stream) {
    if (ctx->cfg.io_dtype == SKETCHSSM_BF16) return launch_decode_shape<KIND, __nv_bfloat16>(ctx, p, stream);
    return launch_decode_shape<KIND, float>(ctx, p, stream);
}

int launch_decode(Ctx* ctx, const Params& p, cudaStream_t stream) {
    switch (ctx->cfg.kind) {
        case SKETCHSSM_MAMBA2: return launch_decode_io<SKETCHSSM_MAMBA2>(ctx, p, stream);
        case SKETCHSSM_GDN: return launch_decode_io<SKETCHSSM_GDN>(ctx, p, stream);
        case SKETCHSSM_KDA: return launch_decode_io<SKETCHSSM_KDA>(ctx, p, stream);
    }
    return SKETCHSSM_INVALID_ARG;
}

}  // namespace sketchssm
