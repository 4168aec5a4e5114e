// State-update (flush) kernel of the SketchSSM hot path (sm_100a), CUDA-core version.
//
// Every V-column of S is an independent K-vector recurrence under all three transitions: the erase
// dot <k_s, S[:, j]> touches one column only.  A CTA owns a tile of VT = 64 columns of one (b, h)
// state; a column lives in the registers of 4 threads (K/4 rows each), so the whole tile is read
// from HBM once, replayed on chip, projected onto Omega for the sketch rows U[g, j] = <S[:, j], omega_g>
// and onto q for the exact output, and written back once (Algorithm 1, flush step; Eq. 3 and Eq. 7).
//
//   delta rule (GDN, KDA), token by token:  col <- D_s col;  e = beta_s (v_s[j] - <k_s, col>);  col += e k_s
//   Mamba-2, closed form of Eq. 3:          col <- d col + sum_s (beta_s prod_{j>s} a_j) v_s[j] k_s
#include "internal.cuh"

namespace sketchssm {

constexpr int kParts = 4;               // threads per column; a CTA owns VT = 64 columns (80 when V = 80) of one head

// shared-memory row of K floats split into kParts parts, each padded by 4 floats so that the four
// parts of a warp read from different banks with 128-bit loads
template <int K>
struct PaddedRow {
    static constexpr int RP = K / kParts;
    static constexpr int stride = K + 4 * kParts;
    __host__ __device__ static constexpr int at(int i) { return i + 4 * (i / RP); }
};

// Packed pairs of fp32 (sm_100: one instruction for two independent IEEE operations): the replay loops are bound by
// instruction issue, and a column's rows are independent.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 r, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

struct UpdateSmem {
    uint32_t k_off, g_off, v_off, beta_off, dec_off, q_off, om_off, total;
};

template <int K>
__host__ __device__ inline UpdateSmem make_update_smem(int kind, int n_tot, int R4, int kVT) {
    UpdateSmem u;
    const int ntok = n_tot > 0 ? n_tot : 1;
    uint32_t off = 0;
    u.k_off = off; off += (uint32_t)(ntok * PaddedRow<K>::stride * 4);
    u.g_off = off; off += kind == SKETCHSSM_KDA ? (uint32_t)(ntok * PaddedRow<K>::stride * 4) : 0u;
    u.v_off = off; off += (uint32_t)(ntok * kVT * 4);
    u.beta_off = off; off += (uint32_t)(((ntok + 3) & ~3) * 4);
    u.dec_off = off; off += (uint32_t)(((ntok + 3) & ~3) * 4);
    u.q_off = off; off += (uint32_t)(PaddedRow<K>::stride * 4);
    u.om_off = off; off += (uint32_t)(kParts * ((K / kParts) * R4 + 4) * 4);
    u.total = off;
    return u;
}

template <int KIND, typename IO, int K, int kVT>
__global__ void __launch_bounds__(kVT * kParts) update_kernel(const Params p) {
    constexpr int kUpdThreads = kVT * kParts;
    using PR = PaddedRow<K>;
    constexpr int RP = PR::RP;
    extern __shared__ __align__(128) unsigned char smem[];

    const int V = p.dv;
    const int R = p.R, H = p.H;
    const int R4 = (R + 3) & ~3;
    const int vtiles = V / kVT;
    const int bh = blockIdx.x / vtiles;
    const int v0 = (blockIdx.x % vtiles) * kVT;
    const int b = bh / H, h = bh % H;
    // ring fill: the call's n_before, or with per-sequence phases the sequence's own (a sequence whose phase says
    // "decode step" is left alone by this kernel)
    int n_ring = p.n_before;
    if (p.n_dev != nullptr) {
        const int ph = p.n_dev[b];
        if (ph >= 0) return;
        n_ring = -ph - 1;
    }
    const int n_tot = n_ring + (p.has_token ? 1 : 0);

    const UpdateSmem us = make_update_smem<K>(KIND, p.n_dev != nullptr ? p.n_cap : n_tot, R4, kVT);
    float* sK = reinterpret_cast<float*>(smem + us.k_off);
    float* sG = reinterpret_cast<float*>(smem + us.g_off);
    float* sV = reinterpret_cast<float*>(smem + us.v_off);
    float* sBeta = reinterpret_cast<float*>(smem + us.beta_off);
    float* sDec = reinterpret_cast<float*>(smem + us.dec_off);
    float* sQ = reinterpret_cast<float*>(smem + us.q_off);
    float* sOm = reinterpret_cast<float*>(smem + us.om_off);

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int part = lane >> 3;                    // 0..3: which quarter of the rows
    const int j = v0 + warp * 8 + (lane & 7);      // this thread's column
    const int jl = j - v0;

    // ---- state tile -> registers (issued first: the long-latency stream) ----
    float col[RP];
    const float* Sg = p.state + (size_t)bh * K * V + (size_t)(part * RP) * V + j;
#pragma unroll
    for (int ii = 0; ii < RP; ++ii) col[ii] = Sg[(size_t)ii * V];

    // ---- ring + current token -> shared memory (fp32) ----
    const unsigned char* rh = p.ring + (size_t)bh * p.rl.head_bytes;
    const IO* rk = reinterpret_cast<const IO*>(rh);
    const IO* rv = reinterpret_cast<const IO*>(rh + p.rl.v_off);
    const float* rbeta = reinterpret_cast<const float*>(rh + p.rl.beta_off);
    for (int idx = tid; idx < n_tot * K; idx += kUpdThreads) {
        const int s = idx / K, i = idx % K;
        float kv, gv = 1.f;
        if (s < n_ring) {
            kv = static_cast<float>(rk[(size_t)s * K + i]);
            if constexpr (KIND == SKETCHSSM_KDA)
                gv = static_cast<float>(reinterpret_cast<const IO*>(rh + p.rl.decay_off)[(size_t)s * K + i]);
        } else {
            kv = static_cast<float>(reinterpret_cast<const IO*>(p.k)[(size_t)bh * K + i]);
            if constexpr (KIND == SKETCHSSM_KDA)
                gv = static_cast<float>(reinterpret_cast<const IO*>(p.decay)[(size_t)bh * K + i]);
        }
        sK[s * PR::stride + PR::at(i)] = kv;
        if constexpr (KIND == SKETCHSSM_KDA) sG[s * PR::stride + PR::at(i)] = gv;
    }
    for (int idx = tid; idx < n_tot * kVT; idx += kUpdThreads) {
        const int s = idx / kVT, c = idx % kVT;
        sV[idx] = s < n_ring ? static_cast<float>(rv[(size_t)s * V + v0 + c])
                             : static_cast<float>(reinterpret_cast<const IO*>(p.v)[(size_t)bh * V + v0 + c]);
    }
    if (tid < n_tot) {
        const int s = tid;
        sBeta[s] = s < n_ring ? rbeta[s] : p.beta[bh];
        if constexpr (KIND != SKETCHSSM_KDA) {
            sDec[s] = s < n_ring ? reinterpret_cast<const float*>(rh + p.rl.decay_off)[s]
                                 : reinterpret_cast<const float*>(p.decay)[bh];
        }
    }
    if (p.q != nullptr) {
        for (int i = tid; i < K; i += kUpdThreads)
            sQ[PR::at(i)] = static_cast<float>(reinterpret_cast<const IO*>(p.q)[(size_t)bh * K + i]);
    }
    if (p.write_sketch) {
        const float* og = p.omega + (size_t)h * K * R;
        for (int idx = tid; idx < K * R4; idx += kUpdThreads) {
            const int i = idx / R4, g = idx % R4;
            sOm[(i / RP) * (RP * R4 + 4) + (i % RP) * R4 + g] = g < R ? og[(size_t)i * R + g] : 0.f;
        }
    }
    __syncthreads();

    if constexpr (KIND == SKETCHSSM_MAMBA2) {
        // sBeta[s] <- beta_s * prod_{j>s} a_j ;  total decay d = prod_j a_j
        __shared__ float s_total;
        if (tid == 0) {
            float suf = 1.f;
            for (int s = n_tot - 1; s >= 0; --s) {
                sBeta[s] *= suf;
                suf *= sDec[s];
            }
            s_total = suf;
        }
        __syncthreads();
        if (n_tot > 0) {
            const float d = s_total;
            f32x2 c2[RP / 2];
#pragma unroll
            for (int i2 = 0; i2 < RP / 2; ++i2) c2[i2] = pack2(col[2 * i2] * d, col[2 * i2 + 1] * d);
            for (int s = 0; s < n_tot; ++s) {
                const float w = sBeta[s] * sV[s * kVT + jl];
                const f32x2 w2 = pack2(w, w);
                const float4* kp = reinterpret_cast<const float4*>(sK + s * PR::stride + part * (RP + 4));
#pragma unroll
                for (int i4 = 0; i4 < RP / 4; ++i4) {
                    const float4 kq = kp[i4];
                    c2[2 * i4] = fma2(pack2(kq.x, kq.y), w2, c2[2 * i4]);
                    c2[2 * i4 + 1] = fma2(pack2(kq.z, kq.w), w2, c2[2 * i4 + 1]);
                }
            }
#pragma unroll
            for (int i2 = 0; i2 < RP / 2; ++i2) unpack2(c2[i2], col[2 * i2], col[2 * i2 + 1]);
        }
    } else {
        f32x2 c2[RP / 2];
#pragma unroll
        for (int i2 = 0; i2 < RP / 2; ++i2) c2[i2] = pack2(col[2 * i2], col[2 * i2 + 1]);
        for (int s = 0; s < n_tot; ++s) {
            const float4* kp = reinterpret_cast<const float4*>(sK + s * PR::stride + part * (RP + 4));
            f32x2 k2[RP / 2];
#pragma unroll
            for (int i4 = 0; i4 < RP / 4; ++i4) {
                const float4 kq = kp[i4];
                k2[2 * i4] = pack2(kq.x, kq.y);
                k2[2 * i4 + 1] = pack2(kq.z, kq.w);
            }
            f32x2 dot01 = pack2(0.f, 0.f), dot23 = dot01;
            if constexpr (KIND == SKETCHSSM_GDN) {
                const float a = sDec[s];
                const f32x2 a2 = pack2(a, a);
#pragma unroll
                for (int i4 = 0; i4 < RP / 4; ++i4) {
                    c2[2 * i4] = mul2(c2[2 * i4], a2);
                    c2[2 * i4 + 1] = mul2(c2[2 * i4 + 1], a2);
                    dot01 = fma2(k2[2 * i4], c2[2 * i4], dot01);
                    dot23 = fma2(k2[2 * i4 + 1], c2[2 * i4 + 1], dot23);
                }
            } else {
                const float4* gp = reinterpret_cast<const float4*>(sG + s * PR::stride + part * (RP + 4));
#pragma unroll
                for (int i4 = 0; i4 < RP / 4; ++i4) {
                    const float4 gq = gp[i4];
                    c2[2 * i4] = mul2(c2[2 * i4], pack2(gq.x, gq.y));
                    c2[2 * i4 + 1] = mul2(c2[2 * i4 + 1], pack2(gq.z, gq.w));
                    dot01 = fma2(k2[2 * i4], c2[2 * i4], dot01);
                    dot23 = fma2(k2[2 * i4 + 1], c2[2 * i4 + 1], dot23);
                }
            }
            float d0, d1, d2, d3;
            unpack2(dot01, d0, d1);
            unpack2(dot23, d2, d3);
            float dot = (d0 + d2) + (d1 + d3);
            dot += __shfl_xor_sync(0xffffffffu, dot, 8);
            dot += __shfl_xor_sync(0xffffffffu, dot, 16);
            const float e = sBeta[s] * (sV[s * kVT + jl] - dot);
            const f32x2 e2 = pack2(e, e);
#pragma unroll
            for (int i2 = 0; i2 < RP / 2; ++i2) c2[i2] = fma2(k2[i2], e2, c2[i2]);
        }
#pragma unroll
        for (int i2 = 0; i2 < RP / 2; ++i2) unpack2(c2[i2], col[2 * i2], col[2 * i2 + 1]);
    }

    // ---- write the updated tile back ----
    if (p.write_state && n_tot > 0) {
        float* So = p.state + (size_t)bh * K * V + (size_t)(part * RP) * V + j;
#pragma unroll
        for (int ii = 0; ii < RP; ++ii) So[(size_t)ii * V] = col[ii];
    }

    // ---- exact output o[j] = <S_new[:, j], q> ----
    if (p.out != nullptr) {
        const float4* qp = reinterpret_cast<const float4*>(sQ + part * (RP + 4));
        float acc = 0.f;
#pragma unroll
        for (int i4 = 0; i4 < RP / 4; ++i4) {
            const float4 qq = qp[i4];
            acc = fmaf(qq.x, col[4 * i4 + 0], acc);
            acc = fmaf(qq.y, col[4 * i4 + 1], acc);
            acc = fmaf(qq.z, col[4 * i4 + 2], acc);
            acc = fmaf(qq.w, col[4 * i4 + 3], acc);
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 8);
        acc += __shfl_xor_sync(0xffffffffu, acc, 16);
        if (part == 0) {
            if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[(size_t)bh * V + j] = __float2bfloat16_rn(acc);
            else reinterpret_cast<float*>(p.out)[(size_t)bh * V + j] = acc;
        }
    }

    // ---- sketch rows U[g, j] = <S_new[:, j], omega_g>, 4 ranks at a time ----
    if (p.write_sketch) {
        const size_t ug = (size_t)bh * R * V + j;
        for (int g0 = 0; g0 < R4; g0 += 4) {
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            const float* op = sOm + (size_t)part * (RP * R4 + 4) + g0;
#pragma unroll
            for (int ii = 0; ii < RP; ++ii) {
                const float4 w = *reinterpret_cast<const float4*>(op + ii * R4);
                a0 = fmaf(w.x, col[ii], a0);
                a1 = fmaf(w.y, col[ii], a1);
                a2 = fmaf(w.z, col[ii], a2);
                a3 = fmaf(w.w, col[ii], a3);
            }
            a0 += __shfl_xor_sync(0xffffffffu, a0, 8);  a0 += __shfl_xor_sync(0xffffffffu, a0, 16);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 8);  a1 += __shfl_xor_sync(0xffffffffu, a1, 16);
            a2 += __shfl_xor_sync(0xffffffffu, a2, 8);  a2 += __shfl_xor_sync(0xffffffffu, a2, 16);
            a3 += __shfl_xor_sync(0xffffffffu, a3, 8);  a3 += __shfl_xor_sync(0xffffffffu, a3, 16);
            // part p stores rank g0 + p
            const float mine = part == 0 ? a0 : part == 1 ? a1 : part == 2 ? a2 : a3;
            if (g0 + part < R) store_sketch(p, ug + (size_t)(g0 + part) * V, mine);
        }
    }
}

template <int KIND, typename IO, int K, int kVT>
static int launch_update_t(Ctx* ctx, Params p, cudaStream_t stream) {
    constexpr int kUpdThreads = kVT * kParts;
    const int V = ctx->cfg.dv;
    const int n_tot = p.n_before + (p.has_token ? 1 : 0);
    const int R4 = (p.R + 3) & ~3;
    if (p.n_dev != nullptr) p.n_cap = n_tot;        // per-sequence phases: n_before is the largest fill any sequence may have
    const UpdateSmem us = make_update_smem<K>(KIND, n_tot, R4, kVT);
    auto kern = update_kernel<KIND, IO, K, kVT>;
    if (us.total > 226u * 1024u) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)us.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    p.dv = V;
    const dim3 grid((unsigned)((size_t)p.B * p.H * (V / kVT)));
    kern<<<grid, kUpdThreads, us.total, stream>>>(p);
    if ((ctx->last_cuda_error = cudaGetLastError()) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

template <int KIND, typename IO>
static int launch_update_shape(Ctx* ctx, const Params& p, cudaStream_t stream) {
    if (ctx->cfg.dk == 128 && ctx->cfg.dv == 80) return launch_update_t<KIND, IO, 128, 80>(ctx, p, stream);
    if (ctx->cfg.dv % 64 != 0) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (ctx->cfg.dk == 128) return launch_update_t<KIND, IO, 128, 64>(ctx, p, stream);
    if (ctx->cfg.dk == 64) return launch_update_t<KIND, IO, 64, 64>(ctx, p, stream);
    return SKETCHSSM_UNSUPPORTED_SHAPE;
}

template <int KIND>
static int launch_update_io(Ctx* ctx, const Params& p, cudaStream_t stream) {
    if (ctx->cfg.io_dtype == SKETCHSSM_BF16) return launch_update_shape<KIND, __nv_bfloat16>(ctx, p, stream);
    return launch_update_shape<KIND, float>(ctx, p, stream);
}

int launch_update(Ctx* ctx, const Params& p, cudaStream_t stream) {
    switch (ctx->cfg.kind) {
        case SKETCHSSM_MAMBA2: return launch_update_io<SKETCHSSM_MAMBA2>(ctx, p, stream);
        case SKETCHSSM_GDN: return launch_update_io<SKETCHSSM_GDN>(ctx, p, stream);
        case SKETCHSSM_KDA: return launch_update_io<SKETCHSSM_KDA>(ctx, p, stream);
    }
    return SKETCHSSM_INVALID_ARG;
}

}  // namespace sketchssm
