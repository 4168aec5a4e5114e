// State-dependent coefficient map, rebuilt at every flush (Section 4.1, Eq. 9; Appendix A.2.2, Eq. 26-37).
//
// After a state update has written S_new and the sketch U = S_new^T Omega (rows U_g = S_new^T omega_g), the map
// C in R^{G x K} with c_t = C q~_t is, for an orthonormal Omega and with mu = ||S||_F^2 / K (1 for a zero state),
//
//   exact ridge form       C = (U^T U + lam mu I)^{-1} U^T S^T
//   pivot approximation    p = min(G, P);  Q = Gram-Schmidt basis of U_1 .. U_p (value space, V x p)
//                          L = S Q / sqrt(mu) (K x p; never formed in rotated coordinates: only L_G = U^T Q / sqrt(mu),
//                          L^T x = Q^T S^T q~ / sqrt(mu) and the first G residual diagonals are needed)
//                          d_g = max((||U_g||^2 - ||Q^T U_g||^2) / mu, 0),  D_G = Diag(d) + lam I
//                          C = (D_G + L_G L_G^T)^{-1} [ L_G Q^T S^T / sqrt(mu) + Diag(d) Omega^T ]
//                          with the inverse through the p x p Woodbury system T_P = I + L_G^T D_G^{-1} L_G.
// Both follow from the paper's basis-aligned statement by carrying the orthogonal change of coordinates R through
// (J^T R = Omega^T, J^T H R = U^T S^T / mu, J^T H J = U^T U / mu); R itself is never needed.
//
// One CTA of 128 threads per (batch, head).  The probe rows (Q_j, or the U_g themselves for the exact form) sit in
// shared memory.  Pivot form: a warp reads whole rows of S (lanes along the value index, every fetched sector used
// once) and the 32 partial products of a block of rows x probes are reduced by one transposing butterfly, giving
// Y[k][j] = <S[k,:], Q_j> and ||S||_F^2; the p x p system is built one entry per thread and inverted by one warp;
// thread k then forms column k of C with the pivot loops unrolled in registers and Omega staged in shared memory
// (stores coalesced across the CTA).  Exact form: thread k streams row k of S against all G sketch rows, Cholesky by
// one warp, one pair of triangular solves per thread.  The kernel runs after the flush kernel of the same call and
// re-reads S_new and U from memory: the map needs the complete sketch before it can contract the state with it.
#include "internal.cuh"
#include "lanegroup.cuh"

namespace sketchssm {

namespace {

constexpr int kCoefThreads = 128;
constexpr int kMaxPivots = 8;

struct CoefSmem {
    uint32_t probe, y, ru, small, om, total;   // byte offsets
    int pitch;                                 // floats per probe row
};

__host__ __device__ inline CoefSmem make_coef_smem(int K, int V, int G, int m) {
    CoefSmem s;
    s.pitch = V + 4;                                          // rows staggered across banks, still 16-byte aligned
    uint32_t off = 0;
    s.probe = off; off += (uint32_t)(G * s.pitch * 4);        // the G sketch rows; the first m become the probe rows
    const int yf = K * (m + 1) > m * V ? K * (m + 1) : m * V;
    s.y = off; off += (uint32_t)(yf * 4);                     // Y[k][0..m) (pitch m + 1); before that, the m raw pivot rows
    s.ru = off; off += (uint32_t)(G * (m + 1 > 8 ? m + 1 : 8) * 4);   // RU[g][j] = <U_g, probe_j> (pitch m + 1 for the exact form, else the padded pivot count)
    s.small = off; off += (uint32_t)((4 * G + 2 * 8 * 8 + 64) * 4);
    s.om = off; off += (uint32_t)(K * (G | 1) * 4);           // Omega of the head index, odd pitch (a thread reads its own row)
    s.total = (off + 15u) & ~15u;
    return s;
}

__device__ __forceinline__ float block_sum(float x, float* scratch) {
    x = warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = x;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += scratch[i];
    return t;
}

}  // namespace

// EXACT = 0: pivot approximation with m = min(G, P) <= PM probe rows (PM = 4 or 8: loops over pivots unroll and stay in
// registers);  EXACT = 1: ridge form with m = G.
template <int K, int V, int EXACT, int PM>
__global__ void __launch_bounds__(kCoefThreads) coef_map_kernel(const Params p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t bh = blockIdx.x;
    const int h = (int)(bh % (size_t)p.H);
    // sketch rank of this head: the configured rank or the caller's per-head table (0: the head reads the full state and has
    // no map); with per-sequence phases only the sequences that were just flushed get a new map
    int G = p.R;
    if (p.head_rank != nullptr) {
        const int r = p.head_rank[h];
        G = r < 0 ? 0 : (r > p.R ? p.R : r);
    }
    if (G == 0) return;
    if (p.n_dev != nullptr && p.n_dev[bh / (size_t)p.H] >= 0) return;
    const int m = EXACT ? G : min(G, p.pivots);
    const CoefSmem sm = make_coef_smem(K, V, p.R, EXACT ? p.R : min(p.R, p.pivots));
    float* sU = reinterpret_cast<float*>(smem + sm.probe);
    float* sY = reinterpret_cast<float*>(smem + sm.y);
    float* sRU = reinterpret_cast<float*>(smem + sm.ru);
    float* sSm = reinterpret_cast<float*>(smem + sm.small);
    float* sUU = sSm;                  // [G] ||U_g||^2, then d_g
    float* sD = sSm + G;               // [G] 1 / D_G
    float* sT = sSm + 2 * G;           // [PM][2 PM] T_P next to the identity, inverted in place (pivot) -- the exact form keeps its Cholesky factor in sRU
    float* sRed = sSm + 2 * G + 2 * 8 * 8; // block reduction scratch
    const int PT = sm.pitch, MP = m + 1;   // MP: pitch of Y (odd or small: the per-row accesses of a warp spread over the banks)
    constexpr int RUP = PM;                // pitch of RU in the pivot form (16- or 32-byte rows, zero beyond m)

    const int RS = p.R;                // row strides of U, C and Omega follow the configured rank
    const float* Ug = p.sketch + bh * (size_t)RS * V;                  // (fp32 storage)
    const float* Sg = p.state + bh * (size_t)K * V;
    // the map is stored like the sketch: fp32, or rounded to bfloat16 once, here
    float* Cg = const_cast<float*>(p.coef) + bh * (size_t)RS * K;
    __nv_bfloat16* Cg16 = reinterpret_cast<__nv_bfloat16*>(const_cast<float*>(p.coef)) + bh * (size_t)RS * K;
    const bool bf = p.sketch_bf16 != 0;
    auto store_c = [&](size_t idx, float x) {
        if (bf) Cg16[idx] = __float2bfloat16_rn(x);
        else Cg[idx] = x;
    };
    const float* Om = p.omega + (size_t)h * K * RS;

    // ---- sketch rows into shared memory ----
    // (with bfloat16 storage the map is built from the sketch as stored, i.e. from the rounded rows)
    if (bf) {
        const uint2* Ug16 = reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(p.sketch) + bh * (size_t)RS * V);
        for (int i = tid; i < G * V / 4; i += kCoefThreads) {
            const int g = i / (V / 4), c = i - g * (V / 4);
            const uint2 t = Ug16[(size_t)g * (V / 4) + c];
            *reinterpret_cast<float4*>(sU + g * PT + 4 * c) =
                make_float4(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u),
                            __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u));
        }
    } else {
        for (int i = tid; i < G * V / 4; i += kCoefThreads) {
            const int g = i / (V / 4), c = i - g * (V / 4);
            *reinterpret_cast<float4*>(sU + g * PT + 4 * c) = *reinterpret_cast<const float4*>(Ug + (size_t)g * V + 4 * c);
        }
    }
    __syncthreads();
    // ||U_g||^2, one row per thread
    for (int g = tid; g < G; g += kCoefThreads) {
        float a = 0.f;
        for (int v = 0; v < V; ++v) a = fmaf(sU[g * PT + v], sU[g * PT + v], a);
        sUU[g] = a;
    }
    if (!EXACT) {
        // ---- Gram-Schmidt on the first m sketch rows, in place, by warp 0 (two sweeps; a row that lies in the span of
        // its predecessors becomes zero) ----
        if (warp == 0) {
            constexpr int EV = (V + 31) / 32;          // elements per lane; beyond V (V = 80) they are zero and never stored
            auto on = [&](int e) { return V % 32 == 0 || lane + 32 * e < V; };
            for (int j = 0; j < m; ++j) {
                float u[EV], ref = 0.f;
#pragma unroll
                for (int e = 0; e < EV; ++e) { u[e] = on(e) ? sU[j * PT + lane + 32 * e] : 0.f; ref = fmaf(u[e], u[e], ref); }
                ref = warp_sum(ref);
                for (int sweep = 0; sweep < 2; ++sweep) {
                    for (int i = 0; i < j; ++i) {
                        float d = 0.f;
#pragma unroll
                        for (int e = 0; e < EV; ++e) d = fmaf(on(e) ? sU[i * PT + lane + 32 * e] : 0.f, u[e], d);
                        d = warp_sum(d);
#pragma unroll
                        for (int e = 0; e < EV; ++e) u[e] = fmaf(-d, on(e) ? sU[i * PT + lane + 32 * e] : 0.f, u[e]);
                    }
                }
                float nn = 0.f;
#pragma unroll
                for (int e = 0; e < EV; ++e) nn = fmaf(u[e], u[e], nn);
                nn = warp_sum(nn);
                const float inv = (ref > 0.f && nn > 1e-12f * ref) ? rsqrtf(nn) : 0.f;
                __syncwarp();
                // the raw row is still needed for <U_j, Q_i> below: park it in the (not yet used) Y area
#pragma unroll
                for (int e = 0; e < EV; ++e) if (on(e)) sY[j * V + lane + 32 * e] = sU[j * PT + lane + 32 * e];
                __syncwarp();
#pragma unroll
                for (int e = 0; e < EV; ++e) if (on(e)) sU[j * PT + lane + 32 * e] = u[e] * inv;
                __syncwarp();
            }
        }
        __syncthreads();
        // RU[g][j] = <U_g, Q_j>; the raw rows g < m were parked in the Y area
        for (int i = tid; i < G * RUP; i += kCoefThreads) {
            const int g = i / RUP, j = i - g * RUP;
            float a = 0.f;
            if (j < m) {
                const float* ur = g < m ? sY + g * V : sU + g * PT;
                for (int v = 0; v < V; ++v) a = fmaf(ur[v], sU[j * PT + v], a);
            }
            sRU[g * RUP + j] = a;
        }
        __syncthreads();
    } else {
        // Gram matrix U^T U (G x G), lower triangle, into sRU (pitch m + 1 = G + 1)
        for (int i = tid; i < G * G; i += kCoefThreads) {
            const int g = i / G, j = i - g * G;
            if (j <= g) {
                float a = 0.f;
                for (int v = 0; v < V; ++v) a = fmaf(sU[g * PT + v], sU[j * PT + v], a);
                sRU[g * MP + j] = a;
            }
        }
        __syncthreads();
    }

    // ---- stream the state: Y[k][j] = <S[k,:], probe_j>, ||S||_F^2 ----
    float ss = 0.f;
    if constexpr (!EXACT) {
        // A warp reads whole rows (lanes along the value index: every fetched sector is used once); the 32 partial dot
        // products of a block of rows (32 / PM rows x PM probes) are reduced over the lanes by one transposing butterfly.
        constexpr int EV = V % 32 == 0 ? V / 32 : 4;
        constexpr int VL = V / EV;
        constexpr int RB = 32 / PM;                 // rows per block
        const bool vlane = VL == 32 || lane < VL;
        float qf[PM][EV];
#pragma unroll
        for (int j = 0; j < PM; ++j)
#pragma unroll
            for (int e = 0; e < EV; ++e) qf[j][e] = (j < m && vlane) ? sU[j * PT + lane * EV + e] : 0.f;
        constexpr int RPW = K / (kCoefThreads / 32);        // rows per warp
        for (int k0 = warp * RPW; k0 < (warp + 1) * RPW; k0 += RB) {
            float part[32];
#pragma unroll
            for (int r = 0; r < RB; ++r) {
                float sv[EV];
#pragma unroll
                for (int e = 0; e < EV; ++e) sv[e] = 0.f;
                if (vlane) load_io<EV>(Sg, (k0 + r) * V + lane * EV, sv);
#pragma unroll
                for (int e = 0; e < EV; ++e) ss = fmaf(sv[e], sv[e], ss);
#pragma unroll
                for (int j = 0; j < PM; ++j) {
                    float a = 0.f;
#pragma unroll
                    for (int e = 0; e < EV; ++e) a = fmaf(sv[e], qf[j][e], a);
                    part[r * PM + j] = a;
                }
            }
            group_reduce_transpose<32, 32>(part, lane);
            const int r = lane / PM, j = lane - r * PM;      // lane l holds the complete sum of entry l
            if (j < m) sY[(k0 + r) * MP + j] = part[0];
        }
        // Omega of this head index into shared memory (coalesced), for the last step
        {
            float* sOm = reinterpret_cast<float*>(smem + sm.om);
            const int OP = p.R | 1;
            for (int i = tid; i < K * RS; i += kCoefThreads) {
                const int kk = i / RS, g = i - kk * RS;
                if (g < G) sOm[kk * OP + g] = Om[i];
            }
        }
    } else {
        for (int k = tid; k < K; k += kCoefThreads) {
            const float* row = Sg + (size_t)k * V;
            constexpr int JB = 8;                                     // probe rows per pass over the (cached) state row
            for (int j0 = 0; j0 < m; j0 += JB) {
                float acc[JB];
#pragma unroll
                for (int j = 0; j < JB; ++j) acc[j] = 0.f;
#pragma unroll 4
                for (int c = 0; c < V / 4; ++c) {
                    const float4 s4 = *reinterpret_cast<const float4*>(row + 4 * c);
                    if (j0 == 0) ss = fmaf(s4.x, s4.x, fmaf(s4.y, s4.y, fmaf(s4.z, s4.z, fmaf(s4.w, s4.w, ss))));
#pragma unroll
                    for (int j = 0; j < JB; ++j) {
                        if (j0 + j < m) {
                            const float4 q4 = *reinterpret_cast<const float4*>(sU + (j0 + j) * PT + 4 * c);
                            acc[j] = fmaf(s4.x, q4.x, fmaf(s4.y, q4.y, fmaf(s4.z, q4.z, fmaf(s4.w, q4.w, acc[j]))));
                        }
                    }
                }
#pragma unroll
                for (int j = 0; j < JB; ++j)
                    if (j0 + j < m) sY[k * MP + j0 + j] = acc[j];
            }
        }
    }
    ss = block_sum(ss, sRed);
    const float mu = ss > 0.f ? ss / (float)K : 1.f;
    const float lam = p.ridge_lambda;

    if constexpr (!EXACT) {
        const float inv_mu = 1.f / mu;
        // d_g and 1 / D_G
        for (int g = tid; g < G; g += kCoefThreads) {
            float r2 = 0.f;
#pragma unroll
            for (int j = 0; j < PM; ++j) r2 = fmaf(sRU[g * RUP + j], sRU[g * RUP + j], r2);
            const float d = fmaxf((sUU[g] - r2) * inv_mu, 0.f);
            sUU[g] = d;
            sD[g] = 1.f / (d + lam);
        }
        __syncthreads();
        // T_P = I + L_G^T D_G^{-1} L_G = I + RU^T D_G^{-1} RU / mu (one entry per thread), next to the identity
        if (tid < PM * PM) {
            const int a = tid / PM, b = tid - a * PM;
            float t = 0.f;
            for (int g = 0; g < G; ++g) t = fmaf(sRU[g * RUP + a] * sD[g], sRU[g * RUP + b], t);
            sT[a * 2 * PM + b] = t * inv_mu + (a == b ? 1.f : 0.f);       // (rows / columns beyond m: identity)
            sT[a * 2 * PM + PM + b] = a == b ? 1.f : 0.f;
        }
        __syncthreads();
        // Gauss-Jordan on [T_P | I] by one warp, lane = column (symmetric positive definite, eigenvalues >= 1: no pivoting)
        if (warp == 0) {
            for (int c = 0; c < PM; ++c) {
                const float piv = 1.f / sT[c * 2 * PM + c];
                __syncwarp();
                if (lane < 2 * PM) sT[c * 2 * PM + lane] *= piv;
                __syncwarp();
                for (int a = 0; a < PM; ++a) {
                    if (a == c) continue;
                    const float f = sT[a * 2 * PM + c];
                    __syncwarp();
                    if (lane < 2 * PM) sT[a * 2 * PM + lane] = fmaf(-f, sT[c * 2 * PM + lane], sT[a * 2 * PM + lane]);
                    __syncwarp();
                }
            }
        }
        __syncthreads();
        // column k of C:  M_g = sum_j RU[g][j] Y[k][j] / mu + d_g Omega[k][g];  z = RU^T D^{-1} M;  w = T_P^{-1} z / mu;
        // C[g][k] = (M_g - sum_j RU[g][j] w_j) / D_g   (L_G = RU / sqrt(mu): the two factors 1 / sqrt(mu) are collected in w)
        for (int k = tid; k < K; k += kCoefThreads) {
            float y[PM], z[PM], wv[PM];
#pragma unroll
            for (int j = 0; j < PM; ++j) { y[j] = j < m ? sY[k * MP + j] : 0.f; z[j] = 0.f; }
            const float* omk = reinterpret_cast<const float*>(smem + sm.om) + k * (p.R | 1);
            for (int g = 0; g < G; ++g) {
                float ru[PM];
#pragma unroll
                for (int j4 = 0; j4 < PM / 4; ++j4) {
                    const float4 r4 = *reinterpret_cast<const float4*>(sRU + g * RUP + 4 * j4);
                    ru[4 * j4] = r4.x; ru[4 * j4 + 1] = r4.y; ru[4 * j4 + 2] = r4.z; ru[4 * j4 + 3] = r4.w;
                }
                float Mg = 0.f;
#pragma unroll
                for (int j = 0; j < PM; ++j) Mg = fmaf(ru[j], y[j], Mg);
                Mg = fmaf(Mg, inv_mu, sUU[g] * omk[g]);
                const float t = Mg * sD[g];
#pragma unroll
                for (int j = 0; j < PM; ++j) z[j] = fmaf(ru[j], t, z[j]);
            }
#pragma unroll
            for (int a = 0; a < PM; ++a) {
                float t = 0.f;
#pragma unroll
                for (int b = 0; b < PM; ++b) t = fmaf(sT[a * 2 * PM + PM + b], z[b], t);
                wv[a] = t * inv_mu;
            }
            for (int g = 0; g < G; ++g) {
                float ru[PM];
#pragma unroll
                for (int j4 = 0; j4 < PM / 4; ++j4) {
                    const float4 r4 = *reinterpret_cast<const float4*>(sRU + g * RUP + 4 * j4);
                    ru[4 * j4] = r4.x; ru[4 * j4 + 1] = r4.y; ru[4 * j4 + 2] = r4.z; ru[4 * j4 + 3] = r4.w;
                }
                float Mg = 0.f, corr = 0.f;
#pragma unroll
                for (int j = 0; j < PM; ++j) { Mg = fmaf(ru[j], y[j], Mg); corr = fmaf(ru[j], wv[j], corr); }
                Mg = fmaf(Mg, inv_mu, sUU[g] * omk[g]);
                store_c((size_t)g * K + k, (Mg - corr) * sD[g]);
            }
        }
    } else {
        // A = U^T U + lam mu I = Lc Lc^T (Cholesky in place in sRU's lower triangle, by warp 0, column by column)
        if (warp == 0) {
            for (int c = 0; c < G; ++c) {
                float dsum = sRU[c * MP + c] + lam * mu;
                for (int j = 0; j < c; ++j) dsum = fmaf(-sRU[c * MP + j], sRU[c * MP + j], dsum);
                const float dc = sqrtf(fmaxf(dsum, 1e-30f));
                __syncwarp();
                for (int r = c + 1 + lane; r < G; r += 32) {
                    float t = sRU[r * MP + c];
                    for (int j = 0; j < c; ++j) t = fmaf(-sRU[r * MP + j], sRU[c * MP + j], t);
                    sRU[r * MP + c] = t / dc;
                }
                if (lane == 0) sRU[c * MP + c] = dc;
                __syncwarp();
            }
        }
        __syncthreads();
        // column k of C: solve A c = Y[k][:] (Y[k][g] = <S[k,:], U_g> = (U^T S^T)[g][k]) in place in sY's row k
        for (int k = tid; k < K; k += kCoefThreads) {
            float* y = sY + k * MP;
            for (int g = 0; g < G; ++g) {
                float t = y[g];
                for (int j = 0; j < g; ++j) t = fmaf(-sRU[g * MP + j], y[j], t);
                y[g] = t / sRU[g * MP + g];
            }
            for (int g = G - 1; g >= 0; --g) {
                float t = y[g];
                for (int j = g + 1; j < G; ++j) t = fmaf(-sRU[j * MP + g], y[j], t);
                y[g] = t / sRU[g * MP + g];
                store_c((size_t)g * K + k, y[g]);
            }
        }
    }
}

template <int K, int V>
static int launch_coef_kv(Ctx* ctx, const Params& p, cudaStream_t stream) {
    const bool exact = p.pivots <= 0;
    const int m = exact ? p.R : (p.R < p.pivots ? p.R : p.pivots);
    const CoefSmem sm = make_coef_smem(K, V, p.R, m);
    auto kern = exact ? coef_map_kernel<K, V, 1, 4> : (m <= 4 ? coef_map_kernel<K, V, 0, 4> : coef_map_kernel<K, V, 0, 8>);
    if (sm.total > 48u * 1024u) {
        if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm.total)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
    }
    const size_t heads = (size_t)p.B * p.H;
    kern<<<dim3((unsigned)heads), dim3(kCoefThreads), sm.total, stream>>>(p);
    if ((ctx->last_cuda_error = cudaGetLastError()) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches += 1;
    return SKETCHSSM_OK;
}

// Rebuild the per-(batch, head) coefficient maps from the state and sketch the preceding flush kernel left in memory.
int launch_coef_map(Ctx* ctx, const Params& p, cudaStream_t stream) {
    if (p.pivots > kMaxPivots) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const int K = ctx->cfg.dk, V = ctx->cfg.dv;
    if (K == 128 && V == 128) return launch_coef_kv<128, 128>(ctx, p, stream);
    if (K == 128 && V == 64) return launch_coef_kv<128, 64>(ctx, p, stream);
    if (K == 128 && V == 80) return launch_coef_kv<128, 80>(ctx, p, stream);
    if (K == 64 && V == 64) return launch_coef_kv<64, 64>(ctx, p, stream);
    if (K == 64 && V == 128) return launch_coef_kv<64, 128>(ctx, p, stream);
    return SKETCHSSM_UNSUPPORTED_SHAPE;
}

}  // namespace sketchssm
