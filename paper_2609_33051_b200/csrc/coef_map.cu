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
// One CTA of 128 threads per (batch, head); the sketch rows sit in shared memory.  Pivot form: one warp orthogonalises
// the pivot rows in registers and leaves them as tf32 high parts and remainders; RU = U Q^T, ||U_g||^2 and
// Y[k][j] = <S[k,:], Q_j> run as mma.sync tiles (three tf32 products per tile, ~2^-21 relative), the stream of S with
// every quarter warp loading one whole 128-byte line of a row (the state is requested into L2 when the CTA starts);
// ||S||_F^2 rides along.  One warp then builds and inverts the p x p system in registers while the others prepare two
// small per-rank tables, and thread k forms column k of C in two passes over the ranks with its row of Omega in
// registers (stores coalesced across the CTA).  The single-warp stages rotate over the warps from CTA to CTA.
// Exact form: thread k streams row k of S against all G sketch rows, Cholesky by one warp, one pair of triangular
// solves per thread.  The kernel runs after the flush kernel of the same call and re-reads S_new and U from memory:
// the map needs the complete sketch before it can contract the state with it.
#include "internal.cuh"
#include "lanegroup.cuh"

namespace sketchssm {

namespace {

constexpr int kCoefThreads = 128;
constexpr int kMaxPivots = 8;

struct CoefSmem {
    uint32_t probe, y, ru, small, q, fe, total;   // byte offsets
    int pitch;                                 // floats per probe row
    int qpitch;                                // floats per row of the split probe rows
};

__host__ __device__ inline CoefSmem make_coef_smem(int K, int V, int G, int m) {
    CoefSmem s;
    s.pitch = V % 32 == 0 ? V + 16 : V;                       // 16 mod 32 floats: 16-byte fragment loads of eight rows x four chunks cover all banks
    uint32_t off = 0;
    s.probe = off; off += (uint32_t)(G * s.pitch * 4);        // the G sketch rows; the first m become the probe rows
    const int yf = K * (m + 1) > m * V ? K * (m + 1) : m * V;
    s.y = off; off += (uint32_t)(yf * 4);                     // Y[k][0..m) (pitch m + 1); before that, the m raw pivot rows
    s.ru = off; off += (uint32_t)(G * (m + 1 > 8 ? m + 1 : 8) * 4);   // RU[g][j] = <U_g, probe_j> (pitch m + 1 for the exact form, else the padded pivot count)
    s.small = off; off += (uint32_t)((4 * G + 2 * 8 * 8 + 64) * 4);
    off = (off + 15u) & ~15u;
    s.qpitch = ((V + 31) & ~31) + 16;                         // whole 32-column blocks (zero beyond V), 16 mod 32 floats
    s.q = off; off += (uint32_t)(2 * 8 * s.qpitch * 4);       // eight probe rows (zero beyond m) as tf32 high parts, then their remainders
    s.fe = off; off += (uint32_t)(((G + 3) & ~3) * 17 * 4);   // F[g][0..8) | E[g][0..8) per rank (zero rows up to a multiple of four), then d_g / D_g
    s.total = (off + 15u) & ~15u;
    return s;
}

// x = hi + lo with hi the nearest tf32 value and lo the tf32 rounding of the remainder (together ~21 mantissa bits)
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));
    const float rem = x - __uint_as_float(hi);
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(lo) : "f"(rem));
}

// d += a b for one 16 x 8 x 8 tile (tf32 operands, fp32 accumulation); fragment layouts as the PTX ISA gives them
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

}  // namespace

// EXACT = 0: pivot approximation with m = min(G, P) <= PM probe rows (PM = 4 or 8: loops over pivots unroll and stay in
// registers);  EXACT = 1: ridge form with m = G.
template <int K, int V, int EXACT, int PM>
__global__ void __launch_bounds__(kCoefThreads) coef_map_kernel(const Params p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Heads in descending order: the flush kernel before this one works through every head index from batch 0 upwards,
    // so what it wrote last -- the part of the new state that is still in L2 -- belongs to the highest batch indices.
    const size_t bh = (size_t)gridDim.x - 1 - blockIdx.x;
    // the single-warp stages (Gram-Schmidt, the p x p system) rotate over the warps from CTA to CTA: the warps of equal
    // index of all resident CTAs share one scheduler of the SM
    const int w0 = (int)(blockIdx.x & 3u);
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

    // the state of this head on its way into L2 while the sketch rows are orthogonalised
    for (int i = tid; i < K * V / 32; i += kCoefThreads)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(Sg + 32 * i));

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
    if (EXACT) {
        // ||U_g||^2, one row per thread
        for (int g = tid; g < G; g += kCoefThreads) {
            float a = 0.f;
            for (int v = 0; v < V; ++v) a = fmaf(sU[g * PT + v], sU[g * PT + v], a);
            sUU[g] = a;
        }
    }
    if (!EXACT) {
        // ---- Gram-Schmidt on the first m sketch rows by one warp (two sweeps; a row that lies in the span of its
        // predecessors becomes zero).  The finished rows stay in registers; what the later stages read are their tf32
        // high parts and remainders (eight rows of whole 32-column blocks, zero beyond m and beyond V), the B operands of
        // both tensor-core products.  The other warps write the zero part meanwhile. ----
        uint32_t* sQh = reinterpret_cast<uint32_t*>(smem + sm.q);
        uint32_t* sQl = sQh + 8 * sm.qpitch;
        const int QP = sm.qpitch;
        if (warp == w0) {
            constexpr int EV = (V + 31) / 32;          // elements per lane; beyond V (V = 80) they are zero and never stored
            auto on = [&](int e) { return V % 32 == 0 || lane + 32 * e < V; };
            float q[PM][EV];
#pragma unroll
            for (int j = 0; j < PM; ++j) {
                if (j < m) {
                    float u[EV], ref = 0.f;
#pragma unroll
                    for (int e = 0; e < EV; ++e) { u[e] = on(e) ? sU[j * PT + lane + 32 * e] : 0.f; ref = fmaf(u[e], u[e], ref); }
                    ref = warp_sum(ref);
#pragma unroll
                    for (int sweep = 0; sweep < 2; ++sweep) {
#pragma unroll
                        for (int i = 0; i < j; ++i) {
                            float d = 0.f;
#pragma unroll
                            for (int e = 0; e < EV; ++e) d = fmaf(q[i][e], u[e], d);
                            d = warp_sum(d);
#pragma unroll
                            for (int e = 0; e < EV; ++e) u[e] = fmaf(-d, q[i][e], u[e]);
                        }
                    }
                    float nn = 0.f;
#pragma unroll
                    for (int e = 0; e < EV; ++e) nn = fmaf(u[e], u[e], nn);
                    nn = warp_sum(nn);
                    const float inv = (ref > 0.f && nn > 1e-12f * ref) ? rsqrtf(nn) : 0.f;
#pragma unroll
                    for (int e = 0; e < EV; ++e) {
                        q[j][e] = u[e] * inv;
                        if (on(e)) {
                            uint32_t hi, lo;
                            split_tf32(q[j][e], hi, lo);
                            sQh[j * QP + lane + 32 * e] = hi;
                            sQl[j * QP + lane + 32 * e] = lo;
                        }
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < EV; ++e) q[j][e] = 0.f;
                }
            }
        } else {
            constexpr int VP = (V + 31) & ~31;
            for (int i = (((warp - w0 - 1) & 3) << 5) + lane; i < 8 * VP; i += kCoefThreads - 32) {
                const int j = i / VP, v = i - j * VP;
                if (j >= m || v >= V) { sQh[j * QP + v] = 0u; sQl[j * QP + v] = 0u; }
            }
        }
        __syncthreads();
        // RU[g][j] = <U_g, Q_j> and ||U_g||^2: one 16 x 8 tensor-core tile per 16 ranks (tf32 high parts and remainders,
        // three products), one warp per tile.  Lane (g8, t4) holds, of rows g8 and g8 + 8, the four values 16 cb + 4 t4 .. + 3
        // of every 16 columns; the first k-step takes .x / .y as contraction indices t4 / t4 + 4, the second .z / .w, and
        // the probe operand is permuted the same way.
        {
            constexpr int CB = V / 16;
            static_assert(V % 16 == 0, "fragment tiling");
            const int g8 = lane >> 2, t4 = lane & 3;
            for (int mt = (warp - w0) & 3; 16 * mt < G; mt += kCoefThreads / 32) {
                const int ga = min(16 * mt + g8, G - 1), gb = min(16 * mt + g8 + 8, G - 1);     // (rows beyond G: a copy, never stored)
                const float* ra = sU + ga * PT + 4 * t4;
                const float* rb = sU + gb * PT + 4 * t4;
                const uint32_t* qh = sQh + g8 * QP + 4 * t4;
                const uint32_t* ql = sQl + g8 * QP + 4 * t4;
                float acc[4] = {0.f, 0.f, 0.f, 0.f}, na = 0.f, nb = 0.f;
#pragma unroll
                for (int cb = 0; cb < CB; ++cb) {
                    const float4 a4 = *reinterpret_cast<const float4*>(ra + 16 * cb);
                    const float4 b4 = *reinterpret_cast<const float4*>(rb + 16 * cb);
                    na = fmaf(a4.x, a4.x, fmaf(a4.y, a4.y, fmaf(a4.z, a4.z, fmaf(a4.w, a4.w, na))));
                    nb = fmaf(b4.x, b4.x, fmaf(b4.y, b4.y, fmaf(b4.z, b4.z, fmaf(b4.w, b4.w, nb))));
                    const float x[8] = {a4.x, b4.x, a4.y, b4.y, a4.z, b4.z, a4.w, b4.w};
                    uint32_t hi[8], lo[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) split_tf32(x[e], hi[e], lo[e]);
                    const uint4 bh4 = *reinterpret_cast<const uint4*>(qh + 16 * cb);
                    const uint4 bl4 = *reinterpret_cast<const uint4*>(ql + 16 * cb);
                    const uint32_t ah0[4] = {hi[0], hi[1], hi[2], hi[3]}, al0[4] = {lo[0], lo[1], lo[2], lo[3]};
                    const uint32_t ah1[4] = {hi[4], hi[5], hi[6], hi[7]}, al1[4] = {lo[4], lo[5], lo[6], lo[7]};
                    mma_tf32(acc, al0, bh4.x, bh4.y);
                    mma_tf32(acc, ah0, bl4.x, bl4.y);
                    mma_tf32(acc, ah0, bh4.x, bh4.y);
                    mma_tf32(acc, al1, bh4.z, bh4.w);
                    mma_tf32(acc, ah1, bl4.z, bl4.w);
                    mma_tf32(acc, ah1, bh4.z, bh4.w);
                }
                na += __shfl_xor_sync(0xffffffffu, na, 1); na += __shfl_xor_sync(0xffffffffu, na, 2);
                nb += __shfl_xor_sync(0xffffffffu, nb, 1); nb += __shfl_xor_sync(0xffffffffu, nb, 2);
                const int g0 = 16 * mt + g8, g1 = g0 + 8, j0 = 2 * t4;
                if (t4 == 0) {
                    if (g0 < G) sUU[g0] = na;
                    if (g1 < G) sUU[g1] = nb;
                }
                if (j0 < RUP) {       // (probes m .. RUP-1 are zero rows: their entries come out as zeros)
                    if (g0 < G) { sRU[g0 * RUP + j0] = acc[0]; sRU[g0 * RUP + j0 + 1] = acc[1]; }
                    if (g1 < G) { sRU[g1 * RUP + j0] = acc[2]; sRU[g1 * RUP + j0 + 1] = acc[3]; }
                }
            }
        }
        // (no barrier here: the stream below reads the split probe rows, which are complete, and writes Y; RU and the
        // norms are read behind the barrier that follows the stream)
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
        // Y = S Q on the tensor cores (mma.sync, tf32 operands split into a high part and a remainder: three products per
        // tile, the remainder x remainder term dropped, ~2^-21 relative).  A warp owns K / 4 rows.
        static_assert(K % 64 == 0, "rows per warp");
        if constexpr (PM == 4) {
        // Up to four probes: a tile is 8 rows of S by 32 columns.  The 16 tile rows are the two 16-column halves of the 8
        // rows (row g8 of the tile: row g8 / 2 of S, half g8 & 1), the 8 tile columns the four probes restricted to the
        // first half and the four restricted to the second; entry (g8 even, j) + entry (g8 + 1, 4 + j) is Y[row][j] and the
        // other entries are discarded.  This way the eight lanes of a quarter warp load one whole 128-byte line of a row
        // (the contraction index inside a half is permuted as above: lane chunk .x / .y, then .z / .w).
        constexpr int NCB = (V + 31) / 32;
        const int g8 = lane >> 2, t4 = lane & 3, l8 = lane & 7;
        const uint32_t* sQh = reinterpret_cast<const uint32_t*>(smem + sm.q);
        const uint32_t* sQl = sQh + 8 * sm.qpitch;
        uint4 bh[NCB], bl[NCB];                     // probe g8 & 3, half g8 >> 2: the same for every tile
#pragma unroll
        for (int c = 0; c < NCB; ++c) {
            const int off = (g8 & 3) * sm.qpitch + 32 * c + 16 * (g8 >> 2) + 4 * t4;
            bh[c] = *reinterpret_cast<const uint4*>(sQh + off);
            bl[c] = *reinterpret_cast<const uint4*>(sQl + off);
        }
        constexpr int RPW = K / (kCoefThreads / 32);        // rows per warp
        for (int r0 = warp * RPW; r0 < (warp + 1) * RPW; r0 += 8) {
            const float* pa = Sg + (size_t)(r0 + (g8 >> 1)) * V + 4 * l8;      // tile rows 0 .. 7: rows r0 .. r0 + 3 of S
            const float* pb = pa + 4 * V;                                       // tile rows 8 .. 15: rows r0 + 4 .. r0 + 7
            float4 s0[NCB], s1[NCB];
#pragma unroll
            for (int c = 0; c < NCB; ++c) {
                if (V % 32 == 0 || 32 * c + 4 * l8 < V) {
                    s0[c] = *reinterpret_cast<const float4*>(pa + 32 * c);
                    s1[c] = *reinterpret_cast<const float4*>(pb + 32 * c);
                } else {
                    s0[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                    s1[c] = s0[c];
                }
            }
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < NCB; ++c) {
                const float x[8] = {s0[c].x, s1[c].x, s0[c].y, s1[c].y, s0[c].z, s1[c].z, s0[c].w, s1[c].w};
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    ss = fmaf(x[e], x[e], ss);
                    split_tf32(x[e], hi[e], lo[e]);
                }
                const uint32_t ah0[4] = {hi[0], hi[1], hi[2], hi[3]}, al0[4] = {lo[0], lo[1], lo[2], lo[3]};
                const uint32_t ah1[4] = {hi[4], hi[5], hi[6], hi[7]}, al1[4] = {lo[4], lo[5], lo[6], lo[7]};
                mma_tf32(acc, al0, bh[c].x, bh[c].y);
                mma_tf32(acc, ah0, bl[c].x, bl[c].y);
                mma_tf32(acc, ah0, bh[c].x, bh[c].y);
                mma_tf32(acc, al1, bh[c].z, bh[c].w);
                mma_tf32(acc, ah1, bl[c].z, bl[c].w);
                mma_tf32(acc, ah1, bh[c].z, bh[c].w);
            }
            // (g8 even, probes 2 t4, 2 t4 + 1 of the first half) + (g8 + 1, the same probes of the second half: lane ^ 6)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 6);
            if ((g8 & 1) == 0 && t4 < 2) {
                const int row = r0 + (g8 >> 1), j0 = 2 * t4;
                if (j0 < m) { sY[row * MP + j0] = acc[0]; sY[(row + 4) * MP + j0] = acc[2]; }
                if (j0 + 1 < m) { sY[row * MP + j0 + 1] = acc[1]; sY[(row + 4) * MP + j0 + 1] = acc[3]; }
            }
        }
        } else {
        // Up to eight probes: a tile is 16 rows of S by 16 columns.  Lane (g8, t4) loads, for every 16 columns, the four
        // consecutive values 4 t4 .. 4 t4 + 3 of rows g8 and g8 + 8; the contraction index is permuted the same way on
        // both operands, so the first k-step takes the values .x / .y as columns t4 / t4 + 4 and the second .z / .w.
        constexpr int CB = V / 16;
        const int g8 = lane >> 2, t4 = lane & 3;
        const uint32_t* sQh = reinterpret_cast<const uint32_t*>(smem + sm.q);
        const uint32_t* sQl = sQh + 8 * sm.qpitch;
        const uint32_t* qh = sQh + g8 * sm.qpitch + 4 * t4;
        const uint32_t* ql = sQl + g8 * sm.qpitch + 4 * t4;
        constexpr int RPW = K / (kCoefThreads / 32);        // rows per warp
        for (int m0 = warp * RPW; m0 < (warp + 1) * RPW; m0 += 16) {
            const float* r0 = Sg + (size_t)(m0 + g8) * V + 4 * t4;
            const float* r1 = r0 + 8 * V;
            float4 s0[CB], s1[CB];
#pragma unroll
            for (int cb = 0; cb < CB; ++cb) {
                s0[cb] = *reinterpret_cast<const float4*>(r0 + 16 * cb);
                s1[cb] = *reinterpret_cast<const float4*>(r1 + 16 * cb);
            }
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int cb = 0; cb < CB; ++cb) {
                const float x[8] = {s0[cb].x, s1[cb].x, s0[cb].y, s1[cb].y, s0[cb].z, s1[cb].z, s0[cb].w, s1[cb].w};
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    ss = fmaf(x[e], x[e], ss);
                    split_tf32(x[e], hi[e], lo[e]);
                }
                const uint4 bh4 = *reinterpret_cast<const uint4*>(qh + 16 * cb);
                const uint4 bl4 = *reinterpret_cast<const uint4*>(ql + 16 * cb);
                const uint32_t ah0[4] = {hi[0], hi[1], hi[2], hi[3]}, al0[4] = {lo[0], lo[1], lo[2], lo[3]};
                const uint32_t ah1[4] = {hi[4], hi[5], hi[6], hi[7]}, al1[4] = {lo[4], lo[5], lo[6], lo[7]};
                mma_tf32(acc, al0, bh4.x, bh4.y);
                mma_tf32(acc, ah0, bl4.x, bl4.y);
                mma_tf32(acc, ah0, bh4.x, bh4.y);
                mma_tf32(acc, al1, bh4.z, bh4.w);
                mma_tf32(acc, ah1, bl4.z, bl4.w);
                mma_tf32(acc, ah1, bh4.z, bh4.w);
            }
            // accumulator fragment: (row g8, probes 2 t4, 2 t4 + 1), (row g8 + 8, the same probes)
            const int j0 = 2 * t4;
            if (j0 < m) { sY[(m0 + g8) * MP + j0] = acc[0]; sY[(m0 + g8 + 8) * MP + j0] = acc[2]; }
            if (j0 + 1 < m) { sY[(m0 + g8) * MP + j0 + 1] = acc[1]; sY[(m0 + g8 + 8) * MP + j0 + 1] = acc[3]; }
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
    // ||S||_F^2 over the CTA: one partial per warp, summed by every thread behind the barrier that also publishes Y
    ss = warp_sum(ss);
    if (lane == 0) sRed[warp] = ss;
    __syncthreads();
    ss = 0.f;
    for (int i = 0; i < kCoefThreads / 32; ++i) ss += sRed[i];
    const float mu = ss > 0.f ? ss / (float)K : 1.f;
    const float lam = p.ridge_lambda;

    if constexpr (!EXACT) {
        const float inv_mu = 1.f / mu;
        // residual diagonal d_g = max((||U_g||^2 - ||Q^T U_g||^2) / mu, 0) and 1 / D_g of one rank
        auto diag = [&](int g, float& d, float& dinv) {
            float r2 = 0.f;
#pragma unroll
            for (int j = 0; j < PM; ++j) r2 = fmaf(sRU[g * RUP + j], sRU[g * RUP + j], r2);
            d = fmaxf((sUU[g] - r2) * inv_mu, 0.f);
            dinv = 1.f / (d + lam);
        };
        if (warp == w0) {
            // One warp: the p x p Woodbury system, start to finish in registers (the other warps build the per-rank tables
            // meanwhile).  Lane (gq, b) holds column b of [T_P | I] for the ranks g = gq mod NG; the groups are summed by
            // shuffles, after which every group holds the whole system.
            //   T_P = I + L_G^T D_G^{-1} L_G = I + RU^T D_G^{-1} RU / mu
            constexpr int W2 = 2 * PM, NG = 32 / W2;
            const int b = lane & (W2 - 1), gq = lane / W2;
            float t[PM];
#pragma unroll
            for (int a = 0; a < PM; ++a) t[a] = 0.f;
            for (int g = gq; g < G; g += NG) {
                float ru[PM], r2 = 0.f;
#pragma unroll
                for (int j = 0; j < PM; ++j) { ru[j] = sRU[g * RUP + j]; r2 = fmaf(ru[j], ru[j], r2); }
                const float d = fmaxf((sUU[g] - r2) * inv_mu, 0.f);
                const float w = b < PM ? sRU[g * RUP + b] / (d + lam) : 0.f;
#pragma unroll
                for (int a = 0; a < PM; ++a) t[a] = fmaf(ru[a], w, t[a]);
            }
#pragma unroll
            for (int o = W2; o < 32; o <<= 1)
#pragma unroll
                for (int a = 0; a < PM; ++a) t[a] += __shfl_xor_sync(0xffffffffu, t[a], o);
#pragma unroll
            for (int a = 0; a < PM; ++a) t[a] = b < PM ? fmaf(t[a], inv_mu, a == b ? 1.f : 0.f) : (a == b - PM ? 1.f : 0.f);
            // Gauss-Jordan on [T_P | I], lane = column (symmetric positive definite, eigenvalues >= 1: no pivoting)
#pragma unroll
            for (int c = 0; c < PM; ++c) {
                float f[PM];
#pragma unroll
                for (int a = 0; a < PM; ++a) f[a] = __shfl_sync(0xffffffffu, t[a], c, W2);     // column c of the system
                t[c] *= 1.f / f[c];
#pragma unroll
                for (int a = 0; a < PM; ++a)
                    if (a != c) t[a] = fmaf(-f[a], t[c], t[a]);
            }
            if (gq == 0) {
#pragma unroll
                for (int a = 0; a < PM; ++a) sT[a * W2 + b] = t[a];
            }
        } else {
            // the per-rank tables of the last step: F[g][j] = RU[g][j] / D_g, E[g][j] = d_g F[g][j], and d_g / D_g (zero
            // rows up to a multiple of four ranks)
            float* sFE = reinterpret_cast<float*>(smem + sm.fe);
            float* sDD = sFE + ((p.R + 3) & ~3) * 16;
            const int G4 = (G + 3) & ~3;
            for (int i = (((warp - w0 - 1) & 3) << 5) + lane; i < G4 * PM; i += kCoefThreads - 32) {
                const int g = i / PM, j = i - g * PM;
                float d = 0.f, dinv = 0.f, f = 0.f;
                if (g < G) {
                    diag(g, d, dinv);
                    f = sRU[g * RUP + j] * dinv;
                }
                sFE[g * 16 + j] = f;
                sFE[g * 16 + 8 + j] = f * d;
                if (j == 0) sDD[g] = d * dinv;
            }
        }
        __syncthreads();
        // column k of C.  With M_g = sum_j RU[g][j] Y[k][j] / mu + d_g Omega[k][g], z = RU^T D^{-1} M and w = T_P^{-1} z / mu
        // the entry is C[g][k] = (M_g - sum_j RU[g][j] w_j) / D_g.  Since RU^T D^{-1} RU / mu = T_P - I this collapses to
        //   yy = T_P^{-1} (Y[k][:] - E^T Omega[k][:]) / mu,   C[g][k] = sum_j F[g][j] yy_j + (d_g / D_g) Omega[k][g],
        // two passes over the ranks with one table row each; thread k reads its own row of Omega from memory (a warp
        // covers 32 consecutive rows: whole sectors).
        {
            const float* sFE = reinterpret_cast<const float*>(smem + sm.fe);
            const float* sDD = sFE + ((p.R + 3) & ~3) * 16;
            const int G4 = (G + 3) & ~3;
            const bool vec = (RS & 3) == 0;
            for (int k = tid; k < K; k += kCoefThreads) {
                const float* omk = Om + (size_t)k * RS;
                auto om4 = [&](int g0, float (&o)[4]) {
                    if (vec) {
                        const float4 t = *reinterpret_cast<const float4*>(omk + g0);
                        o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
                    } else {
#pragma unroll
                        for (int u = 0; u < 4; ++u) o[u] = g0 + u < G ? omk[g0 + u] : 0.f;
                    }
                };
                float y[PM], yy[PM];
#pragma unroll
                for (int j = 0; j < PM; ++j) y[j] = j < m ? sY[k * MP + j] : 0.f;
                // first pass over four ranks: y -= E^T Omega[k][:]
                auto pass1 = [&](int g0, const float (&o)[4]) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
#pragma unroll
                        for (int j4 = 0; j4 < PM / 4; ++j4) {
                            const float4 e4 = *reinterpret_cast<const float4*>(sFE + (g0 + u) * 16 + 8 + 4 * j4);
                            y[4 * j4] = fmaf(-e4.x, o[u], y[4 * j4]);
                            y[4 * j4 + 1] = fmaf(-e4.y, o[u], y[4 * j4 + 1]);
                            y[4 * j4 + 2] = fmaf(-e4.z, o[u], y[4 * j4 + 2]);
                            y[4 * j4 + 3] = fmaf(-e4.w, o[u], y[4 * j4 + 3]);
                        }
                    }
                };
                // second pass: the entries of four ranks
                auto pass2 = [&](int g0, const float (&o)[4]) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float c = sDD[g0 + u] * o[u];
#pragma unroll
                        for (int j4 = 0; j4 < PM / 4; ++j4) {
                            const float4 f4 = *reinterpret_cast<const float4*>(sFE + (g0 + u) * 16 + 4 * j4);
                            c = fmaf(f4.x, yy[4 * j4], fmaf(f4.y, yy[4 * j4 + 1], fmaf(f4.z, yy[4 * j4 + 2], fmaf(f4.w, yy[4 * j4 + 3], c))));
                        }
                        if (g0 + u < G) store_c((size_t)(g0 + u) * K + k, c);
                    }
                };
                auto solve = [&]() {
#pragma unroll
                    for (int a = 0; a < PM; ++a) {
                        float t = 0.f;
#pragma unroll
                        for (int b = 0; b < PM; ++b) t = fmaf(sT[a * 2 * PM + PM + b], y[b], t);
                        yy[a] = t * inv_mu;
                    }
                };
                if (G4 <= 16) {
                    // up to 16 ranks: the row of Omega is read once and kept in registers for both passes
                    float o[4][4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        if (4 * c < G4) om4(4 * c, o[c]);
                        else { o[c][0] = 0.f; o[c][1] = 0.f; o[c][2] = 0.f; o[c][3] = 0.f; }
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (4 * c < G4) pass1(4 * c, o[c]);
                    solve();
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (4 * c < G4) pass2(4 * c, o[c]);
                } else {
                    for (int g0 = 0; g0 < G4; g0 += 4) {
                        float o[4];
                        om4(g0, o);
                        pass1(g0, o);
                    }
                    solve();
                    for (int g0 = 0; g0 < G4; g0 += 4) {
                        float o[4];
                        om4(g0, o);
                        pass2(g0, o);
                    }
                }
            }
        }
    } else {
        // A = U^T U + lam mu I = Lc Lc^T (Cholesky in place in sRU's lower triangle, by warp 0, column by column)
        if (warp == w0) {
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
    // (shared memory carved out for as many CTAs per SM as the registers allow; the kernel makes little use of L1)
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
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
