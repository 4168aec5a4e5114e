// State-update (flush) kernel for the gated delta rule (GDN) on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Replaying n tokens of S_s = a_s S_{s-1} + k_s e_s^T,  e_s = beta_s (v_s - (a_s S_{s-1})^T k_s)  (Eq. 1, 3) one at
// a time is 3 K V n dependent FMA-pipe operations per head and runs at a quarter of the HBM rate.  Unrolled over
// the window it is two contractions around small per-head matrices built from the ring alone:
//     E     = T (V - Kd S_0)                   n x V      e_s stacked;  Kd rows = (prod_{i<=s} a_i) k_s,
//     T     = (I + Bd A)^{-1} Bd               n x n      A_sj = (prod_{j<i<=s} a_i) <k_j, k_s>, j < s (strictly lower),
//     S_new = (prod_i a_i) S_0 + Lambda^T E    K x V      Lambda rows = (prod_{i>s} a_i) k_s,
// which is the WY form of the transition product (Appendix C, Eq. 41-42) applied to the state instead of the query.
// No quotient of decay products is ever formed: every product of decays is built by multiplication.
//
// Tile = one head with V = 128: TMEM lane / thread t = value column j.  Per head:
//   ring only (CUDA cores + mma.sync for the Gram matrix): A, T by forward substitution, Pi = T Kd, W' = T V
//   phase A  : stream S_0 once through registers, split to bf16 hi + lo as the K-major A operand, 32 rows at a time;
//              tcgen05.mma  G[j, s] = sum_i S_0[i, j] Pi[s, i]      (three products hi*hi + lo*hi + hi*lo)
//   epilogue : E[s, j] = W'[s, j] - G[j, s]  ->  bf16 hi + lo A operand;  Lambda hi + lo B operand
//   phase C  : tcgen05.mma  T[j, i] = sum_s E[s, j] Lambda[s, i]
//   epilogue : S_new[i, j] = d S_0[i, j] + T[j, i] (S_0 read a second time, from L2 where it still is), written
//              back; S_new hi + lo -> tcgen05.mma  [U | o] = S_new^T [Omega | q]   (as in the Mamba-2 kernel)
// Domain: GDN, bf16 I/O, K = V = 128, at most 32 tokens per flush.
#include "internal.cuh"
#include "tc_common.cuh"

namespace sketchssm {

using namespace tc;

namespace {

constexpr int kMaxTok = 32;
constexpr int kRowB = 272;           // padded shared-memory row of 128 bf16
constexpr int kTS = 36;              // row stride (floats) of the small n x n matrices

struct DSmem {
    uint32_t r1, ba_hi, ba_lo, b2_hi, b2_lo, kraw, wp, gm, tm, pm, gates, bars, tmem_slot, total;
};

__host__ __device__ inline DSmem make_dsmem(int NP) {
    DSmem s;
    uint32_t off = 0;
    s.r1 = off; off += 32768u;                                   // phase-A chunk buffers / phase-C operands / MMA-2 chunk buffers
    s.ba_hi = off; off += (uint32_t)kMaxTok * kK * 2u;
    s.ba_lo = off; off += (uint32_t)kMaxTok * kK * 2u;
    s.b2_hi = off; off += (uint32_t)NP * kK * 2u;
    s.b2_lo = off; off += (uint32_t)NP * kK * 2u;
    s.kraw = off; off += (uint32_t)kMaxTok * kRowB;
    s.wp = off; off += (uint32_t)kMaxTok * 128u * 4u;             // W'[s][j]
    s.gm = off; off += (uint32_t)kMaxTok * kTS * 4u;
    s.tm = off; off += (uint32_t)kMaxTok * kTS * 4u;
    s.pm = off; off += (uint32_t)kMaxTok * kTS * 4u;
    s.gates = off; off += 192u * 4u;                             // beta[32], alpha[32], cumd[32], dn[32], d_total
    s.bars = off; off += 64u;
    s.tmem_slot = off; off += 64u;
    s.total = off;
    return s;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

}  // namespace

__global__ void __launch_bounds__(kTcThreads) update_tc_gdn_kernel(const Params p) {
    constexpr int K = kK, V = 128;
    extern __shared__ __align__(1024) unsigned char smem[];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = p.R, H = p.H, B = p.B;
    const int NP = (R + 1 + 15) & ~15;
    const int n_ring = p.n_before, n_tot = n_ring + (p.has_token ? 1 : 0);
    const int n_pad = n_tot > 16 ? 32 : 16;
    const DSmem sm = make_dsmem(NP);
    unsigned char* sR1 = smem + sm.r1;
    unsigned char* sBAhi = smem + sm.ba_hi;
    unsigned char* sBAlo = smem + sm.ba_lo;
    __nv_bfloat16* sB2hi = reinterpret_cast<__nv_bfloat16*>(smem + sm.b2_hi);
    __nv_bfloat16* sB2lo = reinterpret_cast<__nv_bfloat16*>(smem + sm.b2_lo);
    unsigned char* sKraw = smem + sm.kraw;
    float* sWp = reinterpret_cast<float*>(smem + sm.wp);
    float* sGm = reinterpret_cast<float*>(smem + sm.gm);
    float* sTm = reinterpret_cast<float*>(smem + sm.tm);
    float* sPm = reinterpret_cast<float*>(smem + sm.pm);
    float* sBeta = reinterpret_cast<float*>(smem + sm.gates);
    float* sAlpha = sBeta + 32;
    float* sCum = sBeta + 64;
    float* sDn = sBeta + 96;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);   // [0] phase A / C, [1..2] chunk buffers, [3] MMA 2 all
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + sm.tmem_slot);

    const uint32_t tmem_cols = NP <= 32 ? 128u : 256u;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(&bars[i], 1);
        mbar_fence_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    grid_dep_wait();
    grid_dep_launch_dependents();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_t = tmem_base;                              // G (n_pad columns), then T (128 columns)
    const uint32_t tmem_u = tmem_base + (NP <= 32 ? 0u : 128u);     // UT
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;

    constexpr uint32_t SBO = 128, LBO_M = 2048;                      // operands with 128 rows on the MN side
    const uint32_t LBO_BA = (uint32_t)n_pad * 16u;                   // Pi^T: n_pad rows on the N side
    const uint32_t LBO2B = (uint32_t)NP * 16u;
    // bf16 x bf16 -> fp32, M = 128
    const uint32_t idescA = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)n_pad >> 3) << 17) | ((128u >> 4) << 24);   // K-major x K-major
    const uint32_t idescC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24); // K-major x MN-major
    const uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)NP >> 3) << 17) | ((128u >> 4) << 24);

    const long long n_tiles = (long long)H * B;
    const int tile0 = (int)(n_tiles * blockIdx.x / gridDim.x);
    const int tile1 = (int)(n_tiles * (blockIdx.x + 1) / gridDim.x);
    const int j = tid;
    int cur_h = -1;
    uint32_t ph0 = 0, ph1[2] = {0, 0}, ph3 = 0;
    bool dead = false;

    for (int tile = tile0; tile < tile1 && !dead; ++tile) {
        const int h = tile / B, b = tile - h * B;
        const size_t bh = (size_t)b * H + h;
        const unsigned char* rh = p.ring + bh * p.rl.head_bytes;

        // ---- W = [Omega | q] hi/lo, K-major; Omega part once per head index ----
        if (h != cur_h) {
            const float* og = p.omega + (size_t)h * K * R;
            for (int idx = tid; idx < K * NP; idx += kTcThreads) {
                const int i = idx / NP, g = idx % NP;
                __nv_bfloat16 hi = __float2bfloat16_rn(0.f), lo = hi;
                if (g < R && p.write_sketch) split_bf16(og[(size_t)i * R + g], hi, lo);
                const uint32_t o2 = ((g & 7) * 16 + (g >> 3) * SBO + (i >> 3) * LBO2B + (i & 7) * 2) >> 1;
                sB2hi[o2] = hi;
                sB2lo[o2] = lo;
            }
            cur_h = h;
            __syncthreads();     // the query columns written next overlap the zero padding written above
        }
        if (p.q != nullptr) {
            const int i = tid, g = R;
            const uint32_t o2 = ((g & 7) * 16 + (g >> 3) * SBO + (i >> 3) * LBO2B + (i & 7) * 2) >> 1;
            sB2hi[o2] = reinterpret_cast<const __nv_bfloat16*>(p.q)[bh * K + i];
        }

        float dtot = 1.f;
        if (n_tot > 0) {
            // ---- ring -> shared memory: keys (rows >= n_tot zero), gates; this thread's value column -> registers ----
            for (int idx = tid; idx < kMaxTok * (K / 8); idx += kTcThreads) {
                const int s = idx / (K / 8), a = idx % (K / 8);
                uint4 val = make_uint4(0, 0, 0, 0);
                if (s < n_ring) val = *reinterpret_cast<const uint4*>(rh + ((size_t)s * K + a * 8) * 2);
                else if (s < n_tot) val = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.k) + bh * K + a * 8);
                *reinterpret_cast<uint4*>(sKraw + (size_t)s * kRowB + a * 16) = val;
            }
            if (tid < kMaxTok) {
                const int s = tid;
                float bt = 0.f, al = 1.f;
                if (s < n_ring) {
                    bt = reinterpret_cast<const float*>(rh + p.rl.beta_off)[s];
                    al = reinterpret_cast<const float*>(rh + p.rl.decay_off)[s];
                } else if (s < n_tot) {
                    bt = p.beta[bh];
                    al = reinterpret_cast<const float*>(p.decay)[bh];
                }
                sBeta[s] = bt;
                sAlpha[s] = al;
            }
            for (int idx = tid; idx < kMaxTok * kTS; idx += kTcThreads) sTm[idx] = 0.f;
            float vreg[kMaxTok];
#pragma unroll
            for (int c = 0; c < kMaxTok; ++c) {
                float x = 0.f;
                if (c < n_ring) x = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(rh + p.rl.v_off)[(size_t)c * V + j]);
                else if (c < n_tot) x = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.v)[bh * V + j]);
                vreg[c] = x;
            }
            __syncthreads();

            // ---- products of decays (no quotients) and the Gram matrix <k_s, k_j> ----
            if (tid < kMaxTok) {
                const int s = tid;
                float pr = 1.f;                                   // P(j, s) = prod_{j < i <= s} alpha_i, for j = s-1 .. 0
                for (int jj = s - 1; jj >= 0; --jj) {
                    pr *= sAlpha[jj + 1];
                    sPm[s * kTS + jj] = pr;
                }
                sCum[s] = pr * sAlpha[0];                         // prod_{i <= s} alpha_i  (pr = prod_{0 < i <= s} when the loop ends)
                float dn = 1.f;
                for (int i = s + 1; i < n_tot; ++i) dn *= sAlpha[i];
                sDn[s] = s < n_tot ? dn : 0.f;
            }
            {
                const int combos = (n_pad / 16) * (n_pad / 8);
                for (int cmb = warp; cmb < combos; cmb += 4) {
                    const int mt = cmb / (n_pad / 8), nt = cmb % (n_pad / 8);
                    float acc[4] = {0.f, 0.f, 0.f, 0.f};
                    const uint32_t abase = smem_u32(sKraw) + (uint32_t)(mt * 16 + (lane & 15)) * kRowB + (uint32_t)(lane >> 4) * 16u;
                    const uint32_t bbase = smem_u32(sKraw) + (uint32_t)(nt * 8 + (lane & 7)) * kRowB + (uint32_t)((lane >> 3) & 1) * 16u;
#pragma unroll
                    for (int ks = 0; ks < K / 16; ++ks) {
                        uint32_t a[4], bb[2];
                        ldmatrix_x4(abase + ks * 32, a);
                        ldmatrix_x2(bbase + ks * 32, bb);
                        mma_16816(acc, a, bb);
                    }
                    const int r0 = mt * 16 + (lane >> 2), c0 = nt * 8 + (lane & 3) * 2;
                    sGm[r0 * kTS + c0] = acc[0];
                    sGm[r0 * kTS + c0 + 1] = acc[1];
                    sGm[(r0 + 8) * kTS + c0] = acc[2];
                    sGm[(r0 + 8) * kTS + c0 + 1] = acc[3];
                }
            }
            __syncthreads();
            // beta_s A_sj in place of the Gram entries (strictly lower triangle)
            if (tid < n_tot) {
                const int s = tid;
                const float bs = sBeta[s];
                for (int jj = 0; jj < s; ++jj) sGm[s * kTS + jj] *= bs * sPm[s * kTS + jj];
            }
            __syncthreads();
            // ---- T = (I + Bd A)^{-1} Bd by forward substitution, one column per thread ----
            if (tid < n_tot) {
                const int c = tid;
                sTm[c * kTS + c] = 1.f;
                for (int s = c + 1; s < n_tot; ++s) {
                    float acc = 0.f;
                    for (int jj = c; jj < s; ++jj) acc = fmaf(sGm[s * kTS + jj], sTm[jj * kTS + c], acc);
                    sTm[s * kTS + c] = -acc;
                }
                const float bc = sBeta[c];
                for (int s = c; s < n_tot; ++s) sTm[s * kTS + c] *= bc;
            }
            __syncthreads();
            dtot = sCum[n_tot - 1];

            // ---- Pi = T Kd (B operand of phase A, bf16 hi/lo) and W' = T V (column j of it), one channel / column per thread ----
            {
                float kreg[kMaxTok];
#pragma unroll
                for (int c = 0; c < kMaxTok; ++c)
                    kreg[c] = c < n_tot ? sCum[c] * __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(sKraw + (size_t)c * kRowB)[tid]) : 0.f;
                for (int s = 0; s < n_pad; ++s) {
                    float pi = 0.f, wp = 0.f;
                    const float4* trow = reinterpret_cast<const float4*>(sTm + s * kTS);
#pragma unroll
                    for (int c4 = 0; c4 < kMaxTok / 4; ++c4) {
                        const float4 t4 = trow[c4];
                        pi = fmaf(t4.x, kreg[4 * c4], pi);     wp = fmaf(t4.x, vreg[4 * c4], wp);
                        pi = fmaf(t4.y, kreg[4 * c4 + 1], pi); wp = fmaf(t4.y, vreg[4 * c4 + 1], wp);
                        pi = fmaf(t4.z, kreg[4 * c4 + 2], pi); wp = fmaf(t4.z, vreg[4 * c4 + 2], wp);
                        pi = fmaf(t4.w, kreg[4 * c4 + 3], pi); wp = fmaf(t4.w, vreg[4 * c4 + 3], wp);
                    }
                    sWp[s * 128 + j] = wp;
                    __nv_bfloat16 hi, lo;
                    split_bf16(pi, hi, lo);
                    const uint32_t off = (s & 7) * 16 + (s >> 3) * SBO + (tid >> 3) * LBO_BA + (tid & 7) * 2;   // (n = s, k = i = tid)
                    *reinterpret_cast<__nv_bfloat16*>(sBAhi + off) = hi;
                    *reinterpret_cast<__nv_bfloat16*>(sBAlo + off) = lo;
                }
            }

            // ---- phase A: G[j, s] = sum_i S_0[i, j] Pi[s, i] ----
            const float* Sg = p.state + bh * (size_t)K * V + j;
            float s0[kChunk];
#pragma unroll
            for (int ii = 0; ii < kChunk; ++ii) s0[ii] = Sg[(size_t)ii * V];
            for (int c = 0; c < K / kChunk; ++c) {
                float s0n[kChunk];
                if (c + 1 < K / kChunk) {
#pragma unroll
                    for (int ii = 0; ii < kChunk; ++ii) s0n[ii] = Sg[(size_t)((c + 1) * kChunk + ii) * V];
                }
                if (c >= 2) {
                    if (!mbar_wait_bounded(&bars[1 + (c & 1)], ph1[c & 1])) { record_fault(p.status, kFaultUpdateWait, 11); dead = true; }
                    ph1[c & 1] ^= 1;
                }
                unsigned char* ahi = sR1 + (size_t)(c & 1) * 16384u;
                unsigned char* alo = ahi + 8192u;
#pragma unroll
                for (int v8 = 0; v8 < kChunk / 8; ++v8) {
                    uint32_t ohi[4], olo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) split_bf16x2(s0[v8 * 8 + 2 * e], s0[v8 * 8 + 2 * e + 1], ohi[e], olo[e]);
                    const uint32_t off = (tid & 7) * 16 + (tid >> 3) * SBO + v8 * LBO_M;
                    *reinterpret_cast<uint4*>(ahi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                    *reinterpret_cast<uint4*>(alo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
                }
                proxy_fence();
                tc_fence_before();
                __syncthreads();
                if (tid == 0) {
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < kChunk / 16; ++ks) {
                        const uint32_t kb = (uint32_t)(c * (kChunk / 8) + ks * 2) * LBO_BA;
                        const uint64_t dahi = make_desc(smem_u32(ahi) + ks * 2 * LBO_M, LBO_M, SBO);
                        const uint64_t dalo = make_desc(smem_u32(alo) + ks * 2 * LBO_M, LBO_M, SBO);
                        const uint64_t dbhi = make_desc(smem_u32(sBAhi) + kb, LBO_BA, SBO);
                        const uint64_t dblo = make_desc(smem_u32(sBAlo) + kb, LBO_BA, SBO);
                        tc_mma_bf16(tmem_t, dahi, dbhi, idescA, (c | ks) ? 1u : 0u);
                        tc_mma_bf16(tmem_t, dalo, dbhi, idescA, 1u);
                        tc_mma_bf16(tmem_t, dahi, dblo, idescA, 1u);
                    }
                    tc_commit(c + 1 < K / kChunk ? &bars[1 + (c & 1)] : &bars[0]);
                }
                if (c + 1 < K / kChunk) {
#pragma unroll
                    for (int ii = 0; ii < kChunk; ++ii) s0[ii] = s0n[ii];
                }
            }
            if (!mbar_wait_bounded(&bars[1], ph1[0])) { record_fault(p.status, kFaultUpdateWait, 12); dead = true; }
            ph1[0] ^= 1;
            if (!mbar_wait_bounded(&bars[0], ph0)) { record_fault(p.status, kFaultUpdateWait, 13); dead = true; }
            ph0 ^= 1;
            tc_fence_after();

            // ---- epilogue A: E[s, j] = W'[s, j] - G[j, s] -> A operand (K-major, k = s); Lambda -> B operand (MN-major) ----
            {
                unsigned char* ehi = sR1;                         // 128 x n_pad bf16
                unsigned char* elo = sR1 + 8192u;
                unsigned char* lhi = sR1 + 16384u;                // n_pad x 128 bf16
                unsigned char* llo = sR1 + 24576u;
                for (int s0c = 0; s0c < n_pad; s0c += 16) {
                    float g[16];
                    tmem_ld16(tmem_t + lane_sel + (uint32_t)s0c, g);
#pragma unroll
                    for (int v8 = 0; v8 < 2; ++v8) {
                        uint32_t ohi[4], olo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int s = s0c + v8 * 8 + 2 * e;
                            const float e0 = sWp[s * 128 + j] - g[v8 * 8 + 2 * e], e1 = sWp[(s + 1) * 128 + j] - g[v8 * 8 + 2 * e + 1];
                            split_bf16x2(e0, e1, ohi[e], olo[e]);
                        }
                        const uint32_t off = (tid & 7) * 16 + (tid >> 3) * SBO + (uint32_t)(s0c / 8 + v8) * LBO_M;
                        *reinterpret_cast<uint4*>(ehi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                        *reinterpret_cast<uint4*>(elo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
                    }
                }
                for (int idx = tid; idx < n_pad * 16; idx += kTcThreads) {
                    const int a = (idx >> 3) & 15, s = (idx & 7) + 8 * (idx >> 7);
                    const uint4 kraw = *reinterpret_cast<const uint4*>(sKraw + (size_t)s * kRowB + a * 16);
                    const float w = sDn[s];
                    const uint32_t vin[4] = {kraw.x, kraw.y, kraw.z, kraw.w};
                    uint32_t ohi[4], olo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        split_bf16x2(w * __uint_as_float(vin[e] << 16), w * __uint_as_float(vin[e] & 0xffff0000u), ohi[e], olo[e]);
                    const uint32_t off = (s & 7) * 16 + a * SBO + (s >> 3) * LBO_M;
                    *reinterpret_cast<uint4*>(lhi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                    *reinterpret_cast<uint4*>(llo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
                }
                proxy_fence();
                tc_fence_before();
                __syncthreads();
                if (tid == 0) {
                    tc_fence_after();
                    for (int ks = 0; ks < n_pad / 16; ++ks) {
                        const uint64_t dehi = make_desc(smem_u32(ehi) + ks * 2 * LBO_M, LBO_M, SBO);
                        const uint64_t delo = make_desc(smem_u32(elo) + ks * 2 * LBO_M, LBO_M, SBO);
                        const uint64_t dlhi = make_desc(smem_u32(lhi) + ks * 2 * LBO_M, LBO_M, SBO);
                        const uint64_t dllo = make_desc(smem_u32(llo) + ks * 2 * LBO_M, LBO_M, SBO);
                        tc_mma_bf16(tmem_t, dehi, dlhi, idescC, ks ? 1u : 0u);
                        tc_mma_bf16(tmem_t, delo, dlhi, idescC, 1u);
                        tc_mma_bf16(tmem_t, dehi, dllo, idescC, 1u);
                    }
                    tc_commit(&bars[0]);
                }
                if (!mbar_wait_bounded(&bars[0], ph0)) { record_fault(p.status, kFaultUpdateWait, 14); dead = true; }
                ph0 ^= 1;
                tc_fence_after();
            }
        }
        dead = __syncthreads_or(dead ? 1 : 0) != 0;
        if (dead) break;

        // ---- epilogue C: S_new = d S_0 + T, written back; S_new hi/lo -> MMA 2 ([U | o] = S_new^T [Omega | q]) ----
        const float* Sg = p.state + bh * (size_t)K * V + j;
        float* So = p.state + bh * (size_t)K * V + j;
        float s0[kChunk];
#pragma unroll
        for (int ii = 0; ii < kChunk; ++ii) s0[ii] = Sg[(size_t)ii * V];
        for (int c = 0; c < K / kChunk; ++c) {
            float s0n[kChunk];
            if (c + 1 < K / kChunk) {
#pragma unroll
                for (int ii = 0; ii < kChunk; ++ii) s0n[ii] = Sg[(size_t)((c + 1) * kChunk + ii) * V];
            }
            float t[kChunk];
            if (n_tot > 0) {
                tmem_ld32(tmem_t + lane_sel + (uint32_t)(c * kChunk), t);
            } else {
#pragma unroll
                for (int ii = 0; ii < kChunk; ++ii) t[ii] = 0.f;
            }
            if (c >= 2) {
                if (!mbar_wait_bounded(&bars[1 + (c & 1)], ph1[c & 1])) { record_fault(p.status, kFaultUpdateWait, 15); dead = true; }
                ph1[c & 1] ^= 1;
            }
            unsigned char* a2hi = sR1 + (size_t)(c & 1) * 16384u;
            unsigned char* a2lo = a2hi + 8192u;
#pragma unroll
            for (int v8 = 0; v8 < kChunk / 8; ++v8) {
                uint32_t ohi[4], olo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i0 = v8 * 8 + 2 * e;
                    const float x0 = fmaf(dtot, s0[i0], t[i0]), x1 = fmaf(dtot, s0[i0 + 1], t[i0 + 1]);
                    if (p.write_state) {
                        So[(size_t)(c * kChunk + i0) * V] = x0;
                        So[(size_t)(c * kChunk + i0 + 1) * V] = x1;
                    }
                    split_bf16x2(x0, x1, ohi[e], olo[e]);
                }
                const uint32_t off = (tid & 7) * 16 + (tid >> 3) * SBO + v8 * LBO_M;
                *reinterpret_cast<uint4*>(a2hi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                *reinterpret_cast<uint4*>(a2lo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
            }
            proxy_fence();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < kChunk / 16; ++ks) {
                    const uint32_t kb = (uint32_t)(c * (kChunk / 8) + ks * 2) * LBO2B;
                    const uint64_t ahi = make_desc(smem_u32(a2hi) + ks * 2 * LBO_M, LBO_M, SBO);
                    const uint64_t alo = make_desc(smem_u32(a2lo) + ks * 2 * LBO_M, LBO_M, SBO);
                    const uint64_t bhi = make_desc(smem_u32(sB2hi) + kb, LBO2B, SBO);
                    const uint64_t blo = make_desc(smem_u32(sB2lo) + kb, LBO2B, SBO);
                    tc_mma_bf16(tmem_u, ahi, bhi, idesc2, (c | ks) ? 1u : 0u);
                    tc_mma_bf16(tmem_u, alo, bhi, idesc2, 1u);
                    tc_mma_bf16(tmem_u, ahi, blo, idesc2, 1u);
                }
                tc_commit(c + 1 < K / kChunk ? &bars[1 + (c & 1)] : &bars[3]);
            }
            if (c + 1 < K / kChunk) {
#pragma unroll
                for (int ii = 0; ii < kChunk; ++ii) s0[ii] = s0n[ii];
            }
        }
        if (!mbar_wait_bounded(&bars[1], ph1[0])) { record_fault(p.status, kFaultUpdateWait, 16); dead = true; }
        ph1[0] ^= 1;
        if (!mbar_wait_bounded(&bars[3], ph3)) { record_fault(p.status, kFaultUpdateWait, 17); dead = true; }
        ph3 ^= 1;
        tc_fence_after();

        for (int g0 = 0; g0 < NP; g0 += 16) {
            float u[16];
            tmem_ld16(tmem_u + lane_sel + (uint32_t)g0, u);
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int g = g0 + e;
                if (g < R && p.write_sketch) p.sketch[(bh * R + g) * (size_t)V + j] = u[e];
                if (g == R && p.out != nullptr) {
                    if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[bh * V + j] = __float2bfloat16_rn(u[e]);
                    else reinterpret_cast<float*>(p.out)[bh * V + j] = u[e];
                }
            }
        }
        tc_fence_before();
        dead = __syncthreads_or(dead ? 1 : 0) != 0;
        tc_fence_after();
    }

    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// Returns SKETCHSSM_UNSUPPORTED_SHAPE outside this kernel's domain.
int launch_update_tc_delta(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    if (c.kind != SKETCHSSM_GDN || c.io_dtype != SKETCHSSM_BF16 || c.dk != kK || c.dv != 128) return SKETCHSSM_UNSUPPORTED_SHAPE;
    Params p = p_in;
    const int n_tot = p.n_before + (p.has_token ? 1 : 0);
    if (n_tot > kMaxTok) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const int NP = (c.rank + 1 + 15) & ~15;
    if (NP > 128) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (ctx->sm_count == 0) {
        int dev = 0, sms = 0;
        if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        if ((ctx->last_cuda_error = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
        ctx->sm_count = sms;
    }
    const DSmem sm = make_dsmem(NP);
    const int tmem_cols = NP <= 32 ? 128 : 256;
    int ctas = (int)((228u * 1024u) / (sm.total + 1024u));
    if (ctas > 512 / tmem_cols) ctas = 512 / tmem_cols;
    if (ctas > 4) ctas = 4;
    if (ctas < 1) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const long long n_tiles = (long long)c.batch * c.heads;
    long long grid = (long long)ctx->sm_count * ctas;
    if (grid > n_tiles) grid = n_tiles;
    auto kern = update_tc_gdn_kernel;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    if ((ctx->last_cuda_error = launch_kernel(kern, dim3((unsigned)grid), dim3(kTcThreads), sm.total, stream, p, p.pdl != 0)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

}  // namespace sketchssm
