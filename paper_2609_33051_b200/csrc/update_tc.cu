// State-update (flush) kernel on the 5th-generation tensor cores (tcgen05 + TMEM), sm_100a.
//
// Mamba-2 transition (M_t = D_t = a_t I): the replay of n buffered tokens is the closed form of Eq. 3
//     S_new = d S_0 + sum_s (beta_s prod_{j>s} a_j) k_s v_s^T,   d = prod_j a_j,
// a rank-n update, and the sketch rows and the exact output are one more contraction over the state rows,
//     U[g, :] = S_new^T omega_g  (Eq. 7),   o = S_new^T q.
// Both contractions run as tcgen05.mma with fp32 accumulators in tensor memory; the fp32 state itself only
// ever passes through registers once (read S_0, fused multiply-add with the accumulator, write S_new), so S is
// streamed from HBM exactly once per update.
//
// Tile: 128 TMEM lanes = the value columns j of one head (V = 128) or of two heads of the same head index
// (V = 64, block-diagonal operand); TMEM columns = the state rows i (K = 128).  Thread t owns lane t.
//   MMA 1 (kind::f16, bf16 x bf16 -> fp32):  T[t, i] = sum_s w_s v_s[j(t)] k_s[i]
//       A = w_s v_s split into bf16 hi + lo (w_s is fp32), B = the raw bf16 keys: exact products, fp32 sums
//   epilogue: S_new[i, j] = d S_0[i, j] + T[t, i]  (coalesced global loads/stores, one element per thread and row),
//       S_new split into bf16 hi + lo and written to shared memory as the A operand of MMA 2, 32 rows at a time
//   MMA 2: UT[t, g] = sum_i S_new[i, j(t)] W[i, g],  W = [Omega | q] split hi + lo; three products
//       (hi*hi + lo*hi + hi*lo) keep ~16 mantissa bits, accumulated in fp32
// Operands use the no-swizzle canonical shared-memory layouts (8 x 16-byte core matrices).
#include "internal.cuh"
#include "tc_common.cuh"

namespace sketchssm {

namespace {

using namespace tc;


struct TcSmem {
    uint32_t a1_hi, a1_lo, b1, a2, b2_hi, b2_lo, w, stg, stg_head, bars, tmem_slot, total;
};

__host__ __device__ inline TcSmem make_tc_smem(int NH, int NP, int V = 64, int L = 16) {
    TcSmem s;
    const uint32_t kd1 = (uint32_t)(kTokBlock * NH);
    uint32_t off = 0;
    // the MMA-1 operands are dead once MMA 1 has completed, before the epilogue writes the MMA-2 chunk buffers:
    // both live in the same region
    s.a1_hi = off;
    s.a1_lo = off + 128u * kd1 * 2u;
    s.b1 = off + 2u * 128u * kd1 * 2u;
    s.a2 = off;
    const uint32_t mma1_bytes = 3u * 128u * kd1 * 2u, mma2_bytes = 2u * 2u * 128u * 16u * 2u;   // two 16-row chunk buffers, hi + lo
    off += mma1_bytes > mma2_bytes ? mma1_bytes : mma2_bytes;
    s.b2_hi = off; off += (uint32_t)NP * kK * 2u;
    s.b2_lo = off; off += (uint32_t)NP * kK * 2u;
    s.w = off; off += 2u * 208u * 4u;                    // per head: w_s (64), total decay (16), beta_s (64), a_s (64)
    // staging of the next tile's raw ring rows (first token block): per head keys [16][256 B], values [16][V*2 B], gates [2L] floats
    s.stg_head = 16u * 256u + 16u * (uint32_t)V * 2u + (((uint32_t)(2 * L * 4) + 127u) & ~127u);
    s.stg = off; off += (uint32_t)NH * s.stg_head;
    s.bars = off; off += 64u;
    s.tmem_slot = off; off += 64u;
    s.total = off;
    return s;
}

}  // namespace

// V = 128: one head per tile; V = 64: two heads (same head index, consecutive batch entries) per tile.
template <int V>
__global__ void __launch_bounds__(kTcThreads) update_tc_mamba2_kernel(const Params p) {
    constexpr int K = kK;
    constexpr int NH = 128 / V;
    constexpr int KD1 = kTokBlock * NH;                 // contraction length of one MMA-1 block
    extern __shared__ __align__(1024) unsigned char smem[];

    const int tid = threadIdx.x, warp = tid >> 5;
    const int R = p.R, H = p.H, B = p.B;
    const int NP = (R + NH + 15) & ~15;                   // sketch ranks + one query column per head, padded
    const int n_ring = p.n_before, n_tot = n_ring + (p.has_token ? 1 : 0);
    const TcSmem sm = make_tc_smem(NH, NP, V, p.L);
    __nv_bfloat16* sA1hi = reinterpret_cast<__nv_bfloat16*>(smem + sm.a1_hi);
    __nv_bfloat16* sA1lo = reinterpret_cast<__nv_bfloat16*>(smem + sm.a1_lo);
    __nv_bfloat16* sB1 = reinterpret_cast<__nv_bfloat16*>(smem + sm.b1);
    unsigned char* sA2 = smem + sm.a2;
    __nv_bfloat16* sB2hi = reinterpret_cast<__nv_bfloat16*>(smem + sm.b2_hi);
    __nv_bfloat16* sB2lo = reinterpret_cast<__nv_bfloat16*>(smem + sm.b2_lo);
    float* sW = reinterpret_cast<float*>(smem + sm.w);
    unsigned char* sStg = smem + sm.stg;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);     // [0] MMA 1, [1..2] MMA 2 chunk buffers, [3] MMA 2 all, [4] staging
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + sm.tmem_slot);

    const uint32_t tmem_cols = NP <= 32 ? 128u : 256u;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int i = 0; i < 5; ++i) mbar_init(&bars[i], 1);
        mbar_fence_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    grid_dep_wait();                 // nothing above reads memory another kernel may write
    grid_dep_launch_dependents();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_t = tmem_base;                          // T: 128 columns
    const uint32_t tmem_u = tmem_base + (NP <= 32 ? 0u : 128u); // UT: NP columns (re-uses consumed T columns if it fits)
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;

    // instruction descriptors: bf16 x bf16 -> fp32
    const uint32_t idesc1 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
    const uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)NP >> 3) << 17) | ((128u >> 4) << 24);

    // canonical no-swizzle layouts (byte offsets)
    //   MN-major (MMA 1): elem(mn, k) at (k%8)*16 + (mn%8)*2 + (mn/8)*128 + (k/8)*2048
    //   K-major  (MMA 2): elem(mn, k) at (mn%8)*16 + (mn/8)*128 + (k/8)*LBO + (k%8)*2,  LBO = 16*MN
    constexpr uint32_t LBO1 = 2048, SBO = 128;
    constexpr uint32_t LBO2A = 2048;
    const uint32_t LBO2B = (uint32_t)NP * 16u;

    const int tiles_per_h = B / NH;
    const long long n_tiles = (long long)H * tiles_per_h;
    const int tile0 = (int)(n_tiles * blockIdx.x / gridDim.x);
    const int tile1 = (int)(n_tiles * (blockIdx.x + 1) / gridDim.x);

    const int my_head = tid / V;          // which head of the tile this thread's lane belongs to
    const int j = tid % V;
    int cur_h = -1;
    uint32_t ph0 = 0, ph1[2] = {0, 0}, ph3 = 0, ph4 = 0;   // mbarrier phases
    bool dead = false;

    // Raw ring rows of a tile's first token block travel to shared memory by bulk copies issued one tile ahead, so that
    // building the MMA-1 operands never waits on global memory.  Rows of later blocks (n > 16) are read directly.
    const int rows0 = n_ring < kTokBlock ? n_ring : kTokBlock;
    const bool tok0 = p.has_token && n_ring < kTokBlock;
    const uint32_t stg_gate_bytes = n_ring > 0 ? (uint32_t)(2 * p.L * 4) : 0u;
    const uint32_t stg_bytes = (uint32_t)NH * ((uint32_t)rows0 * 256u + (uint32_t)rows0 * V * 2u + stg_gate_bytes +
                                              (tok0 ? 256u + (uint32_t)V * 2u : 0u));
    auto stage_tile = [&](int tile) {       // thread 0 only
        const int h = tile / tiles_per_h;
        const int b0 = (tile - h * tiles_per_h) * NH;
        mbar_expect_tx(&bars[4], stg_bytes);
        for (int hd = 0; hd < NH; ++hd) {
            const size_t bw = (size_t)(b0 + hd) * H + h;
            const unsigned char* rh = p.ring + bw * p.rl.head_bytes;
            unsigned char* dst = sStg + (size_t)hd * sm.stg_head;
            if (rows0 > 0) {
                bulk_g2s(dst, rh, (uint32_t)rows0 * 256u, &bars[4]);
                bulk_g2s(dst + 4096, rh + p.rl.v_off, (uint32_t)rows0 * V * 2u, &bars[4]);
            }
            if (stg_gate_bytes) bulk_g2s(dst + 4096 + 16 * V * 2, rh + p.rl.beta_off, stg_gate_bytes, &bars[4]);
            if (tok0) {
                bulk_g2s(dst + (size_t)n_ring * 256, reinterpret_cast<const __nv_bfloat16*>(p.k) + bw * K, 256u, &bars[4]);
                bulk_g2s(dst + 4096 + (size_t)n_ring * V * 2, reinterpret_cast<const __nv_bfloat16*>(p.v) + bw * V, (uint32_t)V * 2u, &bars[4]);
            }
        }
    };
    if (tid == 0 && stg_bytes > 0 && tile0 < tile1) stage_tile(tile0);

    for (int tile = tile0; tile < tile1 && !dead; ++tile) {
        const int h = tile / tiles_per_h;
        const int b0 = (tile - h * tiles_per_h) * NH;
        const size_t bh = (size_t)(b0 + my_head) * H + h;

        // ---- W = [Omega | q ...] hi/lo, K-major; Omega part once per head index ----
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
        if (p.q != nullptr) {       // query columns R .. R+NH-1 (bf16-exact: lo = 0)
            for (int idx = tid; idx < K * NH; idx += kTcThreads) {
                const int i = idx % K, hd = idx / K, g = R + hd;
                const size_t bq = (size_t)(b0 + hd) * H + h;
                const uint32_t o2 = ((g & 7) * 16 + (g >> 3) * SBO + (i >> 3) * LBO2B + (i & 7) * 2) >> 1;
                sB2hi[o2] = reinterpret_cast<const __nv_bfloat16*>(p.q)[bq * K + i];
            }
        }

        // ---- token weights w_s = beta_s prod_{j>s} a_j and the total decay ----
        // the staged rows and gates of this tile must have landed
        if (stg_bytes > 0) {
            if (!cta_wait(&bars[4], ph4)) { record_fault(p.status, kFaultUpdateWait, 6); dead = true; }
            ph4 ^= 1;
        }
        for (int idx = tid; idx < NH * 64; idx += kTcThreads) {
            const int hd = idx >> 6, s = idx & 63;
            if (s < n_tot) {
                const size_t bw = (size_t)(b0 + hd) * H + h;
                const float* sg = reinterpret_cast<const float*>(sStg + (size_t)hd * sm.stg_head + 4096 + 16 * V * 2);
                sW[hd * 208 + 80 + s] = s < n_ring ? sg[s] : p.beta[bw];
                sW[hd * 208 + 144 + s] = s < n_ring ? sg[p.L + s] : reinterpret_cast<const float*>(p.decay)[bw];
            }
        }
        __syncthreads();
        if (tid < NH) {
            float suf = 1.f;
            for (int s = n_tot - 1; s >= 0; --s) {
                sW[tid * 208 + s] = sW[tid * 208 + 80 + s] * suf;
                suf *= sW[tid * 208 + 144 + s];
            }
            sW[tid * 208 + 64] = suf;
        }
        const float* Sg = p.state + bh * (size_t)K * V + j;
        __syncthreads();

        // ---- MMA 1 over blocks of kTokBlock tokens per head ----
        const int n_blocks = (n_tot + kTokBlock - 1) / kTokBlock;
        for (int blk = 0; blk < n_blocks; ++blk) {
            if (blk > 0) {      // the previous block's MMAs must have read the operand buffers
                if (!cta_wait(&bars[0], ph0)) { record_fault(p.status, kFaultUpdateWait, 1); dead = true; }
                ph0 ^= 1;
                tc_fence_after();
            }
            // Operand rows are written 16 bytes per thread; consecutive threads walk the 8 token rows of a core matrix
            // first and then the next 8-element vector, so that a warp writes 512 contiguous bytes (no bank conflicts).
            // B operand: keys, MN-major (mn = state row i, k = token slot)
            for (int idx = tid; idx < KD1 * (K / 8); idx += kTcThreads) {
                const int a = (idx >> 3) % (K / 8), sp = (idx & 7) + 8 * (idx / (8 * (K / 8)));
                const int hd = sp / kTokBlock, s = blk * kTokBlock + sp % kTokBlock;
                const size_t bk = (size_t)(b0 + hd) * H + h;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (blk == 0) {
                    if (s < n_tot) val = *reinterpret_cast<const uint4*>(sStg + (size_t)hd * sm.stg_head + (size_t)s * 256 + a * 16);
                } else if (s < n_ring) {
                    val = *reinterpret_cast<const uint4*>(p.ring + bk * p.rl.head_bytes + ((size_t)s * K + a * 8) * 2);
                } else if (s < n_tot) {
                    val = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.k) + bk * K + a * 8);
                }
                *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(sB1) + (sp & 7) * 16 + a * SBO + (sp >> 3) * LBO1) = val;
            }
            // A operand: w_s v_s hi/lo, MN-major (mn = lane t = head*V + j, k = token slot), block diagonal over heads:
            // lanes of head hd see only the token rows of head hd, the other block is zero
            for (int idx = tid; idx < KD1 * 16; idx += kTcThreads) {
                const int a128 = (idx >> 3) & 15, sp = (idx & 7) + 8 * (idx >> 7);     // a128: vector index over all 128 lanes
                const int hd = sp / kTokBlock, s = blk * kTokBlock + sp % kTokBlock;
                const int hd_lane = a128 / (V / 8), a = a128 % (V / 8);
                const size_t bk = (size_t)(b0 + hd) * H + h;
                uint4 vraw = make_uint4(0, 0, 0, 0);
                float w = 0.f;
                if (hd_lane == hd) {
                    if (blk == 0) {
                        if (s < n_tot) {
                            vraw = *reinterpret_cast<const uint4*>(sStg + (size_t)hd * sm.stg_head + 4096 + (size_t)s * V * 2 + a * 16);
                            w = sW[hd * 208 + s];
                        }
                    } else if (s < n_ring) {
                        vraw = *reinterpret_cast<const uint4*>(p.ring + bk * p.rl.head_bytes + p.rl.v_off + ((size_t)s * V + a * 8) * 2);
                        w = sW[hd * 208 + s];
                    } else if (s < n_tot) {
                        vraw = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.v) + bk * V + a * 8);
                        w = sW[hd * 208 + s];
                    }
                }
                const uint32_t vin[4] = {vraw.x, vraw.y, vraw.z, vraw.w};
                uint32_t ohi[4], olo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float f0 = w * __uint_as_float(vin[e] << 16), f1 = w * __uint_as_float(vin[e] & 0xffff0000u);
                    split_bf16x2(f0, f1, ohi[e], olo[e]);
                }
                const uint32_t off = (sp & 7) * 16 + a128 * SBO + (sp >> 3) * LBO1;
                *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(sA1hi) + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(sA1lo) + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
            }
            proxy_fence();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                if (blk == 0 && stg_bytes > 0 && tile + 1 < tile1) stage_tile(tile + 1);   // staging is free again
#pragma unroll
                for (int ks = 0; ks < KD1 / 16; ++ks) {
                    const uint64_t bd = make_desc(smem_u32(sB1) + ks * 2 * LBO1, LBO1, SBO);
                    tc_mma_bf16(tmem_t, make_desc(smem_u32(sA1hi) + ks * 2 * LBO1, LBO1, SBO), bd, idesc1, (blk | ks) ? 1u : 0u);
                    tc_mma_bf16(tmem_t, make_desc(smem_u32(sA1lo) + ks * 2 * LBO1, LBO1, SBO), bd, idesc1, 1u);
                }
                tc_commit(&bars[0]);
            }
        }
        if (n_blocks > 0) {
            if (!cta_wait(&bars[0], ph0)) { record_fault(p.status, kFaultUpdateWait, 2); dead = true; }
            ph0 ^= 1;
            tc_fence_after();
        }
        if (dead) break;

        // ---- epilogue: S_new = d S_0 + T, written back; S_new hi/lo -> A operand of MMA 2, 16 rows at a time ----
        // The state rows of the next two chunks are in flight in registers while a chunk is processed.
        const float dtot = n_tot > 0 ? sW[my_head * 208 + 64] : 1.f;
        float* So = p.state + bh * (size_t)K * V + j;
        constexpr int CH = 16, NCH = K / CH, PF = 2;
        float sbuf[PF + 1][CH];
#pragma unroll
        for (int c = 0; c < PF; ++c) {
#pragma unroll
            for (int ii = 0; ii < CH; ++ii) sbuf[c][ii] = Sg[(size_t)(c * CH + ii) * V];
        }
        float t01[2 * CH];      // T columns of chunks 0 and 1: both are read before the first MMA 2 overwrites them with UT
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            if (c + PF < NCH) {
#pragma unroll
                for (int ii = 0; ii < CH; ++ii) sbuf[(c + PF) % (PF + 1)][ii] = Sg[(size_t)((c + PF) * CH + ii) * V];
            }
            float t[CH];
            if (n_blocks > 0) {
                if (c == 0) tmem_ld32(tmem_t + lane_sel, t01);
                if (c < 2) {
#pragma unroll
                    for (int ii = 0; ii < CH; ++ii) t[ii] = t01[c * CH + ii];
                } else {
                    tmem_ld16(tmem_t + lane_sel + (uint32_t)(c * CH), t);
                }
            } else {
#pragma unroll
                for (int ii = 0; ii < CH; ++ii) t[ii] = 0.f;
            }
            if (c >= 2) {       // chunk buffer c&1 was read by the MMAs of chunk c-2
                if (!cta_wait(&bars[1 + (c & 1)], ph1[c & 1])) { record_fault(p.status, kFaultUpdateWait, 3); dead = true; }
                ph1[c & 1] ^= 1;
            }
            unsigned char* a2hi = sA2 + (size_t)(c & 1) * (2u * 128u * CH * 2u);
            unsigned char* a2lo = a2hi + 128u * CH * 2u;
#pragma unroll
            for (int v8 = 0; v8 < CH / 8; ++v8) {
                uint32_t ohi[4], olo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i0 = v8 * 8 + 2 * e;
                    const float x0 = fmaf(dtot, sbuf[c % (PF + 1)][i0], t[i0]), x1 = fmaf(dtot, sbuf[c % (PF + 1)][i0 + 1], t[i0 + 1]);
                    if (p.write_state) {
                        So[(size_t)(c * CH + i0) * V] = x0;
                        So[(size_t)(c * CH + i0 + 1) * V] = x1;
                    }
                    split_bf16x2(x0, x1, ohi[e], olo[e]);
                }
                const uint32_t off = (tid & 7) * 16 + (tid >> 3) * SBO + v8 * LBO2A;
                *reinterpret_cast<uint4*>(a2hi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                *reinterpret_cast<uint4*>(a2lo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
            }
            proxy_fence();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                const uint32_t kb = (uint32_t)(c * (CH / 8)) * LBO2B;      // W rows of this K-step
                const uint64_t ahi = make_desc(smem_u32(a2hi), LBO2A, SBO);
                const uint64_t alo = make_desc(smem_u32(a2lo), LBO2A, SBO);
                const uint64_t bhi = make_desc(smem_u32(sB2hi) + kb, LBO2B, SBO);
                const uint64_t blo = make_desc(smem_u32(sB2lo) + kb, LBO2B, SBO);
                tc_mma_bf16(tmem_u, ahi, bhi, idesc2, c ? 1u : 0u);
                tc_mma_bf16(tmem_u, alo, bhi, idesc2, 1u);
                tc_mma_bf16(tmem_u, ahi, blo, idesc2, 1u);
                tc_commit(c + 1 < NCH ? &bars[1 + (c & 1)] : &bars[3]);
            }
        }
        // drain: the final commit covers every MMA issued so far; chunk 6's commit on bars[1] completed with it
        if (!cta_wait(&bars[3], ph3)) { record_fault(p.status, kFaultUpdateWait, 5); dead = true; }
        ph3 ^= 1;
        ph1[0] ^= 1;
        tc_fence_after();

        // ---- UT rows -> sketch and exact output ----
        for (int g0 = 0; g0 < NP; g0 += 16) {
            float u[16];
            tmem_ld16(tmem_u + lane_sel + (uint32_t)g0, u);
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int g = g0 + e;
                if (g < R && p.write_sketch) store_sketch(p, (bh * R + g) * (size_t)V + j, u[e]);
                if (g == R + my_head && p.out != nullptr) {
                    if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[bh * V + j] = __float2bfloat16_rn(u[e]);
                    else reinterpret_cast<float*>(p.out)[bh * V + j] = u[e];
                }
            }
        }
        tc_fence_before();
        dead = __syncthreads_or(dead ? 1 : 0) != 0;   // T / UT are free again; also publishes any fault
        tc_fence_after();
    }

    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// Returns SKETCHSSM_UNSUPPORTED_SHAPE when the configuration is outside this kernel's domain (the caller then
// uses the CUDA-core kernel).
int launch_update_tc(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    if (c.kind != SKETCHSSM_MAMBA2 || c.io_dtype != SKETCHSSM_BF16 || c.dk != kK) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (c.dv != 64 && c.dv != 128) return SKETCHSSM_UNSUPPORTED_SHAPE;       // a tile is 128 value columns: two heads of 64 or one of 128
    if (p_in.n_dev != nullptr) return SKETCHSSM_UNSUPPORTED_SHAPE;            // per-sequence phases: CUDA-core kernel
    const int NH = 128 / c.dv;
    if (c.batch % NH != 0) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const int NP = (c.rank + NH + 15) & ~15;
    if (NP > 128) return SKETCHSSM_UNSUPPORTED_SHAPE;
    Params p = p_in;
    if (ctx->sm_count == 0) {
        int dev = 0, sms = 0;
        if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        if ((ctx->last_cuda_error = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
        ctx->sm_count = sms;
    }
    const TcSmem sm = make_tc_smem(NH, NP, c.dv, c.buf_len);
    const int tmem_cols = NP <= 32 ? 128 : 256;
    int ctas = (int)((228u * 1024u) / (sm.total + 1024u));
    if (ctas > 512 / tmem_cols) ctas = 512 / tmem_cols;     // tensor memory: 512 columns per SM
    if (ctas > 4) ctas = 4;
    if (p.max_warps_per_sm > 0 && ctas > p.max_warps_per_sm / 4) ctas = p.max_warps_per_sm / 4 > 0 ? p.max_warps_per_sm / 4 : 1;
    const long long n_tiles = (long long)c.batch * c.heads / NH;
    long long grid = (long long)ctx->sm_count * ctas;
    if (grid > n_tiles) grid = n_tiles;
    auto kern = c.dv == 128 ? update_tc_mamba2_kernel<128> : update_tc_mamba2_kernel<64>;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)sm.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    if ((ctx->last_cuda_error = launch_kernel(kern, dim3((unsigned)grid), dim3(kTcThreads), sm.total, stream, p, p.pdl != 0)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

}  // namespace sketchssm
