// Warp-specialised state-update (flush) kernel for the delta rule with per-channel decay (KDA) on tcgen05 + TMEM, sm_100a.
//
// Replaying n tokens of S_s = (I - beta_s k_s k_s^T) Diag(g_s) S_{s-1} + beta_s k_s v_s^T (Eq. 1, 3) unrolled over the
// window -- the WY form of Appendix C (Eq. 38-42) applied to the state, with the diagonal decays kept as vectors:
//     G_s   = prod_{m<=s} g_m (per channel),   Dn_s = prod_{m>s} g_m
//     Khat_s = G_s * k_s,   Ktil_s = Dn_s * k_s                  n x K     decayed keys (fp32 values: bf16 hi + lo)
//     A_sj  = sum_i k_s[i] k_j[i] prod_{j<m<=s} g_m[i]  (j < s)  n x n     every product of decays formed by multiplication
//     P     = Khat S_0                                           n x V
//     E     = T (V - P),   T = (I + Bd A)^{-1} Bd                n x V
//     S_new = Diag(G_n) S_0 + Ktil^T E                           K x V
//     [U | o] = S_0^T (G_n * [Omega | q]) + E^T (Ktil [Omega | q])         (Eq. 7 and the exact output of the flush step)
// No quotient of cumulative decays is ever formed (they underflow within a window on real gates).
//
// Tile = one head (K = V = 128), TMEM lane = value column; the state is read once by bulk copies into a ring of
// shared-memory stages; the pass-A group splits the S_0 chunks into bf16 hi + lo and leaves G_n * S_0 in the accumulator
// of Ktil^T E (tcgen05.st); one thread issues every MMA; the pass-B group forms E, writes the accumulator (S_new) back
// and stores the sketch rows; the front group builds the ring-only operands two tiles ahead.  Up to 32 tokens per pass
// (the MMAs over tokens take two k-steps); both key operands and the basis operand are per tile and carry hi + lo
// halves, so the B operand of pass A is a double-buffered per-tile window [Khat (32 rows) | G_n * [Omega | q] (32 rows)].
// The kernel runs one CTA per SM (shared memory) and owns all 512 columns of tensor memory: two 64-column slots
// [P | U0] and two 128-column accumulators for alternating tiles, so pass A of tile k + 1 (issued before the E step of
// tile k) never waits for the write-back of tile k.
//
// Front group, 256 threads, thread = (token block, channel i): reads column i of its block's staged key and decay rows
// into registers, forms the running products and writes its rows of Khat / Ktil / G_n * W in the operand layouts.  The
// 32 x 32 system is handled as two blocks of 16 tokens: the 120 pair sums inside a block are per-channel products of
// that block's threads reduced over the 128 channels by transposing butterflies (per-warp partials summed in a fixed
// order: results are bitwise reproducible); the 16 x 16 block that couples the two blocks is an mma.sync product of
// rescaled keys (the decay product splits at the block boundary without a quotient); T_11 and T_22 by forward
// substitution (one column per thread, one warp each) while six warps form Ktil [Omega | q] with mma.sync.  The E step
// (E_1 = T_11 x_1, E_2 = T_22 (x_2 - A_21 E_1), 528 multiply-adds per lane) runs on the pass-B group, between the
// write-back of one tile and the next, so that the pass-A group only streams.
//
// Domain: KDA, bf16 I/O, K = V = 128, rank <= 16; 1..32 tokens per pass, up to 64 tokens per flush in blocks of 32.
#include <type_traits>
#include "internal.cuh"
#include "lanegroup.cuh"
#include "tc_common.cuh"

namespace sketchssm {

namespace {

using namespace tc;

constexpr int kKThreads = 576;       // pass-A group (4 warps), front group part 1 (4 warps), MMA issue warp, state-load warp, pass-B group (4 warps), front group part 2 (4 warps)
constexpr int kKFront = 256;         // threads of the front group
constexpr int kNT = 32;              // tokens per pass
constexpr int kKStages = 8;          // upper bound on the shared-memory stages of state rows
constexpr int kAS = 36;              // (sizes the work area of A: 32 rows of 36 floats)
constexpr int kAS2 = 20;             // row stride (floats) of the two 16 x 16 triangles of A
constexpr uint32_t kZPitch = 272u;   // bytes between the rows of the rescaled keys Z[token][channel]: 256 + 16, so that the 8 rows of an ldmatrix fall in different banks
constexpr uint32_t kZHalf = 32u * kZPitch;   // hi rows, then lo rows
// Pass-A window [Khat 32 | G_n * W 32]: 64 rows of 16 bytes per group of 8 channels, the groups 16 bytes further apart than
// they need to be, so that the per-channel threads of a warp (4 groups) store to different banks
constexpr uint32_t kLboW = 64u * 16u + 16u;
// Ktil operand (MN-major: 8 channels x 8 tokens per core matrix): the four token groups of a channel group lie side by
// side and the channel groups 16 bytes further apart than that, so the four channel groups a warp stores to for one
// token fall into different banks
constexpr uint32_t kLboT = 128u, kSboT = 4u * 128u + 16u, kKtHalf = (uint32_t)(kK / 8) * kSboT;
constexpr int kKA2 = 2;              // chunk buffers between the pass-A group and the MMA issue warp
constexpr int kNPk = 32;             // columns of [Omega | q]: Omega in 0..R-1, q at column QA = round_up(R, 8) <= 16

struct KSmem {
    uint32_t a2, e, w, w_stride, w_lo, set, set_stride, set_bt, set_bt_lo, set_vv, set_t1, set_bc, set_gn, stg, stg_g, stg_v,
        stg_beta, stg_q, mats, om, bars, misc, sst, sst_bytes, total;
};

__host__ __device__ inline KSmem make_ksmem(int stages) {
    KSmem s;
    uint32_t off = 0;
    s.a2 = off; off += (uint32_t)kKA2 * 2u * 128u * 16u * 2u;     // 16-row chunk buffers, hi + lo
    s.e = off; off += 2u * 128u * (uint32_t)kNT * 2u;             // E hi + lo: A operand of Ktil^T E (128 x 32 tokens each)
    // B operand of pass A, per tile and double-buffered: 64 rows [Khat (32) | G_n * [Omega | q] (32)] x 128 channels, hi then lo
    s.w = off; s.w_lo = (uint32_t)(kK / 8) * kLboW; s.w_stride = 2u * s.w_lo; off += 2u * s.w_stride;
    // per-tile operand set, double-buffered: Ktil as B operand of Ktil^T E (MN-major, hi | lo), raw value rows, T,
    // Ktil [Omega | q] hi | lo (B operand of the sketch correction), G_n
    s.set = off;
    s.set_bt = 0u; s.set_bt_lo = kKtHalf; s.set_vv = 2u * kKtHalf; s.set_t1 = s.set_vv + 8192u; s.set_bc = s.set_t1 + 4096u;
    s.set_gn = s.set_bc + 4096u;
    s.set_stride = s.set_gn + 512u;
    off += 2u * s.set_stride;
    // staging of the next tile's raw rows: keys [32][256 B], decays [32][256 B], values [32][256 B], beta [L] floats, query row.
    // Once a tile's rows are in registers the key / decay area is re-used (A partials, then Ktil in fp32).
    s.stg_g = 8192u; s.stg_v = 16384u; s.stg_beta = 24576u; s.stg_q = 24832u;
    s.stg = off; off += 25088u;
    s.mats = off; off += (uint32_t)kNT * kAS * 4u + 256u;         // A (beta_s A_sj), beta
    s.om = off; off += (uint32_t)kK * 16u * 4u;                   // Omega of the current head index, fp32 [K][16] (zero beyond the rank)
    s.bars = off; off += 512u;
    s.misc = off; off += 128u;
    off = (off + 127u) & ~127u;
    s.sst_bytes = 16u * 128u * 4u;
    s.sst = off; off += (uint32_t)stages * s.sst_bytes;
    s.total = off;
    return s;
}

enum { kPro = 0, kPfull = 2, kTfull = 4, kBdone = 6, kBufFree = 8, kA2free = 10, kA2rdy = 10 + kKA2, kErdy = 10 + 2 * kKA2,
       kStg = 11 + 2 * kKA2, kStDone = 12 + 2 * kKA2, kFull = 14 + 2 * kKA2, kEmpty = 14 + 2 * kKA2 + kKStages,
       kTfree = 14 + 2 * kKA2 + 2 * kKStages, kNumBars = 16 + 2 * kKA2 + 2 * kKStages };

__device__ __forceinline__ void k_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// named barrier 2 over the 256 threads of the front group, and a group-wide bounded wait: one warp polls, the others
// sleep in the barrier
__device__ __forceinline__ void f_sync() { asm volatile("bar.sync 2, 256;" ::: "memory"); }
__device__ __forceinline__ bool f_wait(int ft, uint64_t* bar, uint32_t phase) {
    bool bad = false;
    if (ft < 32) bad = !mbar_wait_bounded(bar, phase);
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 2, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(bad ? 1u : 0u)
        : "memory");
    return r == 0;
}
__device__ __forceinline__ void k_ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void k_ldmatrix_x2(uint32_t addr, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void k_mma_16816(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__device__ __forceinline__ float bf16_at(const unsigned char* base, uint32_t elem) {
    return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[elem]);
}

}  // namespace

__global__ void __launch_bounds__(kKThreads, 1) update_tc_ws_kda_kernel(const Params p) {
    constexpr int K = kK, V = 128, CH = 16, NCH = K / CH, NP = kNPk;
    extern __shared__ __align__(1024) unsigned char smem[];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gt = tid & 127;
    const int R = p.R, H = p.H, B = p.B;
    const int QA = (R + 7) & ~7;                          // column of the query
    const int NS = p.stages;
    const int n_ring = p.n_before, n_tot = n_ring + (p.has_token ? 1 : 0);     // 1..32 per pass (the launcher sees to it)
    const int ksteps = n_tot > 16 ? 2 : 1;                // 16-token k-steps of the MMAs that contract over tokens
    const KSmem sm = make_ksmem(NS);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + sm.misc);
    unsigned char* sStg = smem + sm.stg;

    constexpr uint32_t tmem_cols = 512u;          // one CTA per SM (shared memory): two slots of 64 columns, two accumulators of 128
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        *reinterpret_cast<volatile int*>(smem + sm.misc + 32) = 0;
        for (int i = 0; i < kNumBars; ++i) {
            // one arrival per warp of a stream group: chunk ready, E ready, stage empty, accumulator halves, pass-B done, slot free
            const bool per_warp = (i >= kA2rdy && i <= kErdy) || i == kStDone || i == kStDone + 1 || i >= kEmpty || (i >= kBdone && i < kBdone + 4);
            mbar_init(&bars[i], per_warp ? 4 : 1);
        }
        mbar_fence_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    grid_dep_wait();                 // nothing above reads memory another kernel may write
    grid_dep_launch_dependents();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;

    // instruction descriptors: bf16 x bf16 -> fp32, M = 128
    const uint32_t idescT = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);    // K-major x MN-major, N = 128
    const uint32_t idescU = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)NP >> 3) << 17) | ((128u >> 4) << 24);        // K-major x K-major, N = 32
    const uint32_t idescA = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);                 // K-major x K-major, N = 64
    // canonical no-swizzle layouts (byte offsets)
    //   K-major : elem(mn, k) at (mn%8)*16 + (mn/8)*128 + (k/8)*LBO + (k%8)*2,  LBO = 16*MN
    //   MN-major: elem(mn, k) at (k%8)*16 + (mn%8)*2 + (mn/8)*128 + (k/8)*2048
    constexpr uint32_t SBO = 128, LBO_M = 2048;
    constexpr uint32_t LBO_W = kLboW;                     // pass-A window: 64 rows (+ 16 bytes of padding)
    constexpr uint32_t LBO_C = (uint32_t)NP * 16u;        // Ktil W: 32 rows

    const int tiles_per_h = B;

    // the CTA's sequence of tile numbers (claimed at run time by the front group) travels through a small ring
    volatile int* seq_ring = reinterpret_cast<volatile int*>(smem + sm.misc + 16);
    volatile int* seq_pub = reinterpret_cast<volatile int*>(smem + sm.misc + 32);
    auto seq_get = [&](int k) -> int {          // -2: the wait ran out
        for (uint32_t it = 0; it < (1u << 22); ++it) {
            if (*seq_pub > k) {
                __threadfence_block();
                return seq_ring[k & 3];
            }
            if (it > 32) __nanosleep(100);
        }
        return -2;
    };
    auto set_ptr = [&](int b) { return smem + sm.set + (uint32_t)b * sm.set_stride; };
    auto w_ptr = [&](int b) { return smem + sm.w + (uint32_t)b * sm.w_stride; };

    const int j = (warp & 3) * 32 + lane;      // value column = TMEM lane of this thread (both stream groups)

    if (warp < 4) {
        // =========================== pass-A group: S_0 chunks -> operands, and the E step ===========================
        uint32_t phPro = 0, phA = 0, phF = 0;
        int gc = 0, stage = 0;
        bool bad = false;

        uint32_t phTf = 0;
        // pass A of the CTA's tile number kt with operand set b = kt & 1; the Ktil^T E accumulator b still holds tile kt - 2
        // until the pass-B group has read it
        auto pass_a = [&](int b, int kt) {
            const float* sGn = reinterpret_cast<const float*>(set_ptr(b) + sm.set_gn);
#pragma unroll 2
            for (int c = 0; c < NCH; ++c) {
                if (c == 0 && kt >= 2) {
                    bad |= !mbar_wait_bounded(&bars[kTfree + b], (phTf >> b) & 1u);
                    phTf ^= 1u << b;
                    tc_fence_after();
                }
                bad |= !mbar_wait_bounded(&bars[kFull + stage], phF);
                const float* sS = reinterpret_cast<const float*>(smem + sm.sst + (size_t)stage * sm.sst_bytes) + j;
                float s0[CH];
#pragma unroll
                for (int ii = 0; ii < CH; ++ii) s0[ii] = sS[ii * V];
                __syncwarp();
                if (lane == 0) k_arrive(&bars[kEmpty + stage]);
                {   // G_n * S_0 goes into the Ktil^T E accumulator, so that the MMAs leave S_new there
                    float ds[CH];
#pragma unroll
                    for (int i4 = 0; i4 < CH / 4; ++i4) {
                        const float4 g4 = *reinterpret_cast<const float4*>(sGn + c * CH + i4 * 4);
                        ds[i4 * 4 + 0] = g4.x * s0[i4 * 4 + 0];
                        ds[i4 * 4 + 1] = g4.y * s0[i4 * 4 + 1];
                        ds[i4 * 4 + 2] = g4.z * s0[i4 * 4 + 2];
                        ds[i4 * 4 + 3] = g4.w * s0[i4 * 4 + 3];
                    }
                    if (!bad) tmem_st16(tmem_base + 128u + (uint32_t)b * 128u + lane_sel + (uint32_t)(c * CH), ds);
                }
                const int ab = c & (kKA2 - 1);
                if (gc >= kKA2) {     // the chunk buffer was read by the MMAs issued kKA2 chunks ago
                    bad |= !mbar_wait_bounded(&bars[kA2free + ab], (phA >> ab) & 1u);
                    phA ^= 1u << ab;
                }
                unsigned char* a2hi = smem + sm.a2 + (size_t)ab * (2u * 128u * CH * 2u);
                unsigned char* a2lo = a2hi + 128u * CH * 2u;
#pragma unroll
                for (int v8 = 0; v8 < CH / 8; ++v8) {
                    uint32_t ohi[4], olo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) split_bf16x2(s0[v8 * 8 + 2 * e], s0[v8 * 8 + 2 * e + 1], ohi[e], olo[e]);
                    const uint32_t off = (gt & 7) * 16 + (gt >> 3) * SBO + v8 * LBO_M;
                    *reinterpret_cast<uint4*>(a2hi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                    *reinterpret_cast<uint4*>(a2lo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
                }
                proxy_fence();
                bad = __any_sync(0xffffffffu, bad);
                if (lane == 0 && !bad) k_arrive(&bars[kA2rdy + ab]);
                ++gc;
                if (++stage == NS) { stage = 0; phF ^= 1u; }
            }
            tmem_st_wait();            // this warp's G_n * S_0 columns are in tensor memory
            tc_fence_before();
            bad = __any_sync(0xffffffffu, bad);
            if (lane == 0 && !bad) k_arrive(&bars[kStDone + b]);
        };
        auto wait_pro = [&](int b) {
            bad |= !mbar_wait_bounded(&bars[kPro + b], (phPro >> b) & 1u);
            phPro ^= 1u << b;
        };

        int cur = seq_get(0);
        if (cur >= 0) {
            wait_pro(0);
            pass_a(0, 0);
            for (int k = 0; !bad; ++k) {
                const int b = k & 1;
                const int raw = seq_get(k + 1);
                if (raw < -1) { bad = true; break; }
                if (raw < 0) break;
                wait_pro(b ^ 1);
                pass_a(b ^ 1, k + 1);
            }
        } else if (cur < -1) {
            bad = true;
        }
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 103);
    } else if (warp >= 10 && warp < 14) {
        // =========================== pass-B group: S_new written back, then the sketch rows ===========================
        uint32_t phT = 0, phP = 0;
        bool bad = false;
        // E = T (V - P) with T = (I + Bd A)^{-1} Bd solved in two blocks of 16 tokens -> hi + lo A operand of Ktil^T E
        // (chunk-buffer layout, 32 tokens)
        auto do_e = [&](int b) {
            bad |= !mbar_wait_bounded(&bars[kPfull + b], (phP >> b) & 1u);
            phP ^= 1u << b;
            tc_fence_after();
            const unsigned char* set = set_ptr(b);
            const __nv_bfloat16* sV = reinterpret_cast<const __nv_bfloat16*>(set + sm.set_vv);
            const float* sT1 = reinterpret_cast<const float*>(set + sm.set_t1);
            float x[kNT];
            {
                float x0[16], x1[16];
                if (!bad) {
                    tmem_ld16(tmem_base + (uint32_t)b * 64u + lane_sel, x0);
                    tmem_ld16(tmem_base + (uint32_t)b * 64u + 16u + lane_sel, x1);
                } else {
#pragma unroll
                    for (int t = 0; t < 16; ++t) { x0[t] = 0.f; x1[t] = 0.f; }
                }
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    x[t] = __bfloat162float(sV[t * V + j]) - x0[t];
                    x[16 + t] = __bfloat162float(sV[(16 + t) * V + j]) - x1[t];
                }
            }
            // The 32 x 32 system in two blocks of 16 tokens:  E_1 = T_11 x_1,  E_2 = T_22 (x_2 - A_21 E_1)
            const float* sT11 = sT1;
            const float* sT22 = sT1 + 256;
            const float* sA21 = sT1 + 512;
            float e1[16], e2[16];
#pragma unroll
            for (int s = 0; s < 16; ++s) {
                float acc = 0.f;
#pragma unroll
                for (int t4 = 0; t4 <= s / 4; ++t4) {      // T_11 is lower triangular
                    const float4 tt = *reinterpret_cast<const float4*>(sT11 + s * 16 + t4 * 4);
                    acc = fmaf(tt.x, x[t4 * 4], acc);
                    acc = fmaf(tt.y, x[t4 * 4 + 1], acc);
                    acc = fmaf(tt.z, x[t4 * 4 + 2], acc);
                    acc = fmaf(tt.w, x[t4 * 4 + 3], acc);
                }
                e1[s] = acc;
            }
#pragma unroll
            for (int s = 0; s < 16; ++s) {
                float acc = x[16 + s];
#pragma unroll
                for (int t4 = 0; t4 < 4; ++t4) {
                    const float4 aa = *reinterpret_cast<const float4*>(sA21 + s * 16 + t4 * 4);
                    acc = fmaf(-aa.x, e1[t4 * 4], acc);
                    acc = fmaf(-aa.y, e1[t4 * 4 + 1], acc);
                    acc = fmaf(-aa.z, e1[t4 * 4 + 2], acc);
                    acc = fmaf(-aa.w, e1[t4 * 4 + 3], acc);
                }
                x[16 + s] = acc;
            }
#pragma unroll
            for (int s = 0; s < 16; ++s) {
                float acc = 0.f;
#pragma unroll
                for (int t4 = 0; t4 <= s / 4; ++t4) {      // T_22 is lower triangular
                    const float4 tt = *reinterpret_cast<const float4*>(sT22 + s * 16 + t4 * 4);
                    acc = fmaf(tt.x, x[16 + t4 * 4], acc);
                    acc = fmaf(tt.y, x[16 + t4 * 4 + 1], acc);
                    acc = fmaf(tt.z, x[16 + t4 * 4 + 2], acc);
                    acc = fmaf(tt.w, x[16 + t4 * 4 + 3], acc);
                }
                e2[s] = acc;
            }
            unsigned char* ehi = smem + sm.e;
            unsigned char* elo = ehi + 128u * (uint32_t)kNT * 2u;
#pragma unroll
            for (int v8 = 0; v8 < kNT / 8; ++v8) {
                uint32_t ohi[4], olo[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float ea = v8 < 2 ? e1[(v8 & 1) * 8 + 2 * q] : e2[(v8 & 1) * 8 + 2 * q];
                    const float eb = v8 < 2 ? e1[(v8 & 1) * 8 + 2 * q + 1] : e2[(v8 & 1) * 8 + 2 * q + 1];
                    split_bf16x2(ea, eb, ohi[q], olo[q]);
                }
                const uint32_t off = (gt & 7) * 16 + (gt >> 3) * SBO + v8 * LBO_M;
                *reinterpret_cast<uint4*>(ehi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                *reinterpret_cast<uint4*>(elo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
            }
            proxy_fence();
            tc_fence_before();
            bad = __any_sync(0xffffffffu, bad);
            if (lane == 0 && !bad) k_arrive(&bars[kErdy]);
        };
        int raw = seq_get(0);
        if (raw >= 0) do_e(0);
        else bad = raw < -1;
        for (int k = 0; !bad && raw >= 0; ++k) {
            const int tile = raw;
            const int b = k & 1;
            const int h = tile / tiles_per_h, bb = tile - h * tiles_per_h;
            const size_t bh = (size_t)bb * H + h;
            float* So = p.state + bh * (size_t)K * V + j;
            bad |= !mbar_wait_bounded(&bars[kTfull + b], (phT >> b) & 1u);      // Ktil^T E and the sketch correction are complete
            phT ^= 1u << b;
            tc_fence_after();
#pragma unroll 2
            for (int c = 0; c < NCH; ++c) {
                if (!bad) {
                    float t[CH];
                    tmem_ld16(tmem_base + 128u + (uint32_t)b * 128u + lane_sel + (uint32_t)(c * CH), t);
                    if (c == NCH - 1) {      // this warp is done with the accumulator: pass A of tile k + 2 may overwrite it
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) k_arrive(&bars[kTfree + b]);
                    }
#pragma unroll
                    for (int ii = 0; ii < CH; ++ii) So[(size_t)(c * CH + ii) * V] = t[ii];
                }
            }
            bad = __any_sync(0xffffffffu, bad);
            // [U | o] = S_0^T (G_n * W) + E^T (Ktil W) from the tile's slot of tensor memory: [correction 32 | U0 32]
            if (!bad) {
                const uint32_t slot = tmem_base + (uint32_t)b * 64u + lane_sel;
                auto rows = [&](auto bf) {
                    constexpr bool BF = decltype(bf)::value;
                    const size_t base = (bh * R) * (size_t)V + j;
                    for (int g0 = 0; g0 < R; g0 += 16) {
                        float u0[16], cr[16];
                        tmem_ld16(slot + 32u + (uint32_t)g0, u0);
                        tmem_ld16(slot + (uint32_t)g0, cr);
                        if (g0 + 16 <= R) {
#pragma unroll
                            for (int e = 0; e < 16; ++e) store_sketch_as<BF>(p, base + (size_t)(g0 + e) * V, u0[e] + cr[e]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 16; ++e)
                                if (g0 + e < R) store_sketch_as<BF>(p, base + (size_t)(g0 + e) * V, u0[e] + cr[e]);
                        }
                    }
                };
                if (p.write_sketch) {
                    if (p.sketch_bf16) rows(std::true_type{}); else rows(std::false_type{});
                }
                if (p.out != nullptr) {       // exact output: the query column
                    float ou, oc;
                    tmem_ld1x2(slot + 32u + (uint32_t)QA, slot + (uint32_t)QA, ou, oc);
                    const float o = ou + oc;
                    if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[bh * V + j] = __float2bfloat16_rn(o);
                    else reinterpret_cast<float*>(p.out)[bh * V + j] = o;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) k_arrive(&bars[kBufFree + b]);       // the slot is free for pass A of tile k + 2
            }
            // the E step of the next tile: its P is complete once pass A of that tile is, and the E operand buffer is free
            // because Ktil^T E of this tile has completed (waited for above)
            raw = seq_get(k + 1);
            if (raw < 0) { bad |= raw < -1; break; }
            if (!bad) do_e(b ^ 1);
        }
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 111);
    } else if (warp == 8) {
        // =========================== MMA issue warp (one thread) ===========================
        if (lane == 0) {
            uint32_t phR = 0, phE = 0, phBuf = 0, phSt = 0;
            bool bad = false;
            int where = 104;                // which wait gave up (status detail): 141 slot free, 142 chunk ready, 143 E ready, 145 accumulator written
            const uint32_t a2base = smem_u32(smem + sm.a2);
            auto step_e = [&](int k) {          // Ktil^T E onto G_n * S_0 (128 columns) and the sketch correction E^T (Ktil W) over the spent P
                const int b = k & 1;
                if (!mbar_wait_bounded(&bars[kErdy], phE)) { bad = true; where = 143; return; }
                phE ^= 1u;
                // G_n * S_0 is in accumulator b (the pass-A group stored it after the pass-B group had read tile k - 2 from it)
                if (!mbar_wait_bounded(&bars[kStDone + b], (phSt >> b) & 1u)) { bad = true; where = 145; return; }
                phSt ^= 1u << b;
                tc_fence_after();
                const uint32_t tmem_t = tmem_base + 128u + (uint32_t)b * 128u;
                const uint32_t tmem_c = tmem_base + (uint32_t)b * 64u;
                const uint32_t e = smem_u32(smem + sm.e);
                const uint32_t bt = smem_u32(set_ptr(b) + sm.set_bt);
                const uint32_t bc = smem_u32(set_ptr(b) + sm.set_bc);
                for (int kk = 0; kk < ksteps; ++kk) {
                    const uint64_t ehi = make_desc(e + (uint32_t)kk * 2u * LBO_M, LBO_M, SBO);
                    const uint64_t elo = make_desc(e + 128u * (uint32_t)kNT * 2u + (uint32_t)kk * 2u * LBO_M, LBO_M, SBO);
                    const uint64_t bthi = make_desc(bt + (uint32_t)kk * 2u * kLboT, kLboT, kSboT);
                    const uint64_t btlo = make_desc(bt + sm.set_bt_lo + (uint32_t)kk * 2u * kLboT, kLboT, kSboT);
                    const uint64_t bchi = make_desc(bc + (uint32_t)kk * 2u * LBO_C, LBO_C, SBO);
                    const uint64_t bclo = make_desc(bc + 2048u + (uint32_t)kk * 2u * LBO_C, LBO_C, SBO);
                    tc_mma_bf16(tmem_t, ehi, bthi, idescT, 1u);
                    tc_mma_bf16(tmem_t, elo, bthi, idescT, 1u);
                    tc_mma_bf16(tmem_t, ehi, btlo, idescT, 1u);
                    tc_mma_bf16(tmem_c, ehi, bchi, idescU, kk ? 1u : 0u);
                    tc_mma_bf16(tmem_c, elo, bchi, idescU, 1u);
                    tc_mma_bf16(tmem_c, ehi, bclo, idescU, 1u);
                }
                tc_commit(&bars[kTfull + b]);
            };
            // The E step of a tile is issued as soon as its E operand is ready, also in the middle of the next tile's pass A:
            // every wait of pass A polls for it in turn (pend_e: the tile whose E step is still to be issued, or -1).
            int pend_e = -1;
            auto wait_or_e = [&](uint64_t* bar, uint32_t phase) -> bool {
                for (uint32_t it = 0; it < (1u << 22); ++it) {
                    if (mbar_test_wait(bar, phase)) return true;
                    if (pend_e >= 0 && mbar_test_wait(&bars[kErdy], phE)) {
                        const int ke = pend_e;
                        pend_e = -1;
                        step_e(ke);
                        if (bad) return false;
                    }
                }
                return false;
            };
            // [P | U0](b) = S_0^T [Khat^T | G_n * W] chunk by chunk: one 64-row window per tile
            auto pass_a = [&](int k) {
                const int b = k & 1;
                if (k >= 2) {                   // the slot still holds the sketch data of tile k - 2 until they are stored
                    if (!wait_or_e(&bars[kBufFree + b], (phBuf >> b) & 1u)) { bad = true; where = 141; return; }
                    phBuf ^= 1u << b;
                    tc_fence_after();
                }
                const uint32_t slot = tmem_base + (uint32_t)b * 64u;
                const uint32_t whi0 = smem_u32(w_ptr(b));
                const uint32_t wlo0 = whi0 + sm.w_lo;
#pragma unroll 2
                for (int c = 0; c < NCH; ++c) {
                    const int ab = c & (kKA2 - 1);
                    if (!wait_or_e(&bars[kA2rdy + ab], (phR >> ab) & 1u)) { bad = true; where = 142; return; }
                    phR ^= 1u << ab;
                    tc_fence_after();
                    const uint32_t a2 = a2base + (uint32_t)ab * (2u * 128u * CH * 2u);
                    const uint64_t ahi = make_desc(a2, LBO_M, SBO);
                    const uint64_t alo = make_desc(a2 + 128u * CH * 2u, LBO_M, SBO);
                    const uint64_t whi = make_desc(whi0 + (uint32_t)(c * (CH / 8)) * LBO_W, LBO_W, SBO);
                    const uint64_t wlo = make_desc(wlo0 + (uint32_t)(c * (CH / 8)) * LBO_W, LBO_W, SBO);
                    tc_mma_bf16(slot, ahi, whi, idescA, c ? 1u : 0u);
                    tc_mma_bf16(slot, alo, whi, idescA, 1u);
                    tc_mma_bf16(slot, ahi, wlo, idescA, 1u);
                    tc_commit(&bars[kA2free + ab]);
                    if (c == NCH - 1) tc_commit(&bars[kPfull + b]);
                }
            };
            int cur = seq_get(0);
            if (cur >= 0) {
                // pass A of tile k + 1 starts before the E step of tile k: the stream of S_0 chunks does not wait for the
                // pass-B group (two accumulators); the E step goes out as soon as that group has formed E
                pass_a(0);
                for (int k = 0; !bad; ++k) {
                    pend_e = k;
                    const int raw = seq_get(k + 1);
                    if (raw < -1) { bad = true; break; }
                    if (raw >= 0) pass_a(k + 1);
                    if (bad) break;
                    if (pend_e >= 0) { pend_e = -1; step_e(k); }
                    if (raw < 0) break;
                }
            } else if (cur < -1) {
                bad = true;
            }
            if (bad) record_fault(p.status, kFaultUpdateWait, where);
        }
    } else if (warp == 9) {
        // =========================== state-load warp: keeps the ring of S_0 stages full ===========================
        int stage = 0, round = 0;
        bool bad = false;
        auto load_tile = [&](int tile) {
            const int h = tile / tiles_per_h, bb = tile - h * tiles_per_h;
            const float* src = p.state + ((size_t)bb * H + h) * (size_t)K * V;
            for (int c = 0; c < NCH; ++c) {
                if (round > 0) {     // the stage was released by all four stream warps
                    if (!mbar_wait_bounded(&bars[kEmpty + stage], (uint32_t)(round - 1) & 1u)) { bad = true; return; }
                }
                uint64_t* bar = &bars[kFull + stage];
                if (lane == 0) {
                    mbar_expect_tx(bar, sm.sst_bytes);
                    bulk_g2s(smem + sm.sst + (size_t)stage * sm.sst_bytes, src + (size_t)c * CH * V, (uint32_t)(CH * V * 4), bar);
                }
                if (++stage == NS) { stage = 0; ++round; }
            }
        };
        int cur = seq_get(0);
        if (cur >= 0) {
            load_tile(cur);
            for (int k = 0; !bad; ++k) {
                const int raw = seq_get(k + 1);
                if (raw < -1) { bad = true; break; }
                if (raw < 0) break;
                load_tile(raw);
            }
        } else if (cur < -1) {
            bad = true;
        }
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 107);
    } else {
        // =========================== front group: ring-only operands, tile claiming ===========================
        // 256 threads: thread = (token block fg, channel i).  Block fg holds tokens 16 fg .. 16 fg + 15 of the pass: its
        // threads build that block's triangle of A, its rows of Khat / Ktil and its rescaled keys, so that the two
        // halves of a tile's ring-only work run side by side.
        const int ft = warp < 8 ? tid - 128 : tid - (kKThreads - 128) + 128;      // 0..255 (warps 4-7, then the last four warps)
        const int fg = ft >> 7;               // token block
        const int i = ft & 127;               // this thread's channel
        const int fw = ft >> 5;               // warp of the group, 0..7
        uint32_t phS = 0;
        bool dead = false;
        float* sA = reinterpret_cast<float*>(smem + sm.mats);
        float* sBeta = sA + kNT * kAS;
        float* sOm = reinterpret_cast<float*>(smem + sm.om);
        int cur_h = -1;
        float* sPart = reinterpret_cast<float*>(sStg + 2u * kZHalf);   // [8 warps][4 batches][32] partial pair sums (over the value rows, copied out by then)

        // ---- tile claiming (thread 0 of the group): per-head-index counters behind the status words ----
        int* sched = p.status + kStatusInts;
        int* cnt = sched + 4;
        int h_claim = (int)(((long long)blockIdx.x * H) / gridDim.x);
        int t_raw = 0;
        auto claim_issue = [&]() { t_raw = atomicAdd(&cnt[h_claim], 1); };
        auto claim_resolve = [&]() -> int {
            for (int attempt = 0; attempt <= H; ++attempt) {
                if (t_raw < tiles_per_h) return h_claim * tiles_per_h + t_raw;
                int best = -1, best_c = tiles_per_h;
                for (int ii = 1; ii <= H; ++ii) {
                    int hh = h_claim + ii;
                    if (hh >= H) hh -= H;
                    const int c = *reinterpret_cast<volatile int*>(&cnt[hh]);
                    if (c < best_c) { best_c = c; best = hh; }
                }
                if (best < 0) return -1;
                h_claim = best;
                t_raw = atomicAdd(&cnt[h_claim], 1);
            }
            return -1;
        };
        auto publish = [&](int k, int tile) {
            seq_ring[k & 3] = tile;
            __threadfence_block();
            *seq_pub = k + 1;
        };

        // One bulk copy per thread from per-thread constants, spread over the first four warps of the group: copy number c
        // belongs to lane c / 4 of warp c % 4.  0..3: ring keys, decays, values, gates; 4..7: the token's key, decay, value, the query.
        const uint32_t stg_beta_bytes = n_ring > 0 ? (uint32_t)(p.L * 4) : 0u;
        const uint32_t stg_bytes = (uint32_t)n_ring * 768u + stg_beta_bytes + (p.has_token ? 768u : 0u) + (p.q != nullptr ? 256u : 0u);
        const int cp_c = (ft < 128 && (ft & 31) < 2) ? (ft & 31) * 4 + (ft >> 5) : 32;
        const unsigned char* cp_base = nullptr;
        size_t cp_stride = 0;
        uint32_t cp_dst = 0, cp_bytes = 0;
        switch (cp_c) {
            case 0: cp_base = p.ring + (size_t)p.tok_base * 256u; cp_stride = p.rl.head_bytes; cp_dst = 0u; cp_bytes = (uint32_t)n_ring * 256u; break;
            case 1: cp_base = p.ring + p.rl.decay_off + (size_t)p.tok_base * 256u; cp_stride = p.rl.head_bytes; cp_dst = sm.stg_g; cp_bytes = (uint32_t)n_ring * 256u; break;
            case 2: cp_base = p.ring + p.rl.v_off + (size_t)p.tok_base * 256u; cp_stride = p.rl.head_bytes; cp_dst = sm.stg_v; cp_bytes = (uint32_t)n_ring * 256u; break;
            case 3: cp_base = p.ring + p.rl.beta_off; cp_stride = p.rl.head_bytes; cp_dst = sm.stg_beta; cp_bytes = stg_beta_bytes; break;
            case 4: cp_base = reinterpret_cast<const unsigned char*>(p.k); cp_stride = (size_t)K * 2; cp_dst = (uint32_t)n_ring * 256u; cp_bytes = p.has_token ? 256u : 0u; break;
            case 5: cp_base = reinterpret_cast<const unsigned char*>(p.decay); cp_stride = (size_t)K * 2; cp_dst = sm.stg_g + (uint32_t)n_ring * 256u; cp_bytes = p.has_token ? 256u : 0u; break;
            case 6: cp_base = reinterpret_cast<const unsigned char*>(p.v); cp_stride = (size_t)V * 2; cp_dst = sm.stg_v + (uint32_t)n_ring * 256u; cp_bytes = p.has_token ? 256u : 0u; break;
            case 7: cp_base = reinterpret_cast<const unsigned char*>(p.q); cp_stride = (size_t)K * 2; cp_dst = sm.stg_q; cp_bytes = p.q != nullptr ? 256u : 0u; break;
            default: break;
        }
        auto stage_tile = [&](int tile) {       // whole group
            const int h = tile / tiles_per_h, bb = tile - h * tiles_per_h;
            const size_t bw = (size_t)bb * H + h;
            if (ft == 0) mbar_expect_tx(&bars[kStg], stg_bytes);      // (the phase cannot complete before this arrival, whatever the order of the copies)
            __syncwarp();
            if (cp_bytes) bulk_g2s(sStg + cp_dst, cp_base + bw * cp_stride, cp_bytes, &bars[kStg]);
        };
        auto next_tile = [&](int k) {          // whole group
            if (ft == 0) {
                const int nxt = claim_resolve();
                publish(k, nxt);
                if (nxt >= 0) claim_issue();
            }
            f_sync();                          // the published entry is the hand-off to the other threads
            const int nxt = seq_ring[k & 3];
            if (nxt >= 0) stage_tile(nxt);
        };
        // the first tile: claimed, published and its rows requested before anything else
        if (ft == 0) claim_issue();
        next_tile(0);
        // operand rows that no tile overwrites hold zeros: the padding columns of [Omega | q] in both windows, and the
        // padding columns of Ktil W in both sets
        for (uint32_t o = (uint32_t)ft * 16u; o < 2u * sm.w_stride; o += kKFront * 16u)
            *reinterpret_cast<uint4*>(smem + sm.w + o) = make_uint4(0, 0, 0, 0);
        for (int sb = 0; sb < 2; ++sb)
            for (uint32_t o = (uint32_t)ft * 16u; o < 4096u; o += kKFront * 16u)
                *reinterpret_cast<uint4*>(set_ptr(sb) + sm.set_bc + o) = make_uint4(0, 0, 0, 0);
        f_sync();

        for (int k = 0; !dead; ++k) {
            const int raw_tile = seq_get(k);
            if (raw_tile < 0) {
                if (raw_tile < -1) {
                    if (ft == 0) record_fault(p.status, kFaultUpdateWait, 108);
                    dead = true;
                }
                break;
            }
            const int tile = raw_tile;
            const int b = k & 1;
            const int h = tile / tiles_per_h, bb = tile - h * tiles_per_h;
            const size_t bh = (size_t)bb * H + h;
            unsigned char* set = set_ptr(b);
            unsigned char* wb = w_ptr(b);

            // gate of the current token: requested early
            float tok_beta = 0.f;
            if (ft < kNT && p.has_token) tok_beta = p.beta[bh];
            // Omega of this head index in shared memory (global loads here would sit on the group's critical path)
            if (h != cur_h) {
                const float* omg = p.omega + (size_t)h * K * R;
                for (int idx = ft; idx < K * 16; idx += kKFront) {
                    const int kk2 = idx >> 4, g = idx & 15;
                    sOm[idx] = (g < R && p.write_sketch) ? __ldg(omg + (size_t)kk2 * R + g) : 0.f;
                }
                cur_h = h;            // (visible to the group after the barrier below)
            }
            const float* og = sOm + i * 16;
            // the staged rows, gates and query row of this tile must have landed
            if (!f_wait(ft, &bars[kStg], phS)) {
                if (ft == 0) record_fault(p.status, kFaultUpdateWait, 106);
                dead = true;
                break;
            }
            phS ^= 1;

            // ---- column i of this block's key and decay rows into registers, the product of the other block's decays;
            // value rows into the set; gates ----
            const int t0 = 16 * fg;
            float kk[16], gg[16];
#pragma unroll
            for (int s = 0; s < 16; ++s) {
                const bool on = t0 + s < n_tot;
                kk[s] = on ? bf16_at(sStg, (uint32_t)((t0 + s) * K + i)) : 0.f;
                gg[s] = on ? bf16_at(sStg + sm.stg_g, (uint32_t)((t0 + s) * K + i)) : 1.f;
            }
            float gother = 1.f;
#pragma unroll
            for (int s = 0; s < 16; ++s) {
                const int t = 16 * (1 - fg) + s;
                if (t < n_tot) gother *= bf16_at(sStg + sm.stg_g, (uint32_t)(t * K + i));
            }
            uint4 vrow[2];            // 512 vectors of 16 bytes: 32 value rows, parked in registers until the set is free
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int idx = ft + r * kKFront;
                vrow[r] = make_uint4(0, 0, 0, 0);
                if ((idx >> 4) < n_tot) vrow[r] = *reinterpret_cast<const uint4*>(sStg + sm.stg_v + (size_t)idx * 16);
            }
            const float q_i = p.q != nullptr ? bf16_at(sStg + sm.stg_q, (uint32_t)i) : 0.f;
            if (ft < kNT) {
                const int s = ft;
                float bt = 0.f;
                if (s < n_ring) bt = reinterpret_cast<const float*>(sStg + sm.stg_beta)[p.tok_base + s];
                else if (s < n_tot) bt = tok_beta;
                sBeta[s] = bt;
            }
            f_sync();                  // every thread holds its column: the key / decay rows of the staging area are free

            // ---- pair sums inside this block of 16 tokens (its triangle of A): A_sj = sum_i k_s[i] k_j[i]
            // prod_{j<m<=s} g_m[i] as per-channel products, reduced over the 32 channels of a warp by a transposing
            // butterfly, 32 pairs at a time: rows sa and 16 - sa in entries 0..15, rows sa + 1 and 15 - sa in 16..31 ----
            {
                float* part = sPart + (size_t)fw * 128;
#pragma unroll
                for (int bi = 0; bi < 4; ++bi) {
                    float vals[32];
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int sa = 2 * bi + 1 + hh, o = 16 * hh;
                        {
                            float r = kk[sa];
#pragma unroll
                            for (int jj = 7; jj >= 0; --jj)
                                if (jj < sa) { r *= gg[jj + 1]; vals[o + jj] = r * kk[jj]; }
                        }
                        if (sa < 8) {
                            const int sb2 = 16 - sa;
                            float r = kk[sb2];
#pragma unroll
                            for (int jj = 14; jj >= 0; --jj)
                                if (jj < sb2) { r *= gg[jj + 1]; vals[o + sa + jj] = r * kk[jj]; }
                        } else {
#pragma unroll
                            for (int jj = 8; jj < 16; ++jj) vals[o + jj] = 0.f;
                        }
                    }
                    group_reduce_transpose<32, 32>(vals, lane);      // lane l now holds entry l of the batch
                    part[bi * 32 + lane] = vals[0];
                }
            }

            // Up to here nothing of the operand set and window b was touched: they are free once Ktil^T E of tile k - 2 has
            // completed, so the loads and pair sums above overlap the tail of that tile.
            if (k >= 2) {
                if (!f_wait(ft, &bars[kTfull + b], (uint32_t)((k - 2) >> 1) & 1u)) {
                    if (ft == 0) record_fault(p.status, kFaultUpdateWait, 109);
                    dead = true;
                    break;
                }
            }
#pragma unroll
            for (int r = 0; r < 2; ++r)
                *reinterpret_cast<uint4*>(set + sm.set_vv + (size_t)(ft + r * kKFront) * 16) = vrow[r];

            // ---- running products of this block.  Khat -> window rows 0..31; Ktil -> set (MN-major); G_n * W -> window
            // rows 32..; and for the 16 x 16 block of A that couples the two token blocks, whose decay product splits at
            // the block boundary without a quotient (prod_{j<m<=s} = prod_{16<=m<=s} * prod_{j<m<=15}), the rescaled keys
            // X_s = k_s prod_{16<=m<=s} g_m (s >= 16, by block 1) and Y_j = k_j prod_{j<m<=15} g_m (j < 16, by block 0)
            // as bf16 hi + lo rows Z[token][channel] over the (now free) key / decay rows of the staging area ----
            {
                __nv_bfloat16* whi = reinterpret_cast<__nv_bfloat16*>(wb);
                __nv_bfloat16* wlo = reinterpret_cast<__nv_bfloat16*>(wb + sm.w_lo);
                __nv_bfloat16* bthi = reinterpret_cast<__nv_bfloat16*>(set + sm.set_bt);
                __nv_bfloat16* btlo = reinterpret_cast<__nv_bfloat16*>(set + sm.set_bt_lo);
                __nv_bfloat16* zhi = reinterpret_cast<__nv_bfloat16*>(sStg);
                __nv_bfloat16* zlo = reinterpret_cast<__nv_bfloat16*>(sStg + kZHalf);
                const uint32_t wcol = ((uint32_t)(i >> 3) * LBO_W + (uint32_t)(i & 7) * 2u) >> 1;        // K-major: k = channel
                const uint32_t bcol = ((uint32_t)(i & 7) * 2u + (uint32_t)(i >> 3) * kSboT) >> 1;        // MN-major: mn = channel
                float G = fg ? gother : 1.f, X = 1.f;
#pragma unroll
                for (int s = 0; s < 16; ++s) {
                    G *= gg[s];
                    __nv_bfloat16 hi, lo;
                    split_bf16(G * kk[s], hi, lo);
                    const uint32_t o = wcol + (((uint32_t)(s & 7) * 16u + (uint32_t)((s >> 3) + 2 * fg) * SBO) >> 1);
                    whi[o] = hi;
                    wlo[o] = lo;
                    if (fg) {
                        X *= gg[s];
                        split_bf16(X * kk[s], hi, lo);
                        zhi[(16 + s) * (kZPitch / 2) + i] = hi;
                        zlo[(16 + s) * (kZPitch / 2) + i] = lo;
                    }
                }
                const float Gn = fg ? G : G * gother;       // decay of the whole pass
                float Dn = fg ? 1.f : gother, Yd = 1.f;
#pragma unroll
                for (int s = 15; s >= 0; --s) {
                    const float kt = Dn * kk[s];
                    Dn *= gg[s];
                    __nv_bfloat16 hi, lo;
                    split_bf16(kt, hi, lo);
                    const uint32_t o = bcol + (((uint32_t)(s & 7) * 16u + (uint32_t)((s >> 3) + 2 * fg) * kLboT) >> 1);
                    bthi[o] = hi;
                    btlo[o] = lo;
                    if (!fg) {
                        split_bf16(Yd * kk[s], hi, lo);
                        zhi[s * (kZPitch / 2) + i] = hi;
                        zlo[s * (kZPitch / 2) + i] = lo;
                        Yd *= gg[s];
                    }
                }
                if (!fg) reinterpret_cast<float*>(set + sm.set_gn)[i] = Gn;
                // G_n * [Omega | q]: block 0 takes the first half of the sketch columns, block 1 the rest and the query
                const int Rh = (R + 1) >> 1;
                if (p.write_sketch) {
                    const int g_lo = fg ? Rh : 0, g_hi = fg ? R : Rh;
                    for (int g = g_lo; g < g_hi; ++g) {
                        __nv_bfloat16 hi, lo;
                        split_bf16(Gn * og[g], hi, lo);
                        const uint32_t o = wcol + (((uint32_t)(g & 7) * 16u + (uint32_t)((g >> 3) + 4) * SBO) >> 1);
                        whi[o] = hi;
                        wlo[o] = lo;
                    }
                }
                if (fg && p.q != nullptr) {
                    __nv_bfloat16 hi, lo;
                    split_bf16(Gn * q_i, hi, lo);
                    const uint32_t o = wcol + (((uint32_t)(QA & 7) * 16u + (uint32_t)((QA >> 3) + 4) * SBO) >> 1);
                    whi[o] = hi;
                    wlo[o] = lo;
                }
            }
            f_sync();                  // partial pair sums, Z rows and Ktil are complete

            if (fw == 7) {
                // ---- A_21 = X Y^T (16 x 16, tokens 16..31 against tokens 0..15) as mma.sync products of the Z rows,
                // hi * hi + lo * hi + hi * lo ----
                float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                const uint32_t zb = smem_u32(sStg);
                const uint32_t abase = zb + (uint32_t)(16 + (lane & 15)) * kZPitch + (uint32_t)(lane >> 4) * 16u;
                const uint32_t bbase = zb + (uint32_t)(lane & 7) * kZPitch + (uint32_t)((lane >> 3) & 1) * 16u;
#pragma unroll
                for (int ks = 0; ks < K / 16; ++ks) {
                    uint32_t ahi[4], alo[4];
                    k_ldmatrix_x4(abase + ks * 32, ahi);
                    k_ldmatrix_x4(abase + kZHalf + ks * 32, alo);
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        uint32_t bhi[2], blo[2];
                        k_ldmatrix_x2(bbase + (uint32_t)(nt * 8) * kZPitch + ks * 32, bhi);
                        k_ldmatrix_x2(bbase + (uint32_t)(nt * 8) * kZPitch + kZHalf + ks * 32, blo);
                        k_mma_16816(acc[nt], ahi, bhi);
                        k_mma_16816(acc[nt], alo, bhi);
                        k_mma_16816(acc[nt], ahi, blo);
                    }
                }
                float* sA21 = reinterpret_cast<float*>(set + sm.set_t1) + 512;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    const int r0 = lane >> 2, c0 = nt * 8 + (lane & 3) * 2;
                    sA21[r0 * 16 + c0] = acc[nt][0];
                    sA21[r0 * 16 + c0 + 1] = acc[nt][1];
                    sA21[(r0 + 8) * 16 + c0] = acc[nt][2];
                    sA21[(r0 + 8) * 16 + c0 + 1] = acc[nt][3];
                }
            } else {
                // ---- beta_s A_sj of the two triangles: the partials of a block's four warps summed in a fixed order ----
                for (int idx = ft; idx < 2 * 16 * 16; idx += 224) {
                    const int blk = idx >> 8, s = (idx >> 4) & 15, jj = idx & 15;
                    float a = 0.f;
                    if (jj < s) {
                        const int sa = s <= 8 ? s : 16 - s;
                        const int e = ((sa - 1) >> 1) * 32 + ((sa - 1) & 1) * 16 + (s <= 8 ? jj : sa + jj);
                        const float* pp = sPart + blk * 512 + e;
                        a = ((pp[0] + pp[128]) + pp[256]) + pp[384];
                    }
                    sA[blk * (16 * kAS2) + s * kAS2 + jj] = sBeta[16 * blk + s] * a;
                }
            }
            f_sync();                  // A is complete

            if ((fw & 3) == 0) {
                // ---- T_bb = (I + Bd A_bb)^{-1} Bd of block fw / 4 by forward substitution: one column per thread, in registers ----
                const int blk = fw >> 2;
                if (lane < 16) {
                    const int c = lane;
                    const int nb = min(max(n_tot - 16 * blk, 0), 16);      // tokens of this block
                    const float* sAb = sA + blk * (16 * kAS2);
                    float tcol[16];
#pragma unroll
                    for (int s = 0; s < 16; ++s) {
                        float acc = 0.f;
#pragma unroll
                        for (int j4 = 0; j4 < (s + 3) / 4; ++j4) {
                            const float4 l4 = *reinterpret_cast<const float4*>(sAb + s * kAS2 + j4 * 4);
                            if (j4 * 4 + 0 < s) acc = fmaf(l4.x, tcol[j4 * 4 + 0], acc);
                            if (j4 * 4 + 1 < s) acc = fmaf(l4.y, tcol[j4 * 4 + 1], acc);
                            if (j4 * 4 + 2 < s) acc = fmaf(l4.z, tcol[j4 * 4 + 2], acc);
                            if (j4 * 4 + 3 < s) acc = fmaf(l4.w, tcol[j4 * 4 + 3], acc);
                        }
                        tcol[s] = (s >= nb || s < c || c >= nb) ? 0.f : (s == c ? 1.f : -acc);
                    }
                    const float bc = sBeta[16 * blk + c];
                    float* sT = reinterpret_cast<float*>(set + sm.set_t1) + blk * 256;
#pragma unroll
                    for (int s = 0; s < 16; ++s) sT[s * 16 + c] = tcol[s] * bc;
                }
            } else {
                // ---- Ktil W: 16 tokens (block fw / 4) x 8 columns of [Omega | q] (columns 8 nt .., nt = fw % 4 - 1) as
                // mma.sync products.  A: the Ktil operand just written (its 8 x 8 core matrices are the row-major fragments
                // ldmatrix wants), hi + lo; B: Omega and q from shared memory into fragments, split into hi + lo in registers ----
                const int mt = fw >> 2, nt = (fw & 3) - 1;
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                const uint32_t btb = smem_u32(set + sm.set_bt);
                const uint32_t a_row = btb + (uint32_t)(2 * mt + ((lane >> 3) & 1)) * kLboT + (uint32_t)(lane >> 4) * kSboT + (uint32_t)(lane & 7) * 16u;
                const __nv_bfloat16* sq = reinterpret_cast<const __nv_bfloat16*>(sStg + sm.stg_q);
                const int ncol = p.write_sketch ? R : 0;
                const bool has_q = p.q != nullptr;
                const int g = nt * 8 + (lane >> 2);
                const int src = g < ncol ? 0 : (g == QA && has_q) ? 1 : 2;       // Omega column, query, padding
#pragma unroll 4
                for (int ks = 0; ks < K / 16; ++ks) {
                    uint32_t ahi[4], alo[4];
                    k_ldmatrix_x4(a_row + (uint32_t)(2 * ks) * kSboT, ahi);
                    k_ldmatrix_x4(a_row + sm.set_bt_lo + (uint32_t)(2 * ks) * kSboT, alo);
                    const int i0 = ks * 16 + (lane & 3) * 2;
                    float w[4] = {0.f, 0.f, 0.f, 0.f};
                    if (src == 0) {
                        w[0] = sOm[i0 * 16 + g];
                        w[1] = sOm[(i0 + 1) * 16 + g];
                        w[2] = sOm[(i0 + 8) * 16 + g];
                        w[3] = sOm[(i0 + 9) * 16 + g];
                    } else if (src == 1) {
                        w[0] = __bfloat162float(sq[i0]);
                        w[1] = __bfloat162float(sq[i0 + 1]);
                        w[2] = __bfloat162float(sq[i0 + 8]);
                        w[3] = __bfloat162float(sq[i0 + 9]);
                    }
                    uint32_t bhi[2], blo[2];
                    split_bf16x2(w[0], w[1], bhi[0], blo[0]);
                    split_bf16x2(w[2], w[3], bhi[1], blo[1]);
                    k_mma_16816(acc, ahi, bhi);
                    k_mma_16816(acc, alo, bhi);
                    k_mma_16816(acc, ahi, blo);
                }
                __nv_bfloat16* bchi = reinterpret_cast<__nv_bfloat16*>(set + sm.set_bc);
                __nv_bfloat16* bclo = bchi + 1024;
                auto put = [&](int s, int gc, float x) {
                    __nv_bfloat16 hi, lo;
                    split_bf16(x, hi, lo);
                    const uint32_t o2 = ((uint32_t)(gc & 7) * 16u + (uint32_t)(gc >> 3) * SBO + (uint32_t)(s >> 3) * LBO_C + (uint32_t)(s & 7) * 2u) >> 1;
                    bchi[o2] = hi;
                    bclo[o2] = lo;
                };
                const int s0 = 16 * mt + (lane >> 2), g0 = nt * 8 + (lane & 3) * 2;
                put(s0, g0, acc[0]);
                put(s0, g0 + 1, acc[1]);
                put(s0 + 8, g0, acc[2]);
                put(s0 + 8, g0 + 1, acc[3]);
            }
            proxy_fence();         // operand sets and windows are read by MMAs (async proxy)
            f_sync();
            if (ft == 0) k_arrive(&bars[kPro + b]);
            next_tile(k + 1);      // the staging area has been read: the next tile's rows may come in
        }
        if (ft == 0) {     // scheduler counters back to zero once every CTA is done claiming
            __threadfence();
            if (atomicAdd(&sched[0], 1) == (int)gridDim.x - 1) {
                for (int hh = 0; hh < H; ++hh) cnt[hh] = 0;
                sched[0] = 0;
                __threadfence();
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// One pass of the kernel over all tiles: ring rows tok_base .. tok_base + n_before - 1 (and the current token).
static int launch_kda_pass(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    Params p = p_in;
    const uint32_t budget = 227u * 1024u;
    const KSmem fixed = make_ksmem(0);
    if (fixed.total + 2u * fixed.sst_bytes > budget) return SKETCHSSM_UNSUPPORTED_SHAPE;
    int stages = (int)((budget - fixed.total) / fixed.sst_bytes);
    if (stages > kKStages) stages = kKStages;
    if (p.stages >= 2 && p.stages < stages) stages = p.stages;
    p.stages = stages;
    const KSmem sm = make_ksmem(stages);
    const long long n_tiles = (long long)c.batch * c.heads;
    long long grid = (long long)ctx->sm_count;
    if (grid > n_tiles) grid = n_tiles;
    auto kern = update_tc_ws_kda_kernel;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)sm.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    if ((ctx->last_cuda_error = launch_kernel(kern, dim3((unsigned)grid), dim3(kKThreads), sm.total, stream, p, p.pdl != 0)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    return SKETCHSSM_OK;
}

// Returns SKETCHSSM_UNSUPPORTED_SHAPE outside this kernel's domain (the caller then uses another kernel).  A flush of more
// than 32 tokens is replayed in blocks of 32: every block is one pass over the state, and only the last one (which holds
// the current token) writes the sketch and the exact output.
int launch_update_tc_ws_kda(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    if (c.kind != SKETCHSSM_KDA || c.io_dtype != SKETCHSSM_BF16 || c.dk != kK || c.dv != 128) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (c.rank > 16) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const int n_tot = p_in.n_before + (p_in.has_token ? 1 : 0);
    if (n_tot < 1 || n_tot > 2 * kNT) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (ctx->sm_count == 0) {
        int dev = 0, sms = 0;
        if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        if ((ctx->last_cuda_error = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
        ctx->sm_count = sms;
    }
    const int passes = (n_tot + kNT - 1) / kNT;
    for (int ps = 0; ps < passes; ++ps) {
        Params p = p_in;
        p.tok_base = ps * kNT;
        if (ps + 1 < passes) {          // 32 ring rows, state only
            p.n_before = kNT;
            p.has_token = 0;
            p.q = nullptr;
            p.out = nullptr;
            p.write_sketch = 0;
        } else {
            p.n_before = p_in.n_before - ps * kNT;
        }
        const int rc = launch_kda_pass(ctx, p, stream);
        if (rc != SKETCHSSM_OK) return rc;
    }
    ctx->last_launches = passes;
    return SKETCHSSM_OK;
}

}  // namespace sketchssm
