// Warp-specialised state-update (flush) kernel for the gated delta rule (GDN) on tcgen05 + TMEM, sm_100a.
//
// Replaying n tokens of S_s = a_s S_{s-1} + k_s e_s^T,  e_s = beta_s (v_s - (a_s S_{s-1})^T k_s)  (Eq. 1, 3), unrolled
// over the window (the WY form of Appendix C, Eq. 41-42, applied to the state), is
//     P     = K S_0                                  n x V     raw keys against the old state
//     E'    = T1 (V - C P)                           n x V     T1 = Dn (I + Bd A)^{-1} Bd,  C = diag(prod_{i<=s} a_i),
//                                                              A_sj = (prod_{j<i<=s} a_i) <k_j, k_s> (j < s),  Dn = diag(prod_{i>s} a_i)
//     S_new = (prod_i a_i) S_0 + K^T E'              K x V
//     [U | o] = S_new^T [Omega | q]                            (Eq. 7 and the exact output of the flush step)
// Every product of decays is built by multiplication (no quotients), and all tensor-core operands that come from the
// ring are the raw bf16 keys, so those products are exact; fp32 operands (S_0, S_new, E') are split into bf16 hi + lo.
//
// Tile = one head (K = V = 128); TMEM lane = value column j.  The state is read once: pass A takes the S_0 chunks from a
// ring of shared-memory stages filled by bulk copies, contracts them with the keys (P) and with W = [Omega | q], and
// leaves d S_0 in the accumulator of K^T E' (tcgen05.st), so that the MMAs of the E' step turn it into S_new; pass B
// only writes that accumulator back.  The CTA is specialised:
//   front group (4 warps)   ring-only operands two tiles ahead: key layouts, Gram matrix, T1, K W, tile claiming
//   pass-A group (4 warps)  S_0 chunks -> bf16 hi + lo operands and d S_0 into tensor memory, then the small E' step
//   pass-B group (4 warps)  S_new written back, then the sketch rows and the exact output from tensor memory
//   one thread issues every MMA; one warp keeps the stages full.
// Pass A of tile i + 1 runs while pass B of tile i does (it follows pass B through the accumulator half by half), so no
// MMA round trip is waited for.
//
// The sketch rows never need S_new as a tensor-core operand: [U | o] = d S_0^T W + E'^T (K W), so pass A contracts the
// S_0 chunks with the keys and W in one product (the keys sit next to W in shared memory: a 48-row operand window per
// tile), the small product K W is formed by the front group, and the correction E'^T (K W) rides along with K^T E'.
// Tensor memory per CTA (256 columns): two 64-column slots for alternating tiles ([U0 32 | P 16 | free 16] or
// [free 16 | P 16 | U0 32]; the correction later goes over P and the free columns), and one 128-column accumulator
// for d S_0 + K^T E'.
//
// Shared memory is the busiest unit of this kernel (load/store data pipe ~70 % busy): the staged key rows are padded so
// that ldmatrix reads them without bank conflicts.
//
// Domain: GDN, bf16 I/O, K = V = 128, rank <= 16; 1..16 tokens per pass, up to 64 tokens per flush in blocks of 16
// (one pass over the state per block).
#include <type_traits>
#include "internal.cuh"
#include "tc_common.cuh"

namespace sketchssm {

namespace {

using namespace tc;


constexpr int kGThreads = 448;       // pass-A group (4 warps), front group (4 warps), MMA issue warp, state-load warp, pass-B group (4 warps)
constexpr int kGrp = 128;
constexpr int kNTok = 16;            // tokens per flush
constexpr int kGStages = 8;
constexpr int kGS = 20;              // row stride (floats) of the small n x n work matrices
constexpr uint32_t kKeyRow = 272u;   // bytes between staged key rows: 256 + 16, so that the 8 rows of an ldmatrix fall in different banks
constexpr int kA2 = 2;               // chunk buffers between the pass-A group and the MMA issue warp

struct GSmem {
    uint32_t a2, e, w, set, set_stride, set_bt, set_vv, set_t1, set_bc, set_gates, stg, stg_v, stg_gate, stg_q, mats, bars,
        misc, sst, sst_bytes, total;
};

__host__ __device__ inline GSmem make_gsmem(int NP, int L, int stages) {
    GSmem s;
    uint32_t off = 0;
    s.a2 = off; off += (uint32_t)kA2 * 2u * 128u * 16u * 2u;      // 16-row chunk buffers, hi + lo
    s.e = off; off += 2u * 128u * 16u * 2u;                       // E' hi + lo (same layout as a chunk buffer)
    // B operand of pass A, hi halves: 64 rows [keys of even tiles (16) | Omega | q | q' (NP = 32) | keys of odd tiles (16)],
    // so that a tile's 48-row window [keys | W] or [W | keys] is one operand; then the lo halves of [Omega | q | q']
    s.w = off; off += (64u + (uint32_t)NP) * kK * 2u;
    // per-tile operand set, double-buffered: keys as B operand of K^T E' (MN-major), raw value rows, T1,
    // K [Omega | q] hi | lo (B operand of the sketch correction), gates (C diagonal, total decay)
    s.set = off;
    s.set_bt = 0u; s.set_vv = 4096u; s.set_t1 = 8192u; s.set_bc = 9216u; s.set_gates = 11264u; s.set_stride = 11392u;
    off += 2u * s.set_stride;
    // staging of the next tile's raw rows: keys [16][kKeyRow], values [16][256 B], gates [2L] floats, query row
    s.stg_v = (uint32_t)kNTok * kKeyRow;
    s.stg_gate = s.stg_v + 4096u;
    s.stg_q = s.stg_gate + (((uint32_t)(2 * L * 4) + 127u) & ~127u);
    s.stg = off; off += s.stg_q + 256u;
    s.mats = off; off += 4u * (uint32_t)kNTok * kGS * 4u + 256u;  // Gram / A, decay products, T, beta / alpha / dn
    s.bars = off; off += 384u;
    s.misc = off; off += 64u;
    off = (off + 127u) & ~127u;
    s.sst_bytes = 16u * 128u * 4u;
    s.sst = off; off += (uint32_t)stages * s.sst_bytes;
    s.total = off;
    return s;
}

enum { gPro = 0, gPfull = 2, gTfull = 4, gBdone = 6, gBufFree = 8, gA2free = 10, gA2rdy = 10 + kA2, gErdy = 10 + 2 * kA2,
       gStg = 11 + 2 * kA2, gProW = 12 + 2 * kA2, gFull = 14 + 2 * kA2, gEmpty = 14 + 2 * kA2 + kGStages,
       gTfree = 14 + 2 * kA2 + 2 * kGStages, gNumBars = 16 + 2 * kA2 + 2 * kGStages };

__device__ __forceinline__ void g_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void g_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
__device__ __forceinline__ bool g_or(int id, bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %2, 0;\n\t"
        "bar.red.or.pred p, %1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(flag ? 1u : 0u)
        : "memory");
    return r != 0;
}
// group-wide bounded wait: one warp polls, the others sleep in the named barrier
__device__ __forceinline__ bool g_wait(int id, int gt, uint64_t* bar, uint32_t phase) {
    bool bad = false;
    if (gt < 32) bad = !mbar_wait_bounded(bar, phase);
    return !g_or(id, bad);
}

__device__ __forceinline__ void g_ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void g_ldmatrix_x2(uint32_t addr, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void g_mma_16816(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

}  // namespace

__global__ void __launch_bounds__(kGThreads, 2) update_tc_ws_gdn_kernel(const Params p) {
    constexpr int K = kK, V = 128, CH = 16, NCH = K / CH;
    extern __shared__ __align__(1024) unsigned char smem[];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gt = tid & 127;
    const int R = p.R, H = p.H, B = p.B;
    const int QA = (R + 7) & ~7;                          // first column of query group A; group B follows 8 columns later
    const int NP = (QA + 16 + 15) & ~15;                  // <= 32 (checked by the launcher)
    const int NS = p.stages;
    const int n_ring = p.n_before, n_tot = n_ring + (p.has_token ? 1 : 0);     // 1..16 per pass (the launcher sees to it)
    const GSmem sm = make_gsmem(NP, p.L, NS);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + sm.misc);
    unsigned char* sStg = smem + sm.stg;

    constexpr uint32_t tmem_cols = 256u;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        *reinterpret_cast<volatile int*>(smem + sm.misc + 32) = 0;
        for (int i = 0; i < gNumBars; ++i) {
            const bool per_warp = (i >= gA2rdy && i <= gErdy) || i >= gEmpty /* gTfree too */ || (i >= gBdone && i < gBdone + 4);     // one arrival per warp of a stream group (gBdone, gBufFree too)
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
    const uint32_t idescU = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)NP >> 3) << 17) | ((128u >> 4) << 24);        // K-major x K-major, N = NP
    const uint32_t idescA = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)(NP + 16) >> 3) << 17) | ((128u >> 4) << 24);   // K-major x K-major, N = NP + 16
    // canonical no-swizzle layouts (byte offsets)
    //   K-major : elem(mn, k) at (mn%8)*16 + (mn/8)*128 + (k/8)*LBO + (k%8)*2,  LBO = 16*MN
    //   MN-major: elem(mn, k) at (k%8)*16 + (mn%8)*2 + (mn/8)*128 + (k/8)*2048
    constexpr uint32_t SBO = 128, LBO_M = 2048;
    constexpr uint32_t LBO_WH = 64u * 16u;                // hi halves: 64 rows
    const uint32_t LBO_WL = (uint32_t)NP * 16u;           // lo halves: NP rows
    const uint32_t w_lo_off = 64u * kK * 2u;              // byte offset of the lo halves in the W region

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

    const int j = (warp & 3) * 32 + lane;      // value column = TMEM lane of this thread (both stream groups and the front group)
    volatile float* sDt = reinterpret_cast<volatile float*>(smem + sm.misc + 40);      // total decay of the tile in each operand set

    if (warp < 4) {
        // =========================== pass-A group: S_0 chunks -> operands, and the E' step ===========================
        uint32_t phPro = 0, phP = 0, phT = 0, phA = 0, phF = 0;
        int gc = 0, stage = 0;
        bool bad = false;

        uint32_t phTf = 0;
        // pass A of a tile with operand set b; `later`: not the CTA's first tile, so the K^T E' accumulator still holds
        // the tile before until the pass-B group has read it (half by half)
        auto pass_a = [&](int b, bool later) {
            const float dtile = reinterpret_cast<const float*>(set_ptr(b) + sm.set_gates)[kNTok];
#pragma unroll 2
            for (int c = 0; c < NCH; ++c) {
                if (later && (c == 0 || c == NCH / 2)) {
                    const int hf = c ? 1 : 0;
                    bad |= !mbar_wait_bounded(&bars[gTfree + hf], (phTf >> hf) & 1u);
                    phTf ^= 1u << hf;
                    tc_fence_after();
                }
                bad |= !mbar_wait_bounded(&bars[gFull + stage], phF);
                const float* sS = reinterpret_cast<const float*>(smem + sm.sst + (size_t)stage * sm.sst_bytes) + j;
                float s0[CH];
#pragma unroll
                for (int ii = 0; ii < CH; ++ii) s0[ii] = sS[ii * V];
                __syncwarp();
                if (lane == 0) g_arrive(&bars[gEmpty + stage]);
                {   // d S_0 goes into the K^T E' accumulator, so that the MMAs leave S_new there: pass B reads S_0 no more
                    float ds[CH];
#pragma unroll
                    for (int ii = 0; ii < CH; ++ii) ds[ii] = dtile * s0[ii];
                    if (!bad) tmem_st16(tmem_base + 128u + lane_sel + (uint32_t)(c * CH), ds);
                }
                const int ab = c & (kA2 - 1);
                if (gc >= kA2) {     // the chunk buffer was read by the MMAs issued kA2 chunks ago
                    bad |= !mbar_wait_bounded(&bars[gA2free + ab], (phA >> ab) & 1u);
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
                if (lane == 0 && !bad) g_arrive(&bars[gA2rdy + ab]);
                ++gc;
                if (++stage == NS) { stage = 0; phF ^= 1u; }
            }
        };
        // E'[s, j] = sum_t T1[s, t] (v_t[j] - C_t P[t, j]) -> hi + lo A operand of K^T E' (chunk-buffer layout)
        auto do_e = [&](int b) {
            bad |= !mbar_wait_bounded(&bars[gPfull + b], (phP >> b) & 1u);
            phP ^= 1u << b;
            tc_fence_after();
            const unsigned char* set = set_ptr(b);
            const __nv_bfloat16* sV = reinterpret_cast<const __nv_bfloat16*>(set + sm.set_vv);
            const float* sT1 = reinterpret_cast<const float*>(set + sm.set_t1);
            const float* sC = reinterpret_cast<const float*>(set + sm.set_gates);
            if (lane == 0) sDt[b] = sC[kNTok];
            float x[kNTok];
            if (!bad) tmem_ld16(tmem_base + (uint32_t)b * 64u + (b ? 32u : 16u) + lane_sel, x);
#pragma unroll
            for (int t = 0; t < kNTok; ++t) x[t] = fmaf(-sC[t], x[t], __bfloat162float(sV[t * V + j]));
            float e[kNTok];
#pragma unroll
            for (int s = 0; s < kNTok; ++s) {
                float acc = 0.f;
#pragma unroll
                for (int t4 = 0; t4 <= s / 4; ++t4) {      // T1 is lower triangular
                    const float4 tt = *reinterpret_cast<const float4*>(sT1 + s * kNTok + t4 * 4);
                    acc = fmaf(tt.x, x[t4 * 4], acc);
                    acc = fmaf(tt.y, x[t4 * 4 + 1], acc);
                    acc = fmaf(tt.z, x[t4 * 4 + 2], acc);
                    acc = fmaf(tt.w, x[t4 * 4 + 3], acc);
                }
                e[s] = acc;
            }
            unsigned char* ehi = smem + sm.e;
            unsigned char* elo = ehi + 128u * CH * 2u;
#pragma unroll
            for (int v8 = 0; v8 < 2; ++v8) {
                uint32_t ohi[4], olo[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) split_bf16x2(e[v8 * 8 + 2 * q], e[v8 * 8 + 2 * q + 1], ohi[q], olo[q]);
                const uint32_t off = (gt & 7) * 16 + (gt >> 3) * SBO + v8 * LBO_M;
                *reinterpret_cast<uint4*>(ehi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                *reinterpret_cast<uint4*>(elo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
            }
            proxy_fence();
            tmem_st_wait();            // the d S_0 columns of pass A are in tensor memory
            tc_fence_before();
            bad = __any_sync(0xffffffffu, bad);
            if (lane == 0 && !bad) g_arrive(&bars[gErdy]);
        };
        auto wait_pro = [&](int b) {
            bad |= !mbar_wait_bounded(&bars[gPro + b], (phPro >> b) & 1u);
            phPro ^= 1u << b;
        };

        int cur = seq_get(0);
        if (cur >= 0) {
            wait_pro(0);
            pass_a(0, false);
            do_e(0);
            for (int k = 0; !bad; ++k) {
                const int b = k & 1;
                const int raw = seq_get(k + 1);
                if (raw < -1) { bad = true; break; }
                if (raw < 0) break;
                wait_pro(b ^ 1);
                pass_a(b ^ 1, true);
                // the E' operand buffer is read by K^T E' of tile k: that must be complete before it is rewritten
                bad |= !mbar_wait_bounded(&bars[gTfull + b], (phT >> b) & 1u);
                phT ^= 1u << b;
                do_e(b ^ 1);
            }
        } else if (cur < -1) {
            bad = true;
        }
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 3);
    } else if (warp >= 10) {
        // =========================== pass-B group: S_new written back, then the sketch rows ===========================
        // Pass A left d S_0 in the K^T E' accumulator, so the accumulator holds S_new: nothing is read from memory here.
        uint32_t phT = 0;
        bool bad = false;
        for (int k = 0; !bad; ++k) {
            const int raw = seq_get(k);
            if (raw < 0) { bad = raw < -1; break; }
            const int tile = raw;
            const int b = k & 1;
            const int h = tile / tiles_per_h, bb = tile - h * tiles_per_h;
            const size_t bh = (size_t)bb * H + h;
            float* So = p.state + bh * (size_t)K * V + j;
            bad |= !mbar_wait_bounded(&bars[gTfull + b], (phT >> b) & 1u);      // K^T E' and the sketch correction are complete
            phT ^= 1u << b;
            tc_fence_after();
            const float dtot = sDt[b];
#pragma unroll 2
            for (int c = 0; c < NCH; ++c) {
                if (!bad) {
                    float t[CH];
                    tmem_ld16(tmem_base + 128u + lane_sel + (uint32_t)(c * CH), t);
                    if (c == NCH / 2 - 1 || c == NCH - 1) {      // this warp is done with a half of the accumulator
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) g_arrive(&bars[gTfree + (c == NCH - 1 ? 1 : 0)]);
                    }
#pragma unroll
                    for (int ii = 0; ii < CH; ++ii) So[(size_t)(c * CH + ii) * V] = t[ii];
                }
            }
            // this warp has read its lanes of K^T E': the accumulator may be overwritten
            tc_fence_before();
            bad = __any_sync(0xffffffffu, bad);
            if (lane == 0 && !bad) g_arrive(&bars[gBdone + b]);
            // [U | o] = d S_0^T W + E'^T (K W) from the tile's slot of tensor memory
            if (!bad) {
                const uint32_t slot = tmem_base + (uint32_t)b * 64u + lane_sel;
                const uint32_t s_u0 = slot + (b ? 0u : 32u), s_cr = slot + (b ? 32u : 0u);
                auto rows = [&](auto bf) {
                    constexpr bool BF = decltype(bf)::value;
                    const size_t base = (bh * R) * (size_t)V + j;
                    for (int g0 = 0; g0 < R; g0 += 16) {
                        float u0[16], cr[16];
                        tmem_ld16(s_u0 + (uint32_t)g0, u0);
                        tmem_ld16(s_cr + (uint32_t)g0, cr);
                        if (g0 + 16 <= R) {
#pragma unroll
                            for (int e = 0; e < 16; ++e)
                                store_sketch_as<BF>(p, base + (size_t)(g0 + e) * V, fmaf(dtot, u0[e], cr[e]));
                        } else {
#pragma unroll
                            for (int e = 0; e < 16; ++e)
                                if (g0 + e < R) store_sketch_as<BF>(p, base + (size_t)(g0 + e) * V, fmaf(dtot, u0[e], cr[e]));
                        }
                    }
                };
                if (p.write_sketch) {
                    if (p.sketch_bf16) rows(std::true_type{}); else rows(std::false_type{});
                }
                if (p.out != nullptr) {       // exact output: the query column of this tile's group
                    const uint32_t qc = (uint32_t)(QA + 8 * b);
                    float ou, oc;
                    tmem_ld1x2(s_u0 + qc, s_cr + qc, ou, oc);
                    const float o = fmaf(dtot, ou, oc);
                    if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[bh * V + j] = __float2bfloat16_rn(o);
                    else reinterpret_cast<float*>(p.out)[bh * V + j] = o;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) g_arrive(&bars[gBufFree + b]);       // the slot is free for pass A of tile k + 2
            }
        }
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 11);
    } else if (warp == 8) {
        // =========================== MMA issue warp (one thread) ===========================
        if (lane == 0) {
            uint32_t phR = 0, phE = 0, phBuf = 0;
            bool bad = false;
            int where = 4;                  // which wait gave up (status detail): 41 slot free, 42 chunk ready, 43 E' ready, 44 K^T E' read
            const uint32_t sW = smem_u32(smem + sm.w);
            const uint32_t a2base = smem_u32(smem + sm.a2);
            // [P | U0](b) = S_0^T [K^T | Omega | q] chunk by chunk.  The keys of even tiles sit before [Omega | q] in the
            // operand and those of odd tiles after it, so each tile multiplies one 48-row window; the accumulator columns
            // follow the window: even tiles [free 16 | P 16 | U0 32], odd tiles [U0 32 | P 16 | free 16].
            auto pass_a = [&](int k) {
                const int b = k & 1;
                if (k >= 2) {                   // the slot still holds the sketch data of tile k - 2 until they are stored
                    if (!mbar_wait_bounded(&bars[gBufFree + b], (phBuf >> b) & 1u)) { bad = true; where = 41; return; }
                    phBuf ^= 1u << b;
                    tc_fence_after();
                }
                const uint32_t slot = tmem_base + (uint32_t)b * 64u;
                const uint32_t tmem_win = slot + (b ? 0u : 16u);
                const uint32_t tmem_u0 = slot + (b ? 0u : 32u);
                const uint32_t win = sW + (b ? 2u : 0u) * SBO;
#pragma unroll 2
                for (int c = 0; c < NCH; ++c) {
                    const int ab = c & (kA2 - 1);
                    if (!mbar_wait_bounded(&bars[gA2rdy + ab], (phR >> ab) & 1u)) { bad = true; where = 42; return; }
                    phR ^= 1u << ab;
                    tc_fence_after();
                    const uint32_t a2 = a2base + (uint32_t)ab * (2u * 128u * CH * 2u);
                    const uint64_t ahi = make_desc(a2, LBO_M, SBO);
                    const uint64_t alo = make_desc(a2 + 128u * CH * 2u, LBO_M, SBO);
                    const uint64_t whi = make_desc(win + (uint32_t)(c * (CH / 8)) * LBO_WH, LBO_WH, SBO);
                    const uint64_t wlo = make_desc(sW + w_lo_off + (uint32_t)(c * (CH / 8)) * LBO_WL, LBO_WL, SBO);
                    tc_mma_bf16(tmem_win, ahi, whi, idescA, c ? 1u : 0u);
                    tc_mma_bf16(tmem_win, alo, whi, idescA, 1u);
                    tc_mma_bf16(tmem_u0, ahi, wlo, idescU, 1u);
                    tc_commit(&bars[gA2free + ab]);
                    if (c == NCH - 1) tc_commit(&bars[gPfull + b]);
                }
            };
            auto step_e = [&](int k) {          // T = K^T E' (128 columns) and the sketch correction E'^T (K W) over the spent P
                const int b = k & 1;
                if (!mbar_wait_bounded(&bars[gErdy], phE)) { bad = true; where = 43; return; }
                phE ^= 1u;
                if (k >= 1) {                   // the pass-B group must have read K^T E' of the tile before
                    if (!mbar_wait_bounded(&bars[gBdone + (b ^ 1)], (uint32_t)((k - 1) >> 1) & 1u)) { bad = true; where = 44; return; }
                }
                tc_fence_after();
                const uint32_t tmem_t = tmem_base + 128u;
                const uint32_t tmem_c = tmem_base + (uint32_t)b * 64u + (b ? 32u : 0u);      // over the spent P and the free columns
                const uint32_t e = smem_u32(smem + sm.e);
                const uint64_t ehi = make_desc(e, LBO_M, SBO);
                const uint64_t elo = make_desc(e + 128u * CH * 2u, LBO_M, SBO);
                const uint64_t bt = make_desc(smem_u32(set_ptr(b) + sm.set_bt), LBO_M, SBO);
                const uint32_t bc = smem_u32(set_ptr(b) + sm.set_bc);
                const uint64_t bchi = make_desc(bc, 512u, SBO);
                const uint64_t bclo = make_desc(bc + 1024u, 512u, SBO);
                tc_mma_bf16(tmem_t, ehi, bt, idescT, 1u);      // onto d S_0, which pass A left there
                tc_mma_bf16(tmem_t, elo, bt, idescT, 1u);
                tc_mma_bf16(tmem_c, ehi, bchi, idescU, 0u);
                tc_mma_bf16(tmem_c, elo, bchi, idescU, 1u);
                tc_mma_bf16(tmem_c, ehi, bclo, idescU, 1u);
                tc_commit(&bars[gTfull + b]);
            };
            int cur = seq_get(0);
            if (cur >= 0) {
                pass_a(0);
                if (!bad) step_e(0);
                for (int k = 0; !bad; ++k) {
                    const int raw = seq_get(k + 1);
                    if (raw < -1) { bad = true; break; }
                    if (raw >= 0) pass_a(k + 1);
                    if (raw < 0 || bad) break;
                    step_e(k + 1);       // the pass-A group forms E'(k + 1) right after pass A of tile k + 1
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
                    if (!mbar_wait_bounded(&bars[gEmpty + stage], (uint32_t)(round - 1) & 1u)) { bad = true; return; }
                }
                uint64_t* bar = &bars[gFull + stage];
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
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 7);
    } else {
        // =========================== front group: ring-only operands, tile claiming ===========================
        const int fwarp = gt >> 5;
        int cur_h = -1;
        uint32_t phS = 0;
        bool dead = false;
        float* sGm = reinterpret_cast<float*>(smem + sm.mats);
        float* sPm = sGm + kNTok * kGS;
        float* sTm = sPm + kNTok * kGS;
        float* sBeta = sTm + kNTok * kGS;
        float* sAlpha = sBeta + kNTok;
        float* sDn = sAlpha + kNTok;
        float* sCum = sDn + kNTok;
        __nv_bfloat16* sWhi = reinterpret_cast<__nv_bfloat16*>(smem + sm.w);
        __nv_bfloat16* sWlo = sWhi + (size_t)64 * kK;

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
                for (int i = 1; i <= H; ++i) {
                    int hh = h_claim + i;
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

        const uint32_t stg_gate_bytes = n_ring > 0 ? (uint32_t)(2 * p.L * 4) : 0u;
        const uint32_t stg_bytes = (uint32_t)n_ring * 512u + stg_gate_bytes + (p.has_token ? 512u : 0u) + (p.q != nullptr ? 256u : 0u);
        // One bulk copy per thread from per-thread constants, spread over the four warps of the group (a warp's copies are
        // issued one after the other, ~400 cycles each): copy number c belongs to lane c / 4 of warp c % 4; copies 0..15
        // one key row each (ring rows, then the token's), 16..19 ring values, ring gates, token value, query row.
        const int cp_c = (gt & 31) < 5 ? (gt & 31) * 4 + (gt >> 5) : 32;
        const unsigned char* cp_base = nullptr;
        size_t cp_stride = 0;
        uint32_t cp_dst = 0, cp_bytes = 0;
        if (cp_c < n_ring) {
            cp_base = p.ring + (size_t)(p.tok_base + cp_c) * 256u; cp_stride = p.rl.head_bytes; cp_dst = (uint32_t)cp_c * kKeyRow; cp_bytes = 256u;
        } else if (cp_c == n_ring && p.has_token) {
            cp_base = reinterpret_cast<const unsigned char*>(p.k); cp_stride = (size_t)K * 2; cp_dst = (uint32_t)cp_c * kKeyRow; cp_bytes = 256u;
        }
        switch (cp_c) {
            case 16: cp_base = p.ring + p.rl.v_off + (size_t)p.tok_base * 256u; cp_stride = p.rl.head_bytes; cp_dst = sm.stg_v; cp_bytes = (uint32_t)n_ring * 256u; break;
            case 17: cp_base = p.ring + p.rl.beta_off; cp_stride = p.rl.head_bytes; cp_dst = sm.stg_gate; cp_bytes = stg_gate_bytes; break;
            case 18: cp_base = reinterpret_cast<const unsigned char*>(p.v); cp_stride = (size_t)V * 2; cp_dst = sm.stg_v + (uint32_t)n_ring * 256u; cp_bytes = p.has_token ? 256u : 0u; break;
            case 19: cp_base = reinterpret_cast<const unsigned char*>(p.q); cp_stride = (size_t)K * 2; cp_dst = sm.stg_q; cp_bytes = p.q != nullptr ? 256u : 0u; break;
            default: break;
        }
        auto stage_tile = [&](int tile) {       // whole group
            const int h = tile / tiles_per_h, bb = tile - h * tiles_per_h;
            const size_t bw = (size_t)bb * H + h;
            if (gt == 0) mbar_expect_tx(&bars[gStg], stg_bytes);      // (the phase cannot complete before this arrival, whatever the order of the copies)
            __syncwarp();
            if (cp_bytes) bulk_g2s(sStg + cp_dst, cp_base + bw * cp_stride, cp_bytes, &bars[gStg]);
        };
        // thread 0 resolves the claim, publishes it as entry k of the sequence and issues the next claim; the group then
        // requests the tile's rows
        auto next_tile = [&](int k) {          // whole group
            if (gt == 0) {
                const int nxt = claim_resolve();
                publish(k, nxt);
                if (nxt >= 0) claim_issue();
            }
            g_sync(2);                         // the published entry is the hand-off to the other threads
            const int nxt = seq_ring[k & 3];
            if (nxt >= 0) stage_tile(nxt);
        };
        // the first tile: claimed, published and its rows requested before anything else
        if (gt == 0) claim_issue();
        next_tile(0);
        // W padding columns and lo halves of the query columns hold zeros that no tile overwrites: written once
        for (uint32_t o = (uint32_t)gt * 16u; o < (64u + (uint32_t)NP) * kK * 2u; o += kGrp * 16u)
            *reinterpret_cast<uint4*>(smem + sm.w + o) = make_uint4(0, 0, 0, 0);
        // staged key rows beyond the tokens of a flush are never written by the copies: zero them once, so that the
        // products formed from all 16 rows stay finite
        for (uint32_t o = (uint32_t)gt * 16u; o < (uint32_t)kNTok * kKeyRow; o += kGrp * 16u)
            if ((int)(o / kKeyRow) >= n_tot) *reinterpret_cast<uint4*>(sStg + o) = make_uint4(0, 0, 0, 0);
        if (gt < 2 * 128) {
            const int sb = gt >> 6;           // 64 threads per set: 2 KB of K W operand each
            if (sb < 2) *reinterpret_cast<uint4*>(set_ptr(sb) + sm.set_bc + (uint32_t)(gt & 63) * 32u) = make_uint4(0, 0, 0, 0),
                        *reinterpret_cast<uint4*>(set_ptr(sb) + sm.set_bc + (uint32_t)(gt & 63) * 32u + 16u) = make_uint4(0, 0, 0, 0);
        }
        g_sync(2);

        for (int k = 0; !dead; ++k) {
            const int raw_tile = seq_get(k);
            if (raw_tile < 0) {
                if (raw_tile < -1) {
                    if (gt == 0) record_fault(p.status, kFaultUpdateWait, 8);
                    dead = true;
                }
                break;
            }
            const int tile = raw_tile;
            const int b = k & 1;
            const int h = tile / tiles_per_h, bb = tile - h * tiles_per_h;
            const size_t bh = (size_t)bb * H + h;
            unsigned char* set = set_ptr(b);

            // gates of the current token: requested early
            float tok_beta = 0.f, tok_a = 1.f;
            if (gt < kNTok && p.has_token) {
                tok_beta = p.beta[bh];
                tok_a = reinterpret_cast<const float*>(p.decay)[bh];
            }
            // the operand set of tile k - 2 is free once its K^T E' has completed (E' was formed before it was issued)
            if (k >= 2) {
                if (!g_wait(2, gt, &bars[gTfull + b], (uint32_t)((k - 2) >> 1) & 1u)) {
                    if (gt == 0) record_fault(p.status, kFaultUpdateWait, 9);
                    dead = true;
                    break;
                }
            }
            // the staged rows, gates and query row of this tile must have landed
            if (!g_wait(2, gt, &bars[gStg], phS)) {
                if (gt == 0) record_fault(p.status, kFaultUpdateWait, 6);
                dead = true;
                break;
            }
            phS ^= 1;

            // ---- key layouts, value rows, query column, gates ----
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int idx = gt + r * kGrp;
                const int t8 = idx & 7, a = ((idx >> 3) + t8) & 15, s = (idx >> 7) * 8 + t8;      // a diagonal: the 8 rows of a quarter warp at 8 different vectors (no bank conflicts at a 256-byte pitch)
                uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
                if (s < n_tot) {
                    kv = *reinterpret_cast<const uint4*>(sStg + (size_t)s * kKeyRow + a * 16);
                    vv = *reinterpret_cast<const uint4*>(sStg + sm.stg_v + (size_t)s * 256 + a * 16);
                }
                *reinterpret_cast<uint4*>(smem + sm.w + (s & 7) * 16 + ((s >> 3) + (b ? 6 : 0)) * SBO + a * LBO_WH) = kv;   // K-major, rows (b ? 48 : 0) + s of W
                *reinterpret_cast<uint4*>(set + sm.set_bt + (s & 7) * 16 + a * SBO + (s >> 3) * LBO_M) = kv;      // MN-major: (mn = i, k = s)
                *reinterpret_cast<uint4*>(set + sm.set_vv + (size_t)s * 256 + a * 16) = vv;
            }
            __nv_bfloat16 q_elem = __float2bfloat16_rn(0.f);         // written into W after the tile two before is done with it
            if (p.q != nullptr) q_elem = reinterpret_cast<const __nv_bfloat16*>(sStg + sm.stg_q)[gt];
            if (gt < kNTok) {
                const int s = gt;
                const float* sg = reinterpret_cast<const float*>(sStg + sm.stg_gate);
                float bt = 0.f, al = 1.f;
                if (s < n_ring) { bt = sg[p.tok_base + s]; al = sg[p.L + p.tok_base + s]; }
                else if (s < n_tot) { bt = tok_beta; al = tok_a; }
                sBeta[s] = bt;
                sAlpha[s] = al;
            }
            for (int idx = gt; idx < kNTok * kGS; idx += kGrp) sTm[idx] = 0.f;
            g_sync(2);

            // ---- products of decays (no quotients) and the Gram matrix <k_s, k_j> ----
            if (gt < kNTok) {
                const int s = gt;
                float al[kNTok];
#pragma unroll
                for (int i = 0; i < kNTok; ++i) al[i] = sAlpha[i];
                float pr = 1.f;                                   // Pm(j, s) = prod_{j < i <= s} alpha_i, for j = s-1 .. 0
#pragma unroll
                for (int jj = kNTok - 2; jj >= 0; --jj) {
                    if (jj < s) {
                        pr *= al[jj + 1];
                        sPm[s * kGS + jj] = pr;
                    }
                }
                sCum[s] = s < n_tot ? pr * al[0] : 0.f;           // prod_{i <= s} alpha_i
                float dn = 1.f;
#pragma unroll
                for (int i = 1; i < kNTok; ++i)
                    if (i > s && i < n_tot) dn *= al[i];
                sDn[s] = s < n_tot ? dn : 0.f;
            }
            if (fwarp >= 2) {     // 16 x 16 Gram matrix from the staged keys, one 16 x 8 block per warp
                const int nt = fwarp - 2;
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                const uint32_t abase = smem_u32(sStg) + (uint32_t)(lane & 15) * kKeyRow + (uint32_t)(lane >> 4) * 16u;
                const uint32_t bbase = smem_u32(sStg) + (uint32_t)(nt * 8 + (lane & 7)) * kKeyRow + (uint32_t)((lane >> 3) & 1) * 16u;
#pragma unroll
                for (int ks = 0; ks < K / 16; ++ks) {
                    uint32_t a[4], bbv[2];
                    g_ldmatrix_x4(abase + ks * 32, a);
                    g_ldmatrix_x2(bbase + ks * 32, bbv);
                    g_mma_16816(acc, a, bbv);
                }
                const int r0 = lane >> 2, c0 = nt * 8 + (lane & 3) * 2;
                sGm[r0 * kGS + c0] = acc[0];
                sGm[r0 * kGS + c0 + 1] = acc[1];
                sGm[(r0 + 8) * kGS + c0] = acc[2];
                sGm[(r0 + 8) * kGS + c0 + 1] = acc[3];
            }
            g_sync(2);
            // beta_s A_sj in place of the Gram entries (strictly lower triangle)
            if (gt < n_tot) {
                const int s = gt;
                const float bs = sBeta[s];
                for (int jj = 0; jj < s; ++jj) sGm[s * kGS + jj] *= bs * sPm[s * kGS + jj];
            }
            g_sync(2);
            // ---- T = (I + Bd A)^{-1} Bd by forward substitution: one column per thread, held in registers ----
            if (gt < kNTok) {
                const int c = gt;
                float tcol[kNTok];
#pragma unroll
                for (int s = 0; s < kNTok; ++s) {
                    float acc = 0.f;
#pragma unroll
                    for (int j4 = 0; j4 < (s + 3) / 4; ++j4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(sGm + s * kGS + j4 * 4);
                        if (j4 * 4 + 0 < s) acc = fmaf(l4.x, tcol[j4 * 4 + 0], acc);
                        if (j4 * 4 + 1 < s) acc = fmaf(l4.y, tcol[j4 * 4 + 1], acc);
                        if (j4 * 4 + 2 < s) acc = fmaf(l4.z, tcol[j4 * 4 + 2], acc);
                        if (j4 * 4 + 3 < s) acc = fmaf(l4.w, tcol[j4 * 4 + 3], acc);
                    }
                    tcol[s] = (s >= n_tot || s < c || c >= n_tot) ? 0.f : (s == c ? 1.f : -acc);
                }
                const float bc = sBeta[c];
#pragma unroll
                for (int s = 0; s < kNTok; ++s) sTm[s * kGS + c] = tcol[s] * bc;
            }
            g_sync(2);
            // ---- T1 = Dn T (rows and columns beyond the tokens are zero), C diagonal, total decay ----
            {
                float* sT1 = reinterpret_cast<float*>(set + sm.set_t1);
                float* sC = reinterpret_cast<float*>(set + sm.set_gates);
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int idx = gt + r * kGrp;
                    const int s = idx >> 4, t = idx & 15;
                    sT1[idx] = sDn[s] * sTm[s * kGS + t];
                }
                if (gt < kNTok) sC[gt] = sCum[gt];
                if (gt == 0) sC[kNTok] = sCum[n_tot - 1];
            }
            // ---- W = [Omega | q | q'] (and Omega in fp32 for the product below): the Omega part once per head index.
            // Pass A of the previous tile still reads W, so it is waited for first. ----
            if (h != cur_h) {
                if (k >= 1) {
                    if (!g_wait(2, gt, &bars[gPfull + (b ^ 1)], (uint32_t)((k - 1) >> 1) & 1u)) {
                        if (gt == 0) record_fault(p.status, kFaultUpdateWait, 10);
                        dead = true;
                        break;
                    }
                }
                if (p.write_sketch) {
                    const float* og = p.omega + (size_t)h * K * R;
                    for (int idx = gt; idx < K * R; idx += kGrp) {
                        const int i = idx / R, g = idx - i * R;
                        const float x = og[idx];
                        __nv_bfloat16 hi, lo;
                        split_bf16(x, hi, lo);
                        const uint32_t oc = (g & 7) * 16 + (g >> 3) * SBO + (i & 7) * 2;
                        sWhi[(oc + 2u * SBO + (i >> 3) * LBO_WH) >> 1] = hi;
                        sWlo[(oc + (i >> 3) * LBO_WL) >> 1] = lo;
                    }
                }
                cur_h = h;
                g_sync(2);
            }
            if (p.q != nullptr) {
                const int i = gt, g = QA + 8 * b;
                const uint32_t o2 = ((g & 7) * 16 + ((g >> 3) + 2) * SBO + (i >> 3) * LBO_WH + (i & 7) * 2) >> 1;
                sWhi[o2] = q_elem;
            }
            // ---- K W: 16 tokens x [Omega | q | q'] as mma.sync products of the staged keys with the hi and lo halves of W
            // (whose K-major core matrices are exactly the 8 x 8 B fragments), hi + lo, the B operand of the sketch
            // correction; one block of 8 columns per warp ----
            proxy_fence();
            g_sync(2);             // the query column and (after a change of head index) Omega are in W
            {
                const int nt = fwarp;
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                const uint32_t abase = smem_u32(sStg) + (uint32_t)(lane & 15) * kKeyRow + (uint32_t)(lane >> 4) * 16u;
                const uint32_t wrow = smem_u32(smem + sm.w) + (uint32_t)nt * SBO + (uint32_t)(lane & 7) * 16u;
                const uint32_t whbase = wrow + 2u * SBO + (uint32_t)((lane >> 3) & 1) * LBO_WH;
                const uint32_t wlbase = wrow + w_lo_off + (uint32_t)((lane >> 3) & 1) * LBO_WL;
#pragma unroll
                for (int ks = 0; ks < K / 16; ++ks) {
                    uint32_t a[4], bh2[2], bl2[2];
                    g_ldmatrix_x4(abase + ks * 32, a);
                    g_ldmatrix_x2(whbase + (uint32_t)(ks * 2) * LBO_WH, bh2);
                    g_ldmatrix_x2(wlbase + (uint32_t)(ks * 2) * LBO_WL, bl2);
                    g_mma_16816(acc, a, bh2);
                    g_mma_16816(acc, a, bl2);
                }
                __nv_bfloat16* bchi = reinterpret_cast<__nv_bfloat16*>(set + sm.set_bc);
                __nv_bfloat16* bclo = bchi + 512;
                auto put = [&](int s, int g, float x) {
                    __nv_bfloat16 hi, lo;
                    split_bf16(x, hi, lo);
                    const uint32_t o2 = ((g & 7) * 16 + (g >> 3) * SBO + (s >> 3) * 512 + (s & 7) * 2) >> 1;
                    bchi[o2] = hi;
                    bclo[o2] = lo;
                };
                const int r0 = lane >> 2, c0 = nt * 8 + (lane & 3) * 2;
                put(r0, c0, acc[0]);
                put(r0, c0 + 1, acc[1]);
                put(r0 + 8, c0, acc[2]);
                put(r0 + 8, c0 + 1, acc[3]);
            }
            proxy_fence();         // operand sets and W are read by MMAs (async proxy)
            g_sync(2);
            if (gt == 0) g_arrive(&bars[gPro + b]);
            next_tile(k + 1);      // the staging buffer has been read: the next tile's rows may come in

        }
        if (gt == 0) {     // scheduler counters back to zero once every CTA is done claiming
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
static int launch_gdn_pass(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    Params p = p_in;
    const int NP = ((((c.rank + 7) & ~7) + 16) + 15) & ~15;
    int ctas = 2;                                             // tensor memory: 256 of the SM's 512 columns per CTA
    if (p.max_warps_per_sm > 0 && p.max_warps_per_sm < 28) ctas = 1;
    const uint32_t budget = (228u * 1024u) / (uint32_t)ctas - 1024u;
    const GSmem fixed = make_gsmem(NP, c.buf_len, 0);
    if (fixed.total + 2u * fixed.sst_bytes > budget) return SKETCHSSM_UNSUPPORTED_SHAPE;
    int stages = (int)((budget - fixed.total) / fixed.sst_bytes);
    if (stages > kGStages) stages = kGStages;
    if (p.stages >= 2 && p.stages < stages) stages = p.stages;
    p.stages = stages;
    const GSmem sm = make_gsmem(NP, c.buf_len, stages);
    const long long n_tiles = (long long)c.batch * c.heads;
    long long grid = (long long)ctx->sm_count * ctas;
    if (grid > n_tiles) grid = n_tiles;
    auto kern = update_tc_ws_gdn_kernel;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)sm.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    if ((ctx->last_cuda_error = launch_kernel(kern, dim3((unsigned)grid), dim3(kGThreads), sm.total, stream, p, p.pdl != 0)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    return SKETCHSSM_OK;
}

// Returns SKETCHSSM_UNSUPPORTED_SHAPE outside this kernel's domain (the caller then uses another kernel).  A flush of more
// than 16 tokens is replayed in blocks of 16: every block is one pass over the state, and only the last one (which holds
// the current token) writes the sketch and the exact output.
int launch_update_tc_ws_gdn(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    if (c.kind != SKETCHSSM_GDN || c.io_dtype != SKETCHSSM_BF16 || c.dk != kK || c.dv != 128) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (c.rank > 16) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const int n_tot = p_in.n_before + (p_in.has_token ? 1 : 0);
    if (n_tot < 1 || n_tot > 4 * kNTok) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (ctx->sm_count == 0) {
        int dev = 0, sms = 0;
        if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        if ((ctx->last_cuda_error = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
        ctx->sm_count = sms;
    }
    const int passes = (n_tot + kNTok - 1) / kNTok;
    for (int ps = 0; ps < passes; ++ps) {
        Params p = p_in;
        p.tok_base = ps * kNTok;
        if (ps + 1 < passes) {          // 16 ring rows, state only
            p.n_before = kNTok;
            p.has_token = 0;
            p.q = nullptr;
            p.out = nullptr;
            p.write_sketch = 0;
        } else {
            p.n_before = p_in.n_before - ps * kNTok;
        }
        const int rc = launch_gdn_pass(ctx, p, stream);
        if (rc != SKETCHSSM_OK) return rc;
    }
    ctx->last_launches = passes;
    return SKETCHSSM_OK;
}

}  // namespace sketchssm
