// Warp-specialised state-update (flush) kernel for the Mamba-2 transition on tcgen05 + TMEM, sm_100a.
//
// Same arithmetic as the single-group tensor-core kernel (closed form of Eq. 3, sketch rows of Eq. 7):
//     S_new = d S_0 + sum_s w_s k_s v_s^T,   U[g, :] = S_new^T omega_g,   o = S_new^T q,
// with MMA 1 producing T = sum_s (w_s v_s) k_s^T in tensor memory and MMA 2 contracting the freshly formed
// S_new rows with [Omega | q].  The difference is the schedule.  A CTA holds two warp groups of 128 threads and one
// issue warp:
//
//   front group (warps 4-7), one tile AHEAD: turns the staged raw ring rows of tile i+1 into the MMA-1 operands
//       (token weights, w_s v_s split into bf16 hi + lo, keys, query columns), issues MMA 1 into the other half of a
//       double-buffered accumulator, and stores the sketch rows / exact output of tile i-1 from tensor memory;
//   stream group (warps 0-3): streams the state of tile i in 16-row chunks (S_new = d S_0 + T, written back once),
//       splits S_new into bf16 hi + lo in shared memory, warp by warp without a group barrier;
//   issue warp (warp 8, one thread): issues MMA 2 for a chunk once its four warps have delivered it, and keeps a ring
//       of shared-memory stages full of S_0 chunks by bulk copies (TMA) that run several chunks ahead and across tile
//       boundaries, so the bytes in flight per SM do not depend on registers and the global loads never drain.
//
// Everything that used to sit serially between two tiles' state streams (operand building, MMA-1 latency, sketch
// stores) now overlaps them.  The groups meet only through mbarriers; every wait is bounded.
//
// Domain: Mamba-2, bf16 I/O, K = 128, V in {64, 128}, rank <= 32 (the sketch accumulator [Omega | q | q'] re-uses
// the first 32 or 48 columns of T, read ahead by the stream group, which keeps a CTA at 256 TMEM columns and two
// CTAs per SM).
// W = [Omega | q-group A | q-group B]: consecutive tiles alternate between the two query groups, so the front group
// can write the next tile's query columns while MMA 2 of the current tile still reads the buffer (it then also reads
// half-written columns of the other group, whose outputs nobody uses).
#include <type_traits>
#include "internal.cuh"
#include "tc_common.cuh"

namespace sketchssm {

namespace {

using namespace tc;

constexpr int kWsThreads = 320;       // stream group (4 warps), front group (4 warps), MMA-2 issue warp, state-load warp
constexpr int kGroup = 128;

struct WsSmem {
    uint32_t op, a2, b2, w, w_stride, stg, stg_tile_head, stg_q, stg_blk, stg_blk_head, stg_blk_stride, bars, misc, sst, sst_bytes, total;
};

constexpr int kMaxStages = 8;

// operand set: a1_hi | a1_lo | b1, each 128 x KD1 bf16
__host__ __device__ inline WsSmem make_ws_smem(int NH, int NP, int V, int L, int stages, int stg_bufs) {
    WsSmem s;
    const uint32_t kd1 = (uint32_t)(kTokBlock * NH);
    uint32_t off = 0;
    s.op = off; off += 3u * 128u * kd1 * 2u;
    s.a2 = off; off += 2u * 2u * 128u * 16u * 2u;              // two 16-row chunk buffers, hi + lo
    s.b2 = off; off += 2u * (uint32_t)NP * kK * 2u;             // hi | lo
    s.w = off; s.w_stride = 2u * 208u * 4u; off += 2u * s.w_stride;     // per head: w_s (64), total decay; double-buffered
    // staging of raw ring rows, filled by bulk copies ahead of use: per head and tile the gates [2L] floats and the query
    // row; per head and block of 16 tokens the keys [16][256 B] and values [16][V*2 B], in one or two block buffers
    s.stg_q = ((uint32_t)(2 * L * 4) + 127u) & ~127u;
    s.stg_tile_head = s.stg_q + 256u;
    s.stg = off; off += (uint32_t)NH * s.stg_tile_head;
    s.stg_blk_head = 4096u + 16u * (uint32_t)V * 2u;
    s.stg_blk_stride = (uint32_t)NH * s.stg_blk_head;
    s.stg_blk = off; off += (uint32_t)stg_bufs * s.stg_blk_stride;
    s.bars = off; off += 256u;
    s.misc = off; off += 64u;
    off = (off + 127u) & ~127u;
    s.sst_bytes = 16u * 128u * 4u;                              // one stage: 16 state rows of every lane, fp32
    s.sst = off; off += (uint32_t)stages * s.sst_bytes;
    s.total = off;
    return s;
}

// barrier slots
enum { kBarT = 0, kBarPro = 2, kBarA2 = 4, kBarU = 6, kBarStg = 8, kBarBlk = 10, kBarA2Rdy = 11, kBarFull = 13,
       kBarEmpty = 13 + kMaxStages, kNumBars = 13 + 2 * kMaxStages };

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// named barrier over one 128-thread group
__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

// named barrier with an OR reduction of a per-thread flag
__device__ __forceinline__ bool group_or(int id, bool flag) {
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

// group-wide bounded wait for a barrier that is usually NOT yet complete: one warp polls, the others sleep in the
// named barrier.  Returns false to every thread of the group if the wait ran out.
__device__ __forceinline__ bool group_wait(int id, int gt, uint64_t* bar, uint32_t phase) {
    bool bad = false;
    if (gt < 32) bad = !mbar_wait_bounded(bar, phase);
    return !group_or(id, bad);
}

}  // namespace

// WIDE: the sketch accumulator [Omega | q | q'] takes 48 columns (rank 17..32) instead of 32.
template <int V, bool WIDE>
__global__ void __launch_bounds__(kWsThreads, 2) update_tc_ws_mamba2_kernel(const Params p) {
    constexpr int K = kK;
    constexpr int NH = 128 / V;
    constexpr int KD1 = kTokBlock * NH;
    constexpr uint32_t OPB = 128u * KD1 * 2u;              // bytes of one MMA-1 operand
    extern __shared__ __align__(1024) unsigned char smem[];

    const int tid = threadIdx.x, warp = tid >> 5;
    const int gt = tid & 127;
    const int R = p.R, H = p.H, B = p.B;
    const int QA = (R + 7) & ~7;                          // first column of query group A; group B follows 8 columns later
    const int NP = (QA + 16 + 15) & ~15;                  // 32, or 48 in the WIDE instantiation (chosen by the launcher)
    const int NS = p.stages;                              // state stages in shared memory (set by the launcher)
    const int n_ring = p.n_before, n_tot = n_ring + (p.has_token ? 1 : 0);
    const int stg_bufs = n_tot > kTokBlock ? 2 : 1;      // staging block buffers (the launcher sizes shared memory the same way)
    const WsSmem sm = make_ws_smem(NH, NP, V, p.L, NS, stg_bufs);
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
        for (int i = 0; i < kNumBars; ++i) {
            // chunk-ready and stage-empty barriers take one arrival per stream warp, the others a single arrival
            const bool per_warp = (i >= kBarA2Rdy && i < kBarA2Rdy + 2) || i >= kBarEmpty;
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

    // instruction descriptors: bf16 x bf16 -> fp32
    const uint32_t idesc1 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
    const uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)NP >> 3) << 17) | ((128u >> 4) << 24);
    // canonical no-swizzle layouts (byte offsets)
    //   MN-major (MMA 1): elem(mn, k) at (k%8)*16 + (mn%8)*2 + (mn/8)*128 + (k/8)*2048
    //   K-major  (MMA 2): elem(mn, k) at (mn%8)*16 + (mn/8)*128 + (k/8)*LBO + (k%8)*2,  LBO = 16*MN
    constexpr uint32_t LBO1 = 2048, SBO = 128, LBO2A = 2048;
    const uint32_t LBO2B = (uint32_t)NP * 16u;

    const int tiles_per_h = B / NH;
    const long long n_tiles = (long long)H * tiles_per_h;
    (void)n_tiles;
    const int n_blocks = (n_tot + kTokBlock - 1) / kTokBlock;

    // Tiles are claimed at run time (see the front group); the CTA's sequence of tile numbers travels through a small
    // ring in shared memory: entry k & 3 holds the k-th tile of this CTA (-1: no more), `seq_pub` counts entries.
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

    const int my_head = gt / V;           // which head of the tile this thread's TMEM lane belongs to
    const int j = gt % V;

    if (warp < 4) {
        // =========================== stream group: S_0 -> S_new, MMA 2 ===========================
        constexpr int CH = 16, NCH = K / CH;
        const int lane = tid & 31;
        uint32_t phT = 0, phP = 0, phA = 0;      // barrier phases, one bit per buffer
        int gc = 0, stage = 0;                   // chunks consumed so far, their stage and its phase
        uint32_t phF = 0;
        bool bad = false;
        for (int k = 0; !bad; ++k) {
            const int tile = seq_get(k);
            if (tile < 0) {
                bad = tile < -1;
                break;
            }
            const int b = k & 1;
            const int h = tile / tiles_per_h;
            const int b0 = (tile - h * tiles_per_h) * NH;
            const size_t bh = (size_t)(b0 + my_head) * H + h;
            float* So = p.state + bh * (size_t)K * V + j;
            const uint32_t tmem_t = tmem_base + (uint32_t)b * 128u;
            // operands-ready (plain arrive: orders the front group's shared-memory writes) and MMA 1 complete
            bad |= !mbar_wait_bounded(&bars[kBarPro + b], (phP >> b) & 1u);
            bad |= !mbar_wait_bounded(&bars[kBarT + b], (phT >> b) & 1u);
            phP ^= 1u << b;
            phT ^= 1u << b;
            tc_fence_after();
            const float dtot = n_tot > 0 ? reinterpret_cast<const float*>(smem + sm.w + (uint32_t)b * sm.w_stride)[my_head * 208 + 64] : 1.f;
            // T columns that UT will occupy (chunks 0 and 1, and chunk 2 when UT is 48 wide) are read before the first
            // MMA 2 overwrites them
            float t01[2 * CH];
            float t2[WIDE ? CH : 1];
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                // this chunk's S_0 rows have landed in their stage; once in registers the stage is released
                bad |= !mbar_wait_bounded(&bars[kBarFull + stage], phF);
                const float* sS = reinterpret_cast<const float*>(smem + sm.sst + (size_t)stage * sm.sst_bytes) + my_head * CH * V + j;
                float s0[CH];
#pragma unroll
                for (int ii = 0; ii < CH; ++ii) s0[ii] = sS[ii * V];
                float t[CH];
                if (n_blocks > 0 && !bad) {
                    if (c == 0) {
                        tmem_ld32(tmem_t + lane_sel, t01);
                        if constexpr (WIDE) tmem_ld16(tmem_t + lane_sel + 32u, t2);
                    }
                    if (c < 2) {
#pragma unroll
                        for (int ii = 0; ii < CH; ++ii) t[ii] = t01[c * CH + ii];
                    } else if (WIDE && c == 2) {
#pragma unroll
                        for (int ii = 0; ii < CH; ++ii) t[ii] = t2[WIDE ? ii : 0];
                    } else {
                        tmem_ld16(tmem_t + lane_sel + (uint32_t)(c * CH), t);
                    }
                } else {
#pragma unroll
                    for (int ii = 0; ii < CH; ++ii) t[ii] = 0.f;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[kBarEmpty + stage]);
                if (gc >= 2) {       // chunk buffer c&1 was read by the MMAs issued two chunks ago
                    bad |= !mbar_wait_bounded(&bars[kBarA2 + (c & 1)], (phA >> (c & 1)) & 1u);
                    phA ^= 1u << (c & 1);
                }
                unsigned char* a2hi = smem + sm.a2 + (size_t)(c & 1) * (2u * 128u * CH * 2u);
                unsigned char* a2lo = a2hi + 128u * CH * 2u;
#pragma unroll
                for (int v8 = 0; v8 < CH / 8; ++v8) {
                    uint32_t ohi[4], olo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int i0 = v8 * 8 + 2 * e;
                        const float x0 = fmaf(dtot, s0[i0], t[i0]), x1 = fmaf(dtot, s0[i0 + 1], t[i0 + 1]);
                        if (p.write_state && !bad) {
                            So[(size_t)(c * CH + i0) * V] = x0;
                            So[(size_t)(c * CH + i0 + 1) * V] = x1;
                        }
                        split_bf16x2(x0, x1, ohi[e], olo[e]);
                    }
                    const uint32_t off = (gt & 7) * 16 + (gt >> 3) * SBO + v8 * LBO2A;
                    *reinterpret_cast<uint4*>(a2hi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                    *reinterpret_cast<uint4*>(a2lo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
                }
                // this warp's 32 rows of the chunk are written (and its T columns read): tell the issue warp
                proxy_fence();
                tc_fence_before();
                bad = __any_sync(0xffffffffu, bad);
                if (lane == 0 && !bad) mbar_arrive(&bars[kBarA2Rdy + (c & 1)]);
                ++gc;
                if (++stage == NS) { stage = 0; phF ^= 1u; }
            }
        }
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 3);
    } else if (warp == 8) {
        // =========================== MMA-2 issue warp (one thread) ===========================
        if (gt == 0) {
            constexpr int CH = 16, NCH = K / CH;
            uint32_t phR = 0;                    // chunk-ready phases (bit per buffer)
            bool bad = false;
            const uint32_t sB2 = smem_u32(smem + sm.b2);
            for (int k = 0; !bad; ++k) {
                const int tile = seq_get(k);
                if (tile < 0) {
                    bad = tile < -1;
                    break;
                }
                const int b = k & 1;
                const uint32_t tmem_t = tmem_base + (uint32_t)b * 128u;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    if (!mbar_wait_bounded(&bars[kBarA2Rdy + (c & 1)], (phR >> (c & 1)) & 1u)) { bad = true; break; }
                    phR ^= 1u << (c & 1);
                    tc_fence_after();
                    const uint32_t a2 = smem_u32(smem + sm.a2) + (uint32_t)(c & 1) * (2u * 128u * CH * 2u);
                    const uint32_t kb = (uint32_t)(c * (CH / 8)) * LBO2B;      // W rows of this K-step
                    const uint64_t ahi = make_desc(a2, LBO2A, SBO);
                    const uint64_t alo = make_desc(a2 + 128u * CH * 2u, LBO2A, SBO);
                    const uint64_t bhi = make_desc(sB2 + kb, LBO2B, SBO);
                    const uint64_t blo = make_desc(sB2 + (uint32_t)NP * kK * 2u + kb, LBO2B, SBO);
                    tc_mma_bf16(tmem_t, ahi, bhi, idesc2, c ? 1u : 0u);
                    tc_mma_bf16(tmem_t, alo, bhi, idesc2, 1u);
                    tc_mma_bf16(tmem_t, ahi, blo, idesc2, 1u);
                    tc_commit(&bars[kBarA2 + (c & 1)]);
                    if (c == NCH - 1) tc_commit(&bars[kBarU + b]);     // everything of this tile: UT is complete
                }
            }
            if (bad) record_fault(p.status, kFaultUpdateWait, 4);
        }
    } else if (warp == 9) {
        // =========================== state-load warp: keeps the ring of S_0 stages full (one lane per head) ===========
        constexpr int CH = 16, NCH = K / CH;
        const int lane = gt & 31;
        int stage = 0, round = 0;            // stage to fill next; how often the ring has wrapped
        bool bad = false;
        for (int k = 0; !bad; ++k) {
            const int tile = seq_get(k);
            if (tile < 0) {
                bad = tile < -1;
                break;
            }
            const int h = tile / tiles_per_h;
            const int b0 = (tile - h * tiles_per_h) * NH;
            const float* src = p.state + ((size_t)(b0 + (lane < NH ? lane : 0)) * H + h) * (size_t)K * V;
            for (int c = 0; c < NCH; ++c) {
                if (round > 0) {     // the stage was released by all four stream warps
                    if (!mbar_wait_bounded(&bars[kBarEmpty + stage], (uint32_t)(round - 1) & 1u)) { bad = true; break; }
                }
                uint64_t* bar = &bars[kBarFull + stage];
                if (lane == 0) mbar_expect_tx(bar, sm.sst_bytes);
                __syncwarp();
                if (lane < NH)
                    bulk_g2s(smem + sm.sst + (size_t)stage * sm.sst_bytes + (size_t)lane * CH * V * 4,
                             src + (size_t)c * CH * V, (uint32_t)(CH * V * 4), bar);
                if (++stage == NS) { stage = 0; ++round; }
            }
        }
        if (bad && lane == 0) record_fault(p.status, kFaultUpdateWait, 7);
    } else {
        // =========================== front group: operands, MMA 1, sketch stores ===========================
        const int fwarp = gt >> 5;
        int cur_h = -1;                       // head index whose Omega sits in W
        int ops_built = 0;                    // MMA-1 operand sets written so far (single buffer)
        int prev_tile = -1, last_b = 0;       // the tile whose sketch rows are still to be stored (-1: none) and its buffer
        uint32_t phU = 0, phB = 0;
        bool dead = false;

        // ---- tile claiming (thread 0 of the group) ----
        // Head index h owns a counter of tiles handed out.  A CTA keeps claiming tiles of the head index it works on
        // (its Omega stays in shared memory); when that is exhausted it moves to the head index with the most tiles left.
        // The claim for the tile after next is in flight while a tile's operands are built.  The last CTA to finish
        // zeroes the counters again, so they are zero between launches.
        int* sched = p.status + kStatusInts;  // [0] CTAs finished, [4 + h] tiles of head index h handed out
        int* cnt = sched + 4;
        int h_claim = (int)(((long long)blockIdx.x * H) / gridDim.x);
        int t_raw = 0;
        auto claim_issue = [&]() { t_raw = atomicAdd(&cnt[h_claim], 1); };
        auto claim_resolve = [&]() -> int {   // tile number, or -1 when every tile has been handed out
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

        // Raw ring rows travel to shared memory block by block (16 tokens per head) by bulk copies that run ahead of
        // their use: with one block per tile the next tile's block is requested while this tile's operands are built,
        // with several blocks per tile two block buffers alternate.  A tile's gates and query rows come with its first block.
        const int n_stage_blocks = n_blocks > 0 ? n_blocks : 1;       // a tile without tokens still stages its query rows
        const uint32_t stg_gate_bytes = n_ring > 0 ? (uint32_t)(2 * p.L * 4) : 0u;
        auto block_bytes = [&](int blk) -> uint32_t {
            int rows = n_ring - blk * kTokBlock;
            rows = rows < 0 ? 0 : (rows > kTokBlock ? kTokBlock : rows);
            const bool tok = p.has_token && n_ring / kTokBlock == blk;
            uint32_t by = (uint32_t)rows * 256u + (uint32_t)rows * V * 2u + (tok ? 256u + (uint32_t)V * 2u : 0u);
            if (blk == 0) by += stg_gate_bytes + (p.q != nullptr ? 256u : 0u);
            return (uint32_t)NH * by;
        };
        const bool staging = block_bytes(0) > 0;
        // One bulk copy per thread, spread over the warps of the group (a warp's copies are issued one after the other,
        // ~400 cycles each): copy number c = head * 6 + kind, kind = block keys, block values, token key, token value,
        // gates, query row.  With one token block per tile all four warps share the copies (lane c / 4 of warp c % 4) and
        // thread 0 issues MMA 1; with several blocks per tile, where the front group is the limit, the first three warps
        // share them (lane c / 3 of warp c % 3) and the fourth warp issues MMA 1 meanwhile.  Base pointer and bytes per
        // (batch, head) are per-thread constants.
        const bool split_issue = n_blocks > 1;
        const int mma_thread = split_issue ? 3 * 32 : 0;
        const int cp_c = split_issue ? (((gt >> 5) < 3 && (gt & 31) < 2 * NH) ? (gt & 31) * 3 + (gt >> 5) : 6 * NH)
                                     : ((gt & 31) < 3 * NH ? (gt & 31) * 4 + (gt >> 5) : 6 * NH);
        const int cp_hd = cp_c / 6, cp_kind = cp_c - cp_hd * 6;
        const unsigned char* cp_base = nullptr;
        size_t cp_stride = 0;
        if (cp_c < 6 * NH) {
            switch (cp_kind) {
                case 0: cp_base = p.ring; cp_stride = p.rl.head_bytes; break;
                case 1: cp_base = p.ring + p.rl.v_off; cp_stride = p.rl.head_bytes; break;
                case 2: cp_base = reinterpret_cast<const unsigned char*>(p.k); cp_stride = (size_t)K * 2; break;
                case 3: cp_base = reinterpret_cast<const unsigned char*>(p.v); cp_stride = (size_t)V * 2; break;
                case 4: cp_base = p.ring + p.rl.beta_off; cp_stride = p.rl.head_bytes; break;
                default: cp_base = reinterpret_cast<const unsigned char*>(p.q); cp_stride = (size_t)K * 2; break;
            }
        }
        auto stage_block = [&](int tile, int blk, int buf) {       // whole group
            const int h = tile / tiles_per_h;
            const int b0 = (tile - h * tiles_per_h) * NH;
            int rows = n_ring - blk * kTokBlock;
            rows = rows < 0 ? 0 : (rows > kTokBlock ? kTokBlock : rows);
            const bool tok = p.has_token && n_ring / kTokBlock == blk;
            const int tok_row = n_ring - blk * kTokBlock;
            uint64_t* bar = &bars[kBarStg + buf];
            if (gt == 0) mbar_expect_tx(bar, block_bytes(blk));      // (the phase cannot complete before this arrival, whatever the order of the copies)
            __syncwarp();
            if (cp_c < 6 * NH) {
                const size_t bw = (size_t)(b0 + cp_hd) * H + h;
                const uint32_t blk_dst = sm.stg_blk + (uint32_t)buf * sm.stg_blk_stride + (uint32_t)cp_hd * sm.stg_blk_head;
                const uint32_t tile_dst = sm.stg + (uint32_t)cp_hd * sm.stg_tile_head;
                uint32_t bytes = 0, dst = 0, src_off = 0;
                if (cp_kind == 0) { bytes = (uint32_t)rows * 256u; dst = blk_dst; src_off = (uint32_t)blk * kTokBlock * 256u; }
                else if (cp_kind == 1) { bytes = (uint32_t)rows * V * 2u; dst = blk_dst + 4096u; src_off = (uint32_t)blk * kTokBlock * V * 2u; }
                else if (cp_kind == 2) { bytes = tok ? 256u : 0u; dst = blk_dst + (uint32_t)tok_row * 256u; }
                else if (cp_kind == 3) { bytes = tok ? (uint32_t)V * 2u : 0u; dst = blk_dst + 4096u + (uint32_t)tok_row * V * 2u; }
                else if (cp_kind == 4) { bytes = blk == 0 ? stg_gate_bytes : 0u; dst = tile_dst; }
                else { bytes = (blk == 0 && p.q != nullptr) ? 256u : 0u; dst = tile_dst + sm.stg_q; }
                if (bytes) bulk_g2s(smem + dst, cp_base + bw * cp_stride + src_off, bytes, bar);
            }
        };
        // producer cursor of the staging ring (kept by every thread of the group): the next block to request, and how
        // many tiles have been published
        int sq_tile = 0, sq_blk = 0, sq_idx = 0, pub_k = 0;
        auto stage_next = [&]() {           // whole group: request the next block in sequence; entering a new tile claims it
            if (sq_tile < 0) return;
            if (sq_blk == 0) {              // the claim issued a tile ago is resolved only now, the one after it goes out
                if (gt == 0) {
                    const int nxt = claim_resolve();
                    publish(pub_k, nxt);
                    if (nxt >= 0) claim_issue();
                }
                group_sync(2);              // the published entry is the hand-off to the other threads
                sq_tile = seq_ring[pub_k & 3];
                ++pub_k;
                if (sq_tile < 0) return;
            }
            if (staging) stage_block(sq_tile, sq_blk, sq_idx % stg_bufs);
            ++sq_idx;
            if (++sq_blk == n_stage_blocks) sq_blk = 0;
        };
        int cq_idx = 0;                     // blocks consumed by the group so far
        // sketch rows and exact output of a finished tile: UT sits in the first NP columns of that tile's accumulator
        auto store_ut = [&](int tile, int b) -> bool {
            const int h = tile / tiles_per_h;
            const int b0 = (tile - h * tiles_per_h) * NH;
            const size_t bh = (size_t)(b0 + my_head) * H + h;
            if (!group_wait(2, gt, &bars[kBarU + b], (phU >> b) & 1u)) return false;
            phU ^= 1u << b;
            tc_fence_after();
            // sketch rows: column g of the accumulator is U[g][j]; full groups of 16 ranks take the unpredicated stores
            const uint32_t trow = tmem_base + (uint32_t)b * 128u + lane_sel;
            auto rows = [&](auto bf) {
                constexpr bool BF = decltype(bf)::value;
                const size_t base = (bh * R) * (size_t)V + j;
                for (int g0 = 0; g0 < R; g0 += 16) {
                    float u[16];
                    tmem_ld16(trow + (uint32_t)g0, u);
                    if (g0 + 16 <= R) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) store_sketch_as<BF>(p, base + (size_t)(g0 + e) * V, u[e]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            if (g0 + e < R) store_sketch_as<BF>(p, base + (size_t)(g0 + e) * V, u[e]);
                    }
                }
            };
            if (p.write_sketch) {
                if (p.sketch_bf16) rows(std::true_type{}); else rows(std::false_type{});
            }
            if (p.out != nullptr) {       // exact output: the query column of this head
                const float o = tmem_ld1(trow + (uint32_t)(QA + 8 * b + my_head));
                if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[bh * V + j] = __float2bfloat16_rn(o);
                else reinterpret_cast<float*>(p.out)[bh * V + j] = o;
            }
            tc_fence_before();     // ordered before the next MMA 1 into this accumulator by the group barriers that follow
            return true;
        };

        if (gt == 0) claim_issue();
        stage_next();
        if (stg_bufs > 1 && n_stage_blocks > 1) stage_next();
        // W (padding columns, lo halves of the query columns) and the MMA-1 operands (off-diagonal head blocks) hold
        // zeros that no tile ever overwrites: written once
        for (uint32_t o = (uint32_t)gt * 16u; o < 2u * (uint32_t)NP * kK * 2u; o += kGroup * 16u)
            *reinterpret_cast<uint4*>(smem + sm.b2 + o) = make_uint4(0, 0, 0, 0);
        for (uint32_t o = (uint32_t)gt * 16u; o < 3u * OPB; o += kGroup * 16u)
            *reinterpret_cast<uint4*>(smem + sm.op + o) = make_uint4(0, 0, 0, 0);
        group_sync(2);

        for (int k = 0; !dead; ++k) {
            const int tile = seq_get(k);
            if (tile < 0) {
                if (tile < -1) {
                    if (gt == 0) record_fault(p.status, kFaultUpdateWait, 8);
                    dead = true;
                }
                break;
            }
            const int b = k & 1;
            const int h = tile / tiles_per_h;
            const int b0 = (tile - h * tiles_per_h) * NH;
            __nv_bfloat16* sB2hi = reinterpret_cast<__nv_bfloat16*>(smem + sm.b2);
            __nv_bfloat16* sB2lo = sB2hi + (size_t)NP * kK;
            float* sW = reinterpret_cast<float*>(smem + sm.w + (uint32_t)b * sm.w_stride);
            unsigned char* sA1hi = smem + sm.op;
            unsigned char* sA1lo = sA1hi + OPB;
            unsigned char* sB1 = sA1lo + OPB;

            // gates of the current token (one warp per head needs them for the weight scan): requested early
            float tok_beta = 0.f, tok_a = 1.f;
            if (fwarp < NH && p.has_token) {
                const size_t bw = (size_t)(b0 + fwarp) * H + h;
                tok_beta = p.beta[bw];
                tok_a = reinterpret_cast<const float*>(p.decay)[bw];
            }
            // ---- W = [Omega | q | q'] hi/lo, K-major; the Omega part once per head index.  MMA 2 of the previous tile
            // still reads W, so that tile is finished (and its sketch rows stored) first. ----
            if (h != cur_h) {
                if (prev_tile >= 0) {
                    if (!store_ut(prev_tile, b ^ 1)) {
                        if (gt == 0) record_fault(p.status, kFaultUpdateWait, 5);
                        dead = true;
                        break;
                    }
                    prev_tile = -1;
                    group_sync(2);
                }
                const float* og = p.omega + (size_t)h * K * R;
                if (!p.write_sketch) {
                    // no sketch: the Omega columns stay zero (written once before the tile loop)
                } else if ((R & 3) == 0) {
                    // four ranks of one state row per step; all loads of a thread are in flight together
                    const int per_row = R >> 2, items = K * per_row;
                    for (int base = 0; base < items; base += 4 * kGroup) {
                        float4 x[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int idx = base + u * kGroup + gt;
                            x[u] = idx < items ? *reinterpret_cast<const float4*>(og + (size_t)idx * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int idx = base + u * kGroup + gt;
                            if (idx < items) {
                                const int i = idx / per_row, g4 = (idx - i * per_row) * 4;
                                const float xv[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int g = g4 + e;
                                    __nv_bfloat16 hi, lo;
                                    split_bf16(xv[e], hi, lo);
                                    const uint32_t o2 = ((g & 7) * 16 + (g >> 3) * SBO + (i >> 3) * LBO2B + (i & 7) * 2) >> 1;
                                    sB2hi[o2] = hi;
                                    sB2lo[o2] = lo;
                                }
                            }
                        }
                    }
                } else {
                    for (int idx = gt; idx < K * R; idx += kGroup) {
                        const int i = idx / R, g = idx % R;
                        __nv_bfloat16 hi, lo;
                        split_bf16(og[idx], hi, lo);
                        const uint32_t o2 = ((g & 7) * 16 + (g >> 3) * SBO + (i >> 3) * LBO2B + (i & 7) * 2) >> 1;
                        sB2hi[o2] = hi;
                        sB2lo[o2] = lo;
                    }
                }
                cur_h = h;
            }
            // the first block of this tile (with its gates and query rows) must have landed
            if (staging) {
                if (!group_wait(2, gt, &bars[kBarStg + cq_idx % stg_bufs], (uint32_t)(cq_idx / stg_bufs) & 1u)) {
                    if (gt == 0) record_fault(p.status, kFaultUpdateWait, 6);
                    dead = true;
                    break;
                }
            }
            if (p.q != nullptr) {       // query columns of this tile's group (bf16-exact: lo = 0)
                for (int idx = gt; idx < K * NH; idx += kGroup) {
                    const int i = idx % K, hd = idx / K, g = QA + 8 * b + hd;
                    const uint32_t o2 = ((g & 7) * 16 + (g >> 3) * SBO + (i >> 3) * LBO2B + (i & 7) * 2) >> 1;
                    sB2hi[o2] = reinterpret_cast<const __nv_bfloat16*>(sStg + (size_t)hd * sm.stg_tile_head + sm.stg_q)[i];
                }
            }
            // ---- token weights w_s = beta_s prod_{j>s} a_j and the total decay: one warp per head, suffix scan ----
            if (fwarp < NH) {
                const int hd = fwarp, lane = gt & 31;
                const float* sg = reinterpret_cast<const float*>(sStg + (size_t)hd * sm.stg_tile_head);
                float suf = 1.f;          // product of the decays of all later tokens
                for (int base = ((n_tot + 31) & ~31) - 32; base >= 0; base -= 32) {
                    const int s = base + lane;
                    float beta = 0.f, a = 1.f;
                    if (s < n_ring) { beta = sg[s]; a = sg[p.L + s]; }
                    else if (s < n_tot) { beta = tok_beta; a = tok_a; }
                    // inclusive suffix product of a over lanes >= lane
                    float incl = a;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const float other = __shfl_down_sync(0xffffffffu, incl, o);
                        if (lane + o < 32) incl *= other;
                    }
                    float excl = __shfl_down_sync(0xffffffffu, incl, 1);
                    if (lane == 31) excl = 1.f;
                    if (s < n_tot) sW[hd * 208 + s] = beta * excl * suf;
                    suf *= __shfl_sync(0xffffffffu, incl, 0);
                }
                if (lane == 0) sW[hd * 208 + 64] = suf;
            }
            proxy_fence();         // W is read by MMA 2 (async proxy)
            group_sync(2);

            // ---- MMA 1 over blocks of kTokBlock tokens per head ----
            for (int blk = 0; blk < n_blocks; ++blk) {
                if (ops_built > 0) {      // the previous MMA-1 block (of this or the previous tile) must have read the operand buffers
                    if (!group_wait(2, gt, &bars[kBarBlk], phB)) {
                        if (gt == 0) record_fault(p.status, kFaultUpdateWait, 1);
                        dead = true;
                        break;
                    }
                    phB ^= 1;
                    tc_fence_after();
                }
                // Operand rows are moved 16 bytes per thread.  The 8 lanes of a quarter warp take the 8 token rows of a core
                // matrix, each at a different 8-element vector (a diagonal), so that neither the reads of the staged rows
                // (row pitch 256 or 128 bytes) nor the writes of the core matrices meet in a bank.
                {
                    // rows come from the block's staging buffer; only the diagonal head blocks of A are written
                    if (blk > 0 && staging) {      // (the first block was waited for above)
                        if (!group_wait(2, gt, &bars[kBarStg + cq_idx % stg_bufs], (uint32_t)(cq_idx / stg_bufs) & 1u)) {
                            if (gt == 0) record_fault(p.status, kFaultUpdateWait, 6);
                            dead = true;
                            break;
                        }
                    }
                    const unsigned char* sBlk = smem + sm.stg_blk + (size_t)(cq_idx % stg_bufs) * sm.stg_blk_stride;
                    const int s_base = blk * kTokBlock;
                    constexpr int NB = KD1 * (K / 8) / kGroup;          // B-operand vectors per thread
                    uint4 kv[NB];
#pragma unroll
                    for (int r = 0; r < NB; ++r) {
                        const int idx = gt + r * kGroup;
                        const int a = ((idx >> 3) + (idx & 7)) % (K / 8), sp = (idx & 7) + 8 * (idx / (8 * (K / 8)));
                        const int hd = sp / kTokBlock, s = sp % kTokBlock;
                        kv[r] = s_base + s < n_tot ? *reinterpret_cast<const uint4*>(sBlk + (size_t)hd * sm.stg_blk_head + (size_t)s * 256 + a * 16)
                                                   : make_uint4(0, 0, 0, 0);
                    }
                    constexpr int NA = NH * kTokBlock * (V / 8) / kGroup;      // diagonal A-operand vectors per thread
                    uint4 vv[NA];
                    float wv[NA];
#pragma unroll
                    for (int r = 0; r < NA; ++r) {
                        const int it = gt + r * kGroup;
                        const int t8 = it & 7, a = ((it >> 3) + t8) % (V / 8), rest = it / V;
                        const int hd = rest >> 1, s = (rest & 1) * 8 + t8;
                        const bool live = s_base + s < n_tot;
                        vv[r] = live ? *reinterpret_cast<const uint4*>(sBlk + (size_t)hd * sm.stg_blk_head + 4096 + (size_t)s * V * 2 + a * 16)
                                     : make_uint4(0, 0, 0, 0);
                        wv[r] = live ? sW[hd * 208 + s_base + s] : 0.f;
                    }
#pragma unroll
                    for (int r = 0; r < NB; ++r) {
                        const int idx = gt + r * kGroup;
                        const int a = ((idx >> 3) + (idx & 7)) % (K / 8), sp = (idx & 7) + 8 * (idx / (8 * (K / 8)));
                        *reinterpret_cast<uint4*>(sB1 + (sp & 7) * 16 + a * SBO + (sp >> 3) * LBO1) = kv[r];
                    }
#pragma unroll
                    for (int r = 0; r < NA; ++r) {
                        const int it = gt + r * kGroup;
                        const int t8 = it & 7, a = ((it >> 3) + t8) % (V / 8), rest = it / V;
                        const int hd = rest >> 1, sp = hd * kTokBlock + (rest & 1) * 8 + t8;
                        const int a128 = hd * (V / 8) + a;
                        const uint32_t vin[4] = {vv[r].x, vv[r].y, vv[r].z, vv[r].w};
                        uint32_t ohi[4], olo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float f0 = wv[r] * __uint_as_float(vin[e] << 16), f1 = wv[r] * __uint_as_float(vin[e] & 0xffff0000u);
                            split_bf16x2(f0, f1, ohi[e], olo[e]);
                        }
                        const uint32_t off = (sp & 7) * 16 + a128 * SBO + (sp >> 3) * LBO1;
                        *reinterpret_cast<uint4*>(sA1hi + off) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
                        *reinterpret_cast<uint4*>(sA1lo + off) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
                    }
                    ++cq_idx;
                }
                proxy_fence();
                tc_fence_before();
                group_sync(2);
                ++ops_built;
                if (gt == mma_thread) {
                    tc_fence_after();
                    const uint32_t tmem_t = tmem_base + (uint32_t)b * 128u;
#pragma unroll
                    for (int ks = 0; ks < KD1 / 16; ++ks) {
                        const uint64_t bd = make_desc(smem_u32(sB1) + ks * 2 * LBO1, LBO1, SBO);
                        tc_mma_bf16(tmem_t, make_desc(smem_u32(sA1hi) + ks * 2 * LBO1, LBO1, SBO), bd, idesc1, (blk | ks) ? 1u : 0u);
                        tc_mma_bf16(tmem_t, make_desc(smem_u32(sA1lo) + ks * 2 * LBO1, LBO1, SBO), bd, idesc1, 1u);
                    }
                    tc_commit(&bars[kBarBlk]);
                    if (blk + 1 == n_blocks) {
                        tc_commit(&bars[kBarT + b]);
                        mbar_arrive(&bars[kBarPro + b]);      // after the group barrier: W, weights and decay are written
                    }
                }
                stage_next();        // the block buffer just read is free again
            }
            if (dead) break;
            if (n_blocks == 0) {
                // no token to replay: nothing reads the staging buffer after the query columns; T counts as zero
                ++cq_idx;
                group_sync(2);
                if (gt == 0) {
                    mbar_arrive(&bars[kBarT + b]);
                    mbar_arrive(&bars[kBarPro + b]);
                }
                stage_next();
            }

            // ---- sketch rows and exact output of the previous tile, once the stream group has finished it ----
            if (prev_tile >= 0) {
                if (!store_ut(prev_tile, b ^ 1)) {
                    if (gt == 0) record_fault(p.status, kFaultUpdateWait, 5);
                    dead = true;
                }
            }
            prev_tile = tile;
            last_b = b;
        }
        if (!dead && prev_tile >= 0) {
            // the last tile used buffer (number of tiles - 1) & 1; phU tells which buffer has an odd number of stores
            if (!store_ut(prev_tile, last_b) && gt == 0) record_fault(p.status, kFaultUpdateWait, 5);
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

// Returns SKETCHSSM_UNSUPPORTED_SHAPE when the configuration is outside this kernel's domain (the caller then
// uses the single-group tensor-core kernel or the CUDA-core kernel).
int launch_update_tc_ws(Ctx* ctx, const Params& p_in, cudaStream_t stream) {
    const sketchssm_config& c = ctx->cfg;
    if (c.kind != SKETCHSSM_MAMBA2 || c.io_dtype != SKETCHSSM_BF16 || c.dk != kK) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (c.dv != 64 && c.dv != 128) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const int NH = 128 / c.dv;
    if (c.batch % NH != 0) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (c.rank > 32) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const int NP = ((((c.rank + 7) & ~7) + 16) + 15) & ~15;      // [Omega | q | q']: 32 or 48 columns
    Params p = p_in;
    if (ctx->sm_count == 0) {
        int dev = 0, sms = 0;
        if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        if ((ctx->last_cuda_error = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
        ctx->sm_count = sms;
    }
    // two CTAs per SM (tensor memory: 256 of the SM's 512 columns each) unless capped; the shared memory left after the
    // operand buffers holds the ring of state stages
    int ctas = 2;
    if (p.max_warps_per_sm > 0 && p.max_warps_per_sm < 18) ctas = 1;
    const uint32_t budget = (228u * 1024u) / (uint32_t)ctas - 1024u;
    const int n_tot = p.n_before + (p.has_token ? 1 : 0);
    const int stg_bufs = n_tot > kTokBlock ? 2 : 1;
    const WsSmem fixed = make_ws_smem(NH, NP, c.dv, c.buf_len, 0, stg_bufs);
    if (fixed.total + 2u * fixed.sst_bytes > budget) return SKETCHSSM_UNSUPPORTED_SHAPE;
    int stages = (int)((budget - fixed.total) / fixed.sst_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (p.stages >= 2 && p.stages < stages) stages = p.stages;
    p.stages = stages;
    const WsSmem sm = make_ws_smem(NH, NP, c.dv, c.buf_len, stages, stg_bufs);
    const long long n_tiles = (long long)c.batch * c.heads / NH;
    long long grid = (long long)ctx->sm_count * ctas;
    if (grid > n_tiles) grid = n_tiles;
    auto kern = NP > 32 ? (c.dv == 128 ? update_tc_ws_mamba2_kernel<128, true> : update_tc_ws_mamba2_kernel<64, true>)
                        : (c.dv == 128 ? update_tc_ws_mamba2_kernel<128, false> : update_tc_ws_mamba2_kernel<64, false>);
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)sm.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    if ((ctx->last_cuda_error = launch_kernel(kern, dim3((unsigned)grid), dim3(kWsThreads), sm.total, stream, p, p.pdl != 0)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

}  // namespace sketchssm
