// Decode-step kernel, one warp per (batch, head) (sm_100a): the default for decode_step and full_read_decode.
//
// CTAs are persistent: each walks a contiguous range of (head index, batch) items, so a single wave of CTAs
// covers the launch, the coefficient map C of at most two head indices is staged in shared memory once per CTA,
// and no per-CTA start-up cost is paid more than once per SM slot.  A warp owns one head at a time.  All of the
// head's operands -- the sketch U, the buffered keys / values / gates of the ring and the current token's
// q, k, v rows -- arrive in the warp's private shared-memory stage by 1-D bulk asynchronous copies (TMA, no
// multicast).  The stage is filled in two groups with an mbarrier each: what the ring sweep reads, and the sketch.
// The next head's first group is issued right after the current head's sweep and its sketch right after the current
// sketch has been used, each copy by its own lane, and the token's scalar gates are fetched one head ahead: the
// loads of a head overlap the arithmetic of the one before it without a second stage.
//
// Arithmetic per head (Algorithm 1, non-flush step; Eq. 4):
//   x <- q_t;  for s = t .. 1:  a_s = beta_s <k_s, x>;  x <- D_s (x - a_s k_s)   [Mamba-2: a_s = beta_s (prod_{j>s} a_j) <k_s, q_t>]
//   sketch mode:    o = sum_g (C x)_g U[g,:] + sum_s a_s v_s
//   full-read mode: o = S_0^T x            + sum_s a_s v_s
// Sets of independent dot products (C x, and all of Mamba-2's <k_s, q_t>) are reduced eight at a time with a
// transposing butterfly (9 shuffles per 8 sums instead of 40); the delta-rule chain keeps one 5-step reduction
// per buffered token.
#include "internal.cuh"
#include "lanegroup.cuh"

namespace sketchssm {

namespace {


#define DEC_WAIT(bar, parity) mbar_wait_bounded(bar, parity)
// parity of the sketch barrier's phase for the current head: with one rank for all heads both barriers advance together
// (the ring barrier's parity has already been flipped when the sketch is waited for)
#define PARB (GEN ? parB : (parA ^ 1u))

struct StageLayout {
    uint32_t u_off, u_bytes;        // sketch U (sketch mode only)
    uint32_t c_off, c_bytes;        // the head's own coefficient map (sketch mode with a per-sequence map only)
    uint32_t f_off, f_bytes;        // projected erase vectors of the n buffered tokens (n rows of R floats; erase mode only)
    uint32_t k_off, k_bytes;        // n buffered keys
    uint32_t v_off, v_bytes;        // n buffered values
    uint32_t gate_off, gate_bytes;  // beta[L] (+ decay[L] for scalar kinds)
    uint32_t g_off, g_bytes;        // KDA: n per-channel decays
    uint32_t tq_off, tk_off, tv_off, tg_off, tqk_bytes, tv_bytes, tg_bytes;   // the current token's rows
    uint32_t total;                 // stage stride, multiple of 128
};

__host__ __device__ inline StageLayout make_stage_layout(int kind, int io, int K, int V, int R, int L, int n,
                                                         int full_read, int coef_per_seq, int sketch_bytes = 4,
                                                         int erase = 0) {
    StageLayout s;
    uint32_t off = 0;
    s.u_off = off; s.u_bytes = full_read ? 0u : (uint32_t)(R * V * sketch_bytes); off += (s.u_bytes + 15u) & ~15u;
    // rows padded to the reduction width are read (their sums are never used), so they get room but are not copied
    s.c_off = off; s.c_bytes = (!full_read && coef_per_seq) ? (uint32_t)(R * K * sketch_bytes) : 0u;
    off += (!full_read && coef_per_seq) ? (uint32_t)(((R + 7) & ~7) * K * sketch_bytes) : 0u;
    s.f_off = off; s.f_bytes = (!full_read && erase) ? (uint32_t)(n * R * sketch_bytes) : 0u; off += (s.f_bytes + 15u) & ~15u;
    s.k_off = off; s.k_bytes = (uint32_t)(n * K * io); off += s.k_bytes;
    s.v_off = off; s.v_bytes = (uint32_t)(n * V * io); off += s.v_bytes;
    s.gate_off = off;
    s.gate_bytes = n > 0 ? (uint32_t)((kind == SKETCHSSM_KDA ? 1 : 2) * L * 4) : 0u;
    off += s.gate_bytes;
    s.g_off = off; s.g_bytes = kind == SKETCHSSM_KDA ? (uint32_t)(n * K * io) : 0u; off += s.g_bytes;
    s.tqk_bytes = (uint32_t)(K * io); s.tv_bytes = (uint32_t)(V * io);
    s.tg_bytes = kind == SKETCHSSM_KDA ? (uint32_t)(K * io) : 0u;
    s.tq_off = off; off += s.tqk_bytes;
    s.tk_off = off; off += s.tqk_bytes;
    s.tv_off = off; off += s.tv_bytes;
    s.tg_off = off; off += s.tg_bytes;
    s.total = (off + 127u) & ~127u;
    return s;
}

struct DecodeSmem {
    uint32_t coef_slot_bytes, bar_off, scratch_off, scratch_stride, stage_off, total;
};

__host__ __device__ inline DecodeSmem make_decode_smem(int K, int R, int nwarps, int full_read, int coef_per_seq,
                                                       uint32_t stage_bytes) {
    DecodeSmem d;
    const int RP = (R + 7) & ~7;                       // coefficient rows padded to the reduction width
    d.coef_slot_bytes = (full_read || coef_per_seq) ? 0u : (uint32_t)(RP * K * 4);
    d.bar_off = 2u * d.coef_slot_bytes;
    uint32_t off = d.bar_off + (((uint32_t)(nwarps * 2 * 8 + 16) + 127u) & ~127u);    // two mbarriers per warp, the head counter
    d.scratch_stride = (uint32_t)((K + 80) * 4);       // per warp: q~ (full read) or c (K floats), then 64+ dot products
    d.scratch_off = off; off += (uint32_t)nwarps * d.scratch_stride;
    d.stage_off = off;
    d.total = off + (uint32_t)nwarps * stage_bytes;
    return d;
}

}  // namespace

// RT: the sketch rank as a compile-time constant (loops over ranks unroll fully), or 0 for any rank.
// GEN: 0 = one ring fill and one rank for every head of the launch (copy sizes are per-lane constants);
//      1 = per-sequence phases and / or a per-head rank table (sizes follow the head);
//      2 = 1 with the coefficient vector formed from projected erase vectors (delta-rule kinds).
// UB: the sketch rows and the fixed coefficient map are stored as bfloat16 (a compile-time fact for the lean
//     instantiation; the general ones read the flag of the launch).
template <int KIND, typename IO, int K, int V, int RT, int GEN, bool UB = false>
__global__ void __launch_bounds__(256, (GEN >= 1 || KIND != SKETCHSSM_MAMBA2) ? 3 : 4) decode_kernel(const Params p) {
    constexpr int EK = K / 32;
    constexpr int EV = V % 32 == 0 ? V / 32 : 4;        // value elements per lane ...
    constexpr int VL = V / EV;                          // ... on the first VL lanes (all 32, or 20 for V = 80)
    constexpr int NB = 8;                               // dot products per transposing reduction
    extern __shared__ __align__(128) unsigned char smem[];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int R = RT ? RT : p.R;
    const int L = p.L, H = p.H, B = p.B;
    const int n_cap = p.n_before;                       // ring rows the stage has room for (per-sequence phases: the largest fill)
    const bool vlane = VL == 32 || lane < VL;           // this lane holds value elements
    const bool per_seq = GEN && p.coef_per_seq;         // the head's own coefficient map travels with its sketch rows
    const bool u_bf16 = UB || (GEN && p.sketch_bf16);   // sketch rows (and the fixed coefficient map) stored as bfloat16
    const int su = u_bf16 ? 2 : 4;
    const int RP = (R + 7) & ~7;
    // c_t from the projected erase vectors of the buffered tokens instead of the swept query (delta-rule kinds)
    constexpr bool ER = GEN == 2;
    const bool er = ER && !p.full_read;

    const StageLayout sl = make_stage_layout(KIND, (int)sizeof(IO), K, V, R, L, n_cap, p.full_read, per_seq, su, er);
    const DecodeSmem ds = make_decode_smem(K, R, nwarps, p.full_read, per_seq, sl.total);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ds.bar_off) + warp * 2;
    float* sX = reinterpret_cast<float*>(smem + ds.scratch_off + (size_t)warp * ds.scratch_stride);   // c or q~
    float* sP = sX + K;                                                                               // dot products
    unsigned char* my_stage = smem + ds.stage_off + (size_t)warp * sl.total;

    // contiguous range of items for this CTA; item = h * B + b
    const long long total = (long long)H * B;
    const int item0 = (int)(total * blockIdx.x / gridDim.x);
    const int item1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int h_first = item0 / B;
    const int h_last = item1 > item0 ? (item1 - 1) / B : h_first;

    if (threadIdx.x == 0) {
        for (int i = 0; i < nwarps * 2; ++i) mbar_init(reinterpret_cast<uint64_t*>(smem + ds.bar_off) + i, 1);
        *reinterpret_cast<int*>(smem + ds.bar_off + (size_t)nwarps * 16) = nwarps;
        mbar_fence_init();
    }
    // coefficient maps of the (at most two) head indices of this range, rows padded with zeros.  C is a constant of
    // the layer (never written by these kernels), so it may be staged before the predecessor in the stream is done.
    if (!p.full_read && !per_seq && item1 > item0) {
        const int nslots = h_last > h_first ? 2 : 1;
        for (int s = 0; s < nslots; ++s) {
            float4* dst = reinterpret_cast<float4*>(smem + (size_t)s * ds.coef_slot_bytes);
            if (u_bf16) {        // the map is stored as bfloat16: widened while it is staged
                const uint2* src = reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(p.coef) + (size_t)(h_first + s) * R * K);
                for (int i = threadIdx.x; i < RP * K / 4; i += blockDim.x) {
                    float4 c4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (i < R * K / 4) {
                        const uint2 t = src[i];
                        c4 = make_float4(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u),
                                         __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u));
                    }
                    dst[i] = c4;
                }
            } else {
                const float4* src = reinterpret_cast<const float4*>(p.coef + (size_t)(h_first + s) * R * K);
                for (int i = threadIdx.x; i < RP * K / 4; i += blockDim.x)
                    dst[i] = i < R * K / 4 ? src[i] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    }
    __syncthreads();

    // A warp's stage is filled by two groups of bulk copies, each completing on its own mbarrier: group A holds what
    // the ring sweep reads (the token's rows and the buffered keys / values / gates), group B the sketch U (and, with a
    // per-sequence coefficient map, the head's own C).  Group A of the warp's next head is issued as soon as the sweep of
    // the current head is over and group B as soon as U has been used, so the next head's loads overlap the rest of the
    // current head's arithmetic without a second stage.  Every copy is issued by its own lane from per-lane constants set
    // up once (base pointer, bytes per head, target); its size is fixed, or a multiple of the head's ring fill (the fill
    // is per sequence when the caller passes per-sequence phases) or of the head's sketch rank (per-head rank table).
    const unsigned char* cp_base = nullptr;
    size_t cp_stride = 0;
    uint32_t cp_dst = 0, cp_unit = 0;
    int cp_mode = 0;            // bytes of the copy: 0 cp_unit; 1 cp_unit * ring fill; 2 cp_unit if the ring is not empty; 3 cp_unit * rank
    switch (lane) {
        case 0: cp_base = reinterpret_cast<const unsigned char*>(p.q); cp_stride = (size_t)K * sizeof(IO); cp_dst = sl.tq_off; cp_unit = sl.tqk_bytes; break;
        case 1: cp_base = reinterpret_cast<const unsigned char*>(p.k); cp_stride = (size_t)K * sizeof(IO); cp_dst = sl.tk_off; cp_unit = sl.tqk_bytes; break;
        case 2: cp_base = reinterpret_cast<const unsigned char*>(p.v); cp_stride = (size_t)V * sizeof(IO); cp_dst = sl.tv_off; cp_unit = sl.tv_bytes; break;
        case 3: cp_base = reinterpret_cast<const unsigned char*>(p.decay); cp_stride = (size_t)K * sizeof(IO); cp_dst = sl.tg_off; cp_unit = sl.tg_bytes; break;
        case 4: cp_base = p.ring; cp_stride = p.rl.head_bytes; cp_dst = sl.k_off; cp_unit = (uint32_t)(K * sizeof(IO)); cp_mode = 1; break;
        case 5: cp_base = p.ring + p.rl.beta_off; cp_stride = p.rl.head_bytes; cp_dst = sl.gate_off; cp_unit = (uint32_t)((KIND == SKETCHSSM_KDA ? 1 : 2) * L * 4); cp_mode = 2; break;
        case 6: cp_base = p.ring + p.rl.v_off; cp_stride = p.rl.head_bytes; cp_dst = sl.v_off; cp_unit = (uint32_t)(V * sizeof(IO)); cp_mode = 1; break;
        case 7: cp_base = p.ring + p.rl.decay_off; cp_stride = p.rl.head_bytes; cp_dst = sl.g_off; cp_unit = KIND == SKETCHSSM_KDA ? (uint32_t)(K * sizeof(IO)) : 0u; cp_mode = 1; break;
        case 8: cp_base = reinterpret_cast<const unsigned char*>(p.sketch); cp_stride = (size_t)R * V * su; cp_dst = sl.u_off; cp_unit = (uint32_t)(V * su); cp_mode = 3; break;
        case 9: cp_base = reinterpret_cast<const unsigned char*>(p.coef); cp_stride = (size_t)R * K * su; cp_dst = sl.c_off; cp_unit = per_seq ? (uint32_t)(K * su) : 0u; cp_mode = 3; break;
        case 10: cp_base = reinterpret_cast<const unsigned char*>(p.erase); cp_stride = (size_t)L * R * su; cp_dst = sl.f_off; cp_unit = er ? (uint32_t)(R * su) : 0u; cp_mode = 1; break;
        default: break;
    }
    const uint32_t tokA = 2u * sl.tqk_bytes + sl.tv_bytes + sl.tg_bytes;
    const uint32_t rowA = (uint32_t)((K + V) * sizeof(IO)) + (KIND == SKETCHSSM_KDA ? (uint32_t)(K * sizeof(IO)) : 0u);
    const uint32_t gateA = (uint32_t)((KIND == SKETCHSSM_KDA ? 1 : 2) * L * 4);
    const uint32_t rowB = (uint32_t)(V * su) + (per_seq ? (uint32_t)(K * su) : 0u);
    const int r_uni = p.full_read ? 0 : R;          // GEN = 0: the rank of every head
    // GEN = 0: the size of this lane's copy and the two transaction totals are constants of the launch
    const uint32_t cp_fixed = cp_mode == 0 ? cp_unit : cp_mode == 1 ? cp_unit * (uint32_t)n_cap
                            : cp_mode == 2 ? (n_cap > 0 ? cp_unit : 0u) : cp_unit * (uint32_t)r_uni;
    const uint32_t txA_fixed = tokA + (uint32_t)n_cap * rowA + (n_cap > 0 ? gateA : 0u);
    const uint32_t txB_fixed = (uint32_t)r_uni * rowB;
    uint64_t* barA = &bars[0];
    uint64_t* barB = &bars[1];
    auto issue_a = [&](size_t bh, int n_it) {      // whole warp; n_it: ring fill of the head
        if constexpr (GEN) {
            if (lane == 0) mbar_expect_tx(barA, tokA + (uint32_t)n_it * rowA + (n_it > 0 ? gateA : 0u));
            __syncwarp();
            const uint32_t bytes = cp_mode == 0 ? cp_unit : cp_mode == 1 ? cp_unit * (uint32_t)n_it : (n_it > 0 ? cp_unit : 0u);
            if (lane < 8 && bytes) bulk_g2s(my_stage + cp_dst, cp_base + bh * cp_stride, bytes, barA);
        } else {
            if (lane == 0) mbar_expect_tx(barA, txA_fixed);
            __syncwarp();
            if (lane < 8 && cp_fixed) bulk_g2s(my_stage + cp_dst, cp_base + bh * cp_stride, cp_fixed, barA);
        }
    };
    // whole warp; r_it: sketch rank of the head (0: nothing to fetch), n_it: its ring fill (rows of erase vectors)
    auto issue_b = [&](size_t bh, int r_it, int n_it) {
        if constexpr (GEN) {
            const uint32_t fbytes = er ? (uint32_t)n_it * (uint32_t)(R * su) : 0u;
            if (lane == 8 && r_it > 0) mbar_expect_tx(barB, (uint32_t)r_it * rowB + fbytes);
            __syncwarp();
            if ((lane == 8 || lane == 9) && cp_unit && r_it > 0)
                bulk_g2s(my_stage + cp_dst, cp_base + bh * cp_stride, cp_unit * (uint32_t)r_it, barB);
            if (lane == 10 && fbytes && r_it > 0) bulk_g2s(my_stage + cp_dst, cp_base + bh * cp_stride, fbytes, barB);
        } else {
            if (lane == 8 && txB_fixed) mbar_expect_tx(barB, txB_fixed);
            __syncwarp();
            if ((lane == 8 || lane == 9) && cp_fixed) bulk_g2s(my_stage + cp_dst, cp_base + bh * cp_stride, cp_fixed, barB);
        }
    };

    // The CTA's heads are handed to its warps at run time (a counter in shared memory): a warp claims its next head
    // when it starts the current one, so the warps of a CTA finish within one head of each other whatever the count.
    // The range spans at most two head indices, so (head index, batch) follow from the item number without divisions.
    const int n_items = item1 - item0;
    int* item_ctr = reinterpret_cast<int*>(smem + ds.bar_off + (size_t)nwarps * 16);
    const int second_h_start = (h_first + 1) * B;      // first item of the range's second head index
    auto claim = [&]() -> int {            // whole warp; returns an item number, or item1 when none is left
        int v = 0;
        if (lane == 0) v = atomicAdd(item_ctr, 1);
        v = __shfl_sync(0xffffffffu, v, 0);
        return v < n_items ? item0 + v : item1;
    };
    auto head_of = [&](int item, int& hh, int& bb) {
        hh = item >= second_h_start ? h_first + 1 : h_first;
        bb = item - hh * B;
    };
    // Per-head sketch rank: the configured rank, or the caller's table (0 = this head reads the full state instead).
    // The table is a layer constant like C, so it may be read before the predecessor in the stream is done.
    auto rank_of = [&](int hh) -> int {
        if constexpr (!GEN) return r_uni;
        if (p.full_read) return 0;
        if (p.head_rank == nullptr) return R;
        const int r = p.head_rank[hh];
        return r < 0 ? 0 : (r > R ? R : r);
    };
    // Per-sequence ring fill: the call's n_before, or the caller's per-sequence phase (negative: the sequence takes the
    // flush step in this call and is skipped here).
    auto fill_of = [&](int bb) -> int {
        if constexpr (!GEN) return n_cap;
        return p.n_dev == nullptr ? n_cap : p.n_dev[bb];
    };

    int item = warp < n_items ? item0 + warp : item1;      // the first head of every warp is fixed (the counter starts at nwarps)
    int h = 0, b = 0, hn = 0, bn = 0;
    if (item < item1) head_of(item, h, b);
    int rk = item < item1 ? rank_of(h) : 0, rk_next = 0;
    int n = 0, n_next = 0;

    // the token's scalar gates travel in registers, fetched one head ahead
    auto scalar_gates = [&](size_t bh, float& bt, float& dsc) {
        bt = p.beta[bh];
        dsc = 1.f;
        if constexpr (KIND != SKETCHSSM_KDA) dsc = reinterpret_cast<const float*>(p.decay)[bh];
    };
    float bt_next = 0.f, dsc_next = 1.f;
    // Only a state update writes the sketch; unless one may still be running (the caller of the launcher knows), the first
    // head's sketch rows are requested before the predecessor in the stream is waited for, so they travel during its tail.
    // (Not with per-sequence phases: whether the head takes part at all is only known after the wait.)
    const bool early_u = p.early_sketch != 0 && p.n_dev == nullptr;
    if (item < item1 && early_u) issue_b((size_t)b * H + h, rk, 0);
    grid_dep_wait();                 // from here on the ring and the token tensors (and otherwise the sketch) are read
    // Dependents are released only now: a successor that reads its sketch early must not start before this kernel has
    // seen its own predecessor (possibly a state update) complete.
    grid_dep_launch_dependents();
    if (item < item1) {
        const size_t bh0 = (size_t)b * H + h;
        n = fill_of(b);
        if (!GEN || n >= 0) {
            issue_a(bh0, n);
            if (!early_u) issue_b(bh0, rk, n);
            scalar_gates(bh0, bt_next, dsc_next);
        }
    }
    // A wait that runs out ends the warp's loop; the decision is taken by vote so that all lanes leave together.
    // pendA / pendB: parity of a phase whose copies may still be in flight when the loop is left that way (-1: none).
    int pendA = -1, pendB = -1;
    uint32_t parA = 0, parB = 0;     // phase parities of the two barriers (a phase passes only for heads that issued copies)

    while (item < item1) {
        if constexpr (!GEN) { n = n_cap; n_next = n_cap; rk = r_uni; rk_next = r_uni; }      // launch constants
        const size_t bh = (size_t)b * H + h;
        const int item_next = claim();
        const bool has_next = item_next < item1;
        if (has_next) {
            head_of(item_next, hn, bn);
            rk_next = rank_of(hn);
            n_next = fill_of(bn);
        }
        const bool go_next = has_next && (!GEN || n_next >= 0);          // the next head takes a decode step in this call
        const size_t bh_next = (size_t)bn * H + hn;
        const float bt = bt_next, dsc = dsc_next;
        if (go_next) scalar_gates(bh_next, bt_next, dsc_next);

        if constexpr (GEN) {
            if (n < 0) {             // this sequence takes the flush step in this call: nothing to do here
                if (go_next) { issue_a(bh_next, n_next); issue_b(bh_next, rk_next, n_next); }
                item = item_next; h = hn; b = bn; n = n_next; rk = rk_next;
                continue;
            }
        }
        const bool full = rk == 0;   // exact read of the whole state for this head
        const bool er_h = er && !full;       // this head forms c_t from projected erase vectors

        if (__any_sync(0xffffffffu, !DEC_WAIT(barA, parA))) {
            if (lane == 0) record_fault(p.status, p.full_read ? kFaultFullReadWait : kFaultDecodeWait, (int)blockIdx.x);
            pendA = (int)parA;
            pendB = full ? -1 : (int)(GEN ? parB : parA);
            break;
        }
        parA ^= 1u;
        const unsigned char* sb = my_stage;
        const IO* sK = reinterpret_cast<const IO*>(sb + sl.k_off);
        const IO* sV = reinterpret_cast<const IO*>(sb + sl.v_off);
        const float* sBeta = reinterpret_cast<const float*>(sb + sl.gate_off);
        const float* sDec = sBeta + L;
        const IO* sG = reinterpret_cast<const IO*>(sb + sl.g_off);

        float q0[EK], x[EK], kk[EK], gg[EK], vv[EV], o[EV];
        load_io<EK>(reinterpret_cast<const IO*>(sb + sl.tq_off), lane * EK, q0);
        load_io<EK>(reinterpret_cast<const IO*>(sb + sl.tk_off), lane * EK, kk);
#pragma unroll
        for (int e = 0; e < EV; ++e) vv[e] = 0.f;
        if (vlane) load_io<EV>(reinterpret_cast<const IO*>(sb + sl.tv_off), lane * EV, vv);
        if constexpr (KIND == SKETCHSSM_KDA) load_io<EK>(reinterpret_cast<const IO*>(sb + sl.tg_off), lane * EK, gg);

        if (p.append) {
            unsigned char* rh = p.ring + bh * p.rl.head_bytes;
            store_io<EK>(reinterpret_cast<IO*>(rh) + (size_t)n * K, lane * EK, kk);
            if (vlane) store_io<EV>(reinterpret_cast<IO*>(rh + p.rl.v_off) + (size_t)n * V, lane * EV, vv);
            if constexpr (KIND == SKETCHSSM_KDA) {
                store_io<EK>(reinterpret_cast<IO*>(rh + p.rl.decay_off) + (size_t)n * K, lane * EK, gg);
                if (lane == 0) reinterpret_cast<float*>(rh + p.rl.beta_off)[n] = bt;
            } else if (lane == 0) {
                reinterpret_cast<float*>(rh + p.rl.beta_off)[n] = bt;
                reinterpret_cast<float*>(rh + p.rl.decay_off)[n] = dsc;
            }
        }

        // ---- current token, s = t ----
        float dsuf = 1.f;
        float kq_t;                  // <k_t, q_t>
        {
            float part = 0.f;
#pragma unroll
            for (int e = 0; e < EK; ++e) part = fmaf(kk[e], q0[e], part);
            kq_t = warp_sum(part);
            const float a = bt * kq_t;
#pragma unroll
            for (int e = 0; e < EV; ++e) o[e] = a * vv[e];
            if constexpr (KIND == SKETCHSSM_MAMBA2) {
                dsuf = dsc;
            } else if constexpr (KIND == SKETCHSSM_GDN) {
#pragma unroll
                for (int e = 0; e < EK; ++e) x[e] = dsc * fmaf(-a, kk[e], q0[e]);
            } else {
#pragma unroll
                for (int e = 0; e < EK; ++e) x[e] = gg[e] * fmaf(-a, kk[e], q0[e]);
            }
        }

        // ---- buffered tokens ----
        if constexpr (KIND == SKETCHSSM_MAMBA2) {
            // independent dot products <k_s, q_t>, eight per transposing reduction; lane l ends up with slot s0 + l/4
            int s0 = 0;
            for (; s0 + 4 < n; s0 += NB) {      // blocks of eight while more than four slots remain
                float part[NB];
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    float kr[EK];
                    load_io<EK>(sK, min(s0 + i, n - 1) * K + lane * EK, kr);
                    float acc = 0.f;
#pragma unroll
                    for (int e = 0; e < EK; ++e) acc = fmaf(kr[e], q0[e], acc);
                    part[i] = acc;
                }
                group_reduce_transpose<32, NB>(part, lane);
                if ((lane & 3) == 0) sP[s0 + (lane >> 2)] = part[0];
            }
            if (s0 < n) {                       // one to four slots left: lane l ends up with slot s0 + l/8
                float part[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float kr[EK];
                    load_io<EK>(sK, min(s0 + i, n - 1) * K + lane * EK, kr);
                    float acc = 0.f;
#pragma unroll
                    for (int e = 0; e < EK; ++e) acc = fmaf(kr[e], q0[e], acc);
                    part[i] = acc;
                }
                group_reduce_transpose<32, 4>(part, lane);
                if ((lane & 7) == 0) sP[s0 + (lane >> 3)] = part[0];
            }
            __syncwarp();
#pragma unroll 4
            for (int s = n - 1; s >= 0; --s) {
                const float a = sBeta[s] * dsuf * sP[s];
                dsuf *= sDec[s];
                if (vlane) {
                    float vr[EV];
                    load_io<EV>(sV, s * V + lane * EV, vr);
#pragma unroll
                    for (int e = 0; e < EV; ++e) o[e] = fmaf(a, vr[e], o[e]);
                }
            }
#pragma unroll
            for (int e = 0; e < EK; ++e) x[e] = dsuf * q0[e];
        } else {
            // Erase mode: before the sweep (which the exact output of the buffered tokens needs anyway), the left factors
            // l_s(t) = (D_t ... D_{s+1}) k_s give <l_s(t), q_t> and <l_s(t), k_t> for every slot (Eq. 46: from the stored keys
            // and the running product of the decays), eight slots per transposing reduction, from the newest slot down.
            // KDA: dlv ends up as the cumulative decay d_[t].  GDN: the dot products are those of the raw keys, scaled by
            // the running scalar product inside the sweep below, where dl ends up as d_[t].
            float dl = dsc;
            float dlv[EK];
#pragma unroll
            for (int e = 0; e < EK; ++e) dlv[e] = KIND == SKETCHSSM_KDA ? gg[e] : 1.f;
            float dl_lane = 1.f;          // GDN, erase mode: lane l holds the product of the decays after slot l (the token's included)
            if constexpr (ER) {
                if (er_h) {
                    if constexpr (KIND == SKETCHSSM_GDN) {
                        float incl = lane < n ? sDec[lane] : 1.f;       // inclusive suffix product over the slots
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const float other = __shfl_down_sync(0xffffffffu, incl, o);
                            if (lane + o < 32) incl *= other;
                        }
                        float excl = __shfl_down_sync(0xffffffffu, incl, 1);
                        if (lane == 31) excl = 1.f;
                        dl_lane = dsc * excl;
                        dl = dsc * __shfl_sync(0xffffffffu, incl, 0);     // the cumulative decay d_[t]
                    }
                    for (int sb = n - 1; sb >= 0; sb -= NB) {
                        float pq[NB], pk[NB];
#pragma unroll
                        for (int i = 0; i < NB; ++i) {
                            const int s = sb - i;
                            const int sc = s < 0 ? 0 : s;              // (rows below slot 0: computed, never stored)
                            float kr[EK];
                            load_io<EK>(sK, sc * K + lane * EK, kr);
                            float aq = 0.f, ak = 0.f;
#pragma unroll
                            for (int e = 0; e < EK; ++e) {
                                const float le = KIND == SKETCHSSM_KDA ? dlv[e] * kr[e] : kr[e];
                                aq = fmaf(le, q0[e], aq);
                                ak = fmaf(le, kk[e], ak);
                            }
                            pq[i] = aq;
                            pk[i] = ak;
                            if constexpr (KIND == SKETCHSSM_KDA) {
                                if (s >= 0) {
                                    float gr[EK];
                                    load_io<EK>(sG, s * K + lane * EK, gr);
#pragma unroll
                                    for (int e = 0; e < EK; ++e) dlv[e] *= gr[e];
                                }
                            }
                        }
                        group_reduce_transpose<32, NB>(pq, lane);       // lane l holds entry l / 4: slot sb - l / 4
                        group_reduce_transpose<32, NB>(pk, lane);
                        const int s = sb - (lane >> 2);
                        float sc = 1.f;
                        if constexpr (KIND == SKETCHSSM_GDN) sc = __shfl_sync(0xffffffffu, dl_lane, s < 0 ? 0 : s);
                        if ((lane & 3) == 0 && s >= 0) { sP[s] = pq[0] * sc; sP[32 + s] = pk[0] * sc; }
                    }
                    __syncwarp();
                }
            }
#pragma unroll 2
            for (int s = n - 1; s >= 0; --s) {
                float kr[EK], vr[EV];
                load_io<EK>(sK, s * K + lane * EK, kr);
#pragma unroll
                for (int e = 0; e < EV; ++e) vr[e] = 0.f;
                if (vlane) load_io<EV>(sV, s * V + lane * EV, vr);
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < EK; ++e) part = fmaf(kr[e], x[e], part);
                const float a = sBeta[s] * warp_sum(part);
                if constexpr (KIND == SKETCHSSM_GDN) {
                    const float d = sDec[s];
#pragma unroll
                    for (int e = 0; e < EK; ++e) x[e] = d * fmaf(-a, kr[e], x[e]);
                } else {
                    float gr[EK];
                    load_io<EK>(sG, s * K + lane * EK, gr);
#pragma unroll
                    for (int e = 0; e < EK; ++e) x[e] = gr[e] * fmaf(-a, kr[e], x[e]);
                }
#pragma unroll
                for (int e = 0; e < EV; ++e) o[e] = fmaf(a, vr[e], o[e]);
            }
            if constexpr (ER) {
                if (er_h) {      // x <- d_[t] * q_t; kk <- d_[t] * k_t (the token's key has been stored and swept by now)
#pragma unroll
                    for (int e = 0; e < EK; ++e) {
                        const float d = KIND == SKETCHSSM_KDA ? dlv[e] : dl;
                        x[e] = d * q0[e];
                        kk[e] *= d;
                    }
                }
            }
        }

        // the sweep is done with the ring part of the stage: the next head's group A may come in
        __syncwarp();
        if (go_next) issue_a(bh_next, n_next);
        if (!full) {
            // c = C x, eight coefficients per transposing reduction, handed to all lanes through the scratch
            const float* sC = per_seq ? reinterpret_cast<const float*>(sb + sl.c_off)
                                             : reinterpret_cast<const float*>(smem + (size_t)(h - h_first) * ds.coef_slot_bytes);
            __syncwarp();
            if (per_seq) {        // the head's own map arrives with its sketch rows
                if (__any_sync(0xffffffffu, !DEC_WAIT(barB, PARB))) {
                    if (lane == 0) record_fault(p.status, kFaultDecodeWait, (int)blockIdx.x);
                    pendB = (int)PARB;
                    pendA = go_next ? (int)parA : -1;
                    break;
                }
            }
            const bool c16 = GEN && per_seq && u_bf16;       // the head's own map travels as bfloat16 (the shared map was widened when staged)
            const int rp_it = RT ? ((RT + 7) & ~7) : ((rk + 7) & ~7);
            bool both = false;       // erase mode: C (d_[t] * q_t) and C (d_[t] * k_t) in one pass over the rows of C
            if constexpr (ER) both = er_h;
            if (!both) {
#pragma unroll
            for (int g0 = 0; g0 < (RT ? ((RT + 7) & ~7) : rp_it); g0 += NB) {
                float part[NB];
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    float cw[EK];
                    if (c16) load_io<EK>(reinterpret_cast<const __nv_bfloat16*>(sC), (g0 + i) * K + lane * EK, cw);
                    else load_io<EK>(sC, (g0 + i) * K + lane * EK, cw);
                    float acc = 0.f;
#pragma unroll
                    for (int e = 0; e < EK; ++e) acc = fmaf(cw[e], x[e], acc);
                    part[i] = acc;
                }
                group_reduce_transpose<32, NB>(part, lane);
                if ((lane & 3) == 0) sX[g0 + (lane >> 2)] = part[0];
            }
            } else {
                if constexpr (ER) {
                    for (int g0 = 0; g0 < rp_it; g0 += NB) {
                        float part[2 * NB];
#pragma unroll
                        for (int i = 0; i < NB; ++i) {
                            float cw[EK];
                            if (c16) load_io<EK>(reinterpret_cast<const __nv_bfloat16*>(sC), (g0 + i) * K + lane * EK, cw);
                            else load_io<EK>(sC, (g0 + i) * K + lane * EK, cw);
                            float aq = 0.f, ak = 0.f;
#pragma unroll
                            for (int e = 0; e < EK; ++e) { aq = fmaf(cw[e], x[e], aq); ak = fmaf(cw[e], kk[e], ak); }
                            part[i] = aq;
                            part[NB + i] = ak;
                        }
                        group_reduce_transpose<32, 2 * NB>(part, lane);      // lane l holds entry l / 2
                        const int en = lane >> 1;
                        if ((lane & 1) == 0) sX[(en < NB ? g0 + en : rp_it + g0 + en - NB)] = part[0];
                    }
                }
            }
            __syncwarp();
            if (!per_seq) {
                if (__any_sync(0xffffffffu, !DEC_WAIT(barB, PARB))) {
                    if (lane == 0) record_fault(p.status, kFaultDecodeWait, (int)blockIdx.x);
                    pendB = (int)PARB;
                    pendA = go_next ? (int)parA : -1;
                    break;
                }
            }
            if constexpr (GEN) parB ^= 1u;
            if constexpr (ER) {
                if (er_h) {
                    // f_t = beta_t [C (d_[t] * k_t) - sum_{s<t} f_s <l_s(t), k_t>]  (Eq. 45), stored for the later steps;
                    // c_t = C (d_[t] * q_t) - sum_{s<t} f_s <l_s(t), q_t> - f_t <k_t, q_t>  (Eq. 44).  One coefficient per lane.
                    // (with bfloat16 storage the vectors are rounded once, where they are stored; this step uses the rounded f_t too)
                    const float* sF = reinterpret_cast<const float*>(sb + sl.f_off);
                    const __nv_bfloat16* sF16 = reinterpret_cast<const __nv_bfloat16*>(sb + sl.f_off);
                    for (int g = lane; g < rk; g += 32) {
                        float fq = sX[g], fk = sX[rp_it + g];
                        for (int s = 0; s < n; ++s) {
                            const float f = u_bf16 ? __bfloat162float(sF16[s * R + g]) : sF[s * R + g];
                            fq = fmaf(-f, sP[s], fq);
                            fk = fmaf(-f, sP[32 + s], fk);
                        }
                        float f_t = bt * fk;
                        if (u_bf16) f_t = __bfloat162float(__float2bfloat16_rn(f_t));
                        sX[g] = fmaf(-f_t, kq_t, fq);
                        if (p.append) {
                            const size_t idx = (bh * L + n) * (size_t)R + g;
                            if (u_bf16) reinterpret_cast<__nv_bfloat16*>(p.erase)[idx] = __float2bfloat16_rn(f_t);
                            else p.erase[idx] = f_t;
                        }
                    }
                    __syncwarp();
                }
            }
            const float* sU = reinterpret_cast<const float*>(sb + sl.u_off);
            if (vlane) {
#pragma unroll (RT ? RT : 4)
                for (int g = 0; g < (RT ? RT : rk); ++g) {
                    const float cg = sX[g];
                    float uu[EV];
                    if (u_bf16) load_io<EV>(reinterpret_cast<const __nv_bfloat16*>(sU), g * V + lane * EV, uu);
                    else load_io<EV>(sU, g * V + lane * EV, uu);
#pragma unroll
                    for (int e = 0; e < EV; ++e) o[e] = fmaf(cg, uu[e], o[e]);
                }
            }
            __syncwarp();
            if (go_next) issue_b(bh_next, rk_next, n_next);
        } else {
            __syncwarp();
            store_io<EK>(sX, lane * EK, x);
            __syncwarp();
            if (vlane) {
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
            }
            // a head that reads the full state fetched no sketch rows; the next head's are requested here
            if (go_next) issue_b(bh_next, rk_next, n_next);
        }

        if (vlane) {
            if (p.out_bf16) {
                store_io<EV>(reinterpret_cast<__nv_bfloat16*>(p.out) + bh * V, lane * EV, o);
            } else {
                store_io<EV>(reinterpret_cast<float*>(p.out) + bh * V, lane * EV, o);
            }
        }

        __syncwarp();  // every lane is done with the scratch before it is reused
        item = item_next;
        h = hn;
        b = bn;
        n = n_next;
        rk = rk_next;
    }
    // Left on a timeout: bulk copies already issued into this warp's stage get a short, bounded grace period, so that
    // they do not land in shared memory that has meanwhile been handed to another CTA.
    if (pendA >= 0) mbar_wait_bounded(barA, (uint32_t)pendA, 1u << 14);
    if (pendB >= 0) mbar_wait_bounded(barB, (uint32_t)pendB, 1u << 14);
}

template <int KIND, typename IO, int K, int V>
static int launch_decode_t(Ctx* ctx, Params p, cudaStream_t stream) {
    const int io = (int)sizeof(IO);
    const int erase = (KIND != SKETCHSSM_MAMBA2 && p.erase != nullptr && !p.full_read) ? 1 : 0;
    const StageLayout sl = make_stage_layout(KIND, io, K, V, p.R, p.L, p.n_before, p.full_read, p.coef_per_seq, p.sketch_bf16 ? 2 : 4, erase);   // (the general instantiation runs whenever coef_per_seq or sketch_bf16 is set)
    const uint32_t smem_budget = 227u * 1024u;
    if (ctx->sm_count == 0) {
        int dev = 0, sms = 0;
        if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        if ((ctx->last_cuda_error = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
        ctx->sm_count = sms;
    }
    // warps per CTA / CTAs per SM: as many resident warps per SM as shared memory allows (capped), preferring
    // fewer, larger CTAs
    const int cap = p.max_warps_per_sm > 0 ? p.max_warps_per_sm : 32;
    // bfloat16 storage with nothing else that needs the general kernel: the lean rank-16 instantiation reads it too
    const bool lean_bf16 = p.sketch_bf16 && p.R == 16 && !p.full_read && p.head_rank == nullptr && p.n_dev == nullptr &&
                           !p.coef_per_seq && !erase;
    const bool gen = p.head_rank != nullptr || p.n_dev != nullptr || p.coef_per_seq || (p.sketch_bf16 && !lean_bf16) || erase;
    const bool fixed16 = p.R == 16 && !gen;     // the unrolled rank-16 instantiation needs one rank for all heads
    auto kern = gen ? decode_kernel<KIND, IO, K, V, 0, 1> : fixed16 ? decode_kernel<KIND, IO, K, V, 16, 0> : decode_kernel<KIND, IO, K, V, 0, 0>;
    // rank 32 unrolled as well (state rows of 128 only: every instantiation costs build time; rank 8 measured no gain)
    bool fixed32 = false;
    if constexpr (K == 128) {
        if (!gen && p.R == 32) { kern = decode_kernel<KIND, IO, K, V, 32, 0>; fixed32 = true; }
    }
    if (lean_bf16) kern = decode_kernel<KIND, IO, K, V, 16, 0, true>;
    if constexpr (KIND != SKETCHSSM_MAMBA2) {
        if (erase) kern = decode_kernel<KIND, IO, K, V, 0, 2>;
    }
    // registers per thread of the two instantiations (queried once): they bound the resident warps like shared memory does
    static int regs_per_thread[6] = {0, 0, 0, 0, 0, 0};
    int& regs = regs_per_thread[fixed32 ? 5 : lean_bf16 ? 4 : erase ? 3 : gen ? 2 : fixed16 ? 1 : 0];
    if (regs == 0) {
        cudaFuncAttributes fa;
        if ((ctx->last_cuda_error = cudaFuncGetAttributes(&fa, kern)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        regs = fa.numRegs > 0 ? fa.numRegs : 64;
    }
    const int reg_warps = 65536 / (regs * 32);          // warps the register file holds
    int best_nw = 0, best_ctas = 1, best_warps = 0;
    for (int nw = 8; nw >= 1; --nw) {
        if (p.warps_per_cta && nw != p.warps_per_cta) continue;
        const DecodeSmem d = make_decode_smem(K, p.R, nw, p.full_read, p.coef_per_seq, sl.total);
        if (d.total > smem_budget) continue;
        int ctas = (int)((228u * 1024u) / (d.total + 1024u));
        if (ctas * nw > cap) ctas = cap / nw;
        if (ctas * nw > reg_warps) ctas = reg_warps / nw;
        if (ctas < 1) continue;
        if (ctas * nw > best_warps) { best_warps = ctas * nw; best_nw = nw; best_ctas = ctas; }
    }
    if (best_nw == 0) return SKETCHSSM_UNSUPPORTED_SHAPE;
    const DecodeSmem d = make_decode_smem(K, p.R, best_nw, p.full_read, p.coef_per_seq, sl.total);
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)d.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    long long grid = (long long)ctx->sm_count * best_ctas;
    const long long total = (long long)p.B * p.H;
    if (p.batches_per_cta > 0) grid = (total + p.batches_per_cta - 1) / p.batches_per_cta;   // explicit items per CTA
    if (grid > (total + best_nw - 1) / best_nw) grid = (total + best_nw - 1) / best_nw;      // at least one head per warp
    if (grid < p.H) grid = p.H;                                  // a CTA's range then spans at most two head indices
    if (grid > total) grid = total;
    if ((ctx->last_cuda_error = launch_kernel(kern, dim3((unsigned)grid), dim3(best_nw * 32), d.total, stream, p, p.pdl != 0)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

template <int KIND, typename IO>
static int launch_decode_shape(Ctx* ctx, const Params& p, cudaStream_t stream) {
    const int K = ctx->cfg.dk, V = ctx->cfg.dv;
    if (K == 128 && V == 128) return launch_decode_t<KIND, IO, 128, 128>(ctx, p, stream);
    if (K == 128 && V == 64) return launch_decode_t<KIND, IO, 128, 64>(ctx, p, stream);
    if (K == 128 && V == 80) return launch_decode_t<KIND, IO, 128, 80>(ctx, p, stream);
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
