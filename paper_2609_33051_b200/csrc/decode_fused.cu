// Decode-step kernel, fused version (sm_100a): lane groups form the weights from shared-memory stages, then the
// output rows are streamed from global memory through registers.
//
// A group of 8 lanes owns one (batch, head); a warp serves four heads at once, so every shuffle, shared-memory
// load and issue slot is shared by them.  Phase 1 forms the buffer weights a_s and the coefficient vector
// c = C q~_t (Eq. 4, Section 4.1) from the query, the buffered keys and the gates, which arrive in the group's
// private shared-memory stage by 1-D bulk asynchronous copies (TMA, no multicast) completing on an mbarrier.
// Phase 2 forms o = sum_g c_g U[g,:] + sum_s a_s v_s as a weighted sum of rows read with 128-bit loads straight
// from global memory: those rows (the sketch and the buffered values, most of the bytes of a step) are requested
// into L2 with a bulk prefetch when the stage copies are issued, one iteration earlier, so HBM latency is paid
// while the weights are formed, and the rows never occupy shared memory: only the keys do, which doubles the
// heads resident per SM.  CTAs are persistent, each walking a contiguous range of (head, batch) items so that
// the coefficient map C of at most two head indices is staged once per CTA.
//
//   x <- q_t;  for s = t .. 1:  a_s = beta_s <k_s, x>;  x <- D_s (x - a_s k_s)   [Mamba-2: a_s = beta_s (prod_{j>s} a_j) <k_s, q_t>]
//   sketch mode:    o = sum_g (C x)_g U[g,:] + sum_s a_s v_s
//   full-read mode: o = S_0^T x            + sum_s a_s v_s
#include "internal.cuh"
#include "lanegroup.cuh"

namespace sketchssm {

namespace {

struct WStage {
    uint32_t k_off, k_bytes, gate_off, gate_bytes, g_off, g_bytes;
    uint32_t tq_off, tk_off, tg_off, tqk_bytes, tg_bytes;
    uint32_t total;
};

__host__ __device__ inline WStage make_wstage(int kind, int io, int K, int L, int n) {
    WStage s;
    uint32_t off = 0;
    s.k_off = off; s.k_bytes = (uint32_t)(n * K * io); off += s.k_bytes;
    s.g_off = off; s.g_bytes = kind == SKETCHSSM_KDA ? (uint32_t)(n * K * io) : 0u; off += s.g_bytes;
    s.gate_off = off;
    s.gate_bytes = n > 0 ? (uint32_t)((kind == SKETCHSSM_KDA ? 1 : 2) * L * 4) : 0u;
    off += s.gate_bytes;
    s.tqk_bytes = (uint32_t)(K * io);
    s.tg_bytes = kind == SKETCHSSM_KDA ? (uint32_t)(K * io) : 0u;
    s.tq_off = off; off += s.tqk_bytes;
    s.tk_off = off; off += s.tqk_bytes;
    s.tg_off = off; off += s.tg_bytes;
    // stagger consecutive stages by 64 bytes so that groups reading the same row offset hit different banks
    s.total = ((off + 127u) & ~127u) + 64u;
    return s;
}

struct WSmem {
    uint32_t coef_slot_bytes, cbar_off, bar_off, scratch_off, scratch_stride, stage_off, total;
};

__host__ __device__ inline WSmem make_fsmem(int K, int RP, int groups, int stages, int full_read, uint32_t stage_bytes) {
    WSmem d;
    d.coef_slot_bytes = full_read ? 0u : (uint32_t)(RP * K * 4);
    uint32_t off = 2u * d.coef_slot_bytes;
    d.cbar_off = off; off += 128u;
    d.bar_off = off; off += (((uint32_t)(groups * stages * 8)) + 127u) & ~127u;
    d.scratch_stride = (uint32_t)((K + 80) * 4);   // c or q~ (K floats), then up to 64 buffer weights
    d.scratch_off = off; off += (uint32_t)groups * d.scratch_stride;
    d.stage_off = off;
    d.total = off + (uint32_t)(groups * stages) * stage_bytes;
    return d;
}

}  // namespace

template <int KIND, typename IO, int K, int V, int LPH, int RP>
__global__ void __launch_bounds__(256) decode_fused_kernel(const Params p) {
    constexpr int EV = V / LPH;          // value columns per lane
    constexpr int RB = EV >= 16 ? 4 : 8; // rows in flight per lane in the row phase
    constexpr int HPW = 32 / LPH;
    constexpr int EK = K / LPH;
    constexpr int CPL = RP >= LPH ? RP / LPH : 1;
    extern __shared__ __align__(128) unsigned char smem[];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int grp = lane / LPH;
    const int j = lane % LPH;
    const int R = p.R, L = p.L, H = p.H, B = p.B, n = p.n_before;
    const int stages = p.stages;
    const int groups = nwarps * HPW;
    const int gid = warp * HPW + grp;

    const WStage sl = make_wstage(KIND, (int)sizeof(IO), K, L, n);
    const WSmem ds = make_fsmem(K, RP, groups, stages, p.full_read, sl.total);
    uint64_t* cbar = reinterpret_cast<uint64_t*>(smem + ds.cbar_off);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ds.bar_off) + gid * stages;
    float* sW = reinterpret_cast<float*>(smem + ds.scratch_off + (size_t)gid * ds.scratch_stride);  // c (or q~)
    float* sA = sW + K;                                                                               // a_s
    unsigned char* my_stage = smem + ds.stage_off + (size_t)gid * stages * sl.total;

    const long long total = (long long)H * B;
    const int item0 = (int)(total * blockIdx.x / gridDim.x);
    const int item1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int h_first = item0 / B;
    const int h_last = item1 > item0 ? (item1 - 1) / B : h_first;

    if (threadIdx.x == 0) {
        mbar_init(cbar, 1);
        for (int i = 0; i < groups * stages; ++i) mbar_init(reinterpret_cast<uint64_t*>(smem + ds.bar_off) + i, 1);
        mbar_fence_init();
    }
    if (!p.full_read && R < RP) {
        for (int s = 0; s < 2; ++s) {
            float* pad = reinterpret_cast<float*>(smem + (size_t)s * ds.coef_slot_bytes) + R * K;
            for (int i = threadIdx.x; i < (RP - R) * K; i += blockDim.x) pad[i] = 0.f;
        }
    }
    __syncthreads();
    if (!p.full_read && threadIdx.x == 0 && item1 > item0) {
        const uint32_t cb = (uint32_t)(R * K * 4);
        const int nslots = h_last > h_first ? 2 : 1;
        mbar_expect_tx(cbar, cb * nslots);
        for (int s = 0; s < nslots; ++s)
            bulk_g2s(smem + (size_t)s * ds.coef_slot_bytes, p.coef + (size_t)(h_first + s) * R * K, cb, cbar);
    }

    const uint32_t tx_bytes = sl.k_bytes + sl.g_bytes + sl.gate_bytes + 2u * sl.tqk_bytes + sl.tg_bytes;

    auto issue = [&](int item, int st) {   // leader lane of an active group
        uint64_t* bar = &bars[st];
        unsigned char* sb = my_stage + (size_t)st * sl.total;
        const int h = item / B, b = item - h * B;
        const size_t bh = (size_t)b * H + h;
        const unsigned char* rh = p.ring + bh * p.rl.head_bytes;
        mbar_expect_tx(bar, tx_bytes);
        bulk_g2s(sb + sl.tq_off, reinterpret_cast<const IO*>(p.q) + bh * K, sl.tqk_bytes, bar);
        bulk_g2s(sb + sl.tk_off, reinterpret_cast<const IO*>(p.k) + bh * K, sl.tqk_bytes, bar);
        if (sl.tg_bytes) bulk_g2s(sb + sl.tg_off, reinterpret_cast<const IO*>(p.decay) + bh * K, sl.tg_bytes, bar);
        if (sl.k_bytes) {
            bulk_g2s(sb + sl.k_off, rh, sl.k_bytes, bar);
            bulk_g2s(sb + sl.gate_off, rh + p.rl.beta_off, sl.gate_bytes, bar);
            if (sl.g_bytes) bulk_g2s(sb + sl.g_off, rh + p.rl.decay_off, sl.g_bytes, bar);
        }
        if (p.l2_prefetch) {
            // the rows of the output phase are read straight from global memory once the weights are known;
            // ask L2 for them now so that HBM latency is paid while the weights are being formed
            if (p.full_read) prefetch_l2(p.state + bh * (size_t)K * V, (uint32_t)(K * V * 4));
            else prefetch_l2(p.sketch + bh * (size_t)R * V, (uint32_t)(R * V * 4));
            if (n > 0) prefetch_l2(rh + p.rl.v_off, (uint32_t)(n * V * sizeof(IO)));
            prefetch_l2(reinterpret_cast<const IO*>(p.v) + bh * V, (uint32_t)(V * sizeof(IO)));
        }
    };

    const int n_items = item1 - item0;
    const int n_quads = (n_items + HPW - 1) / HPW;
    const int my_quads = warp < n_quads ? (n_quads - warp + nwarps - 1) / nwarps : 0;
    auto item_of = [&](int it) { return item0 + (warp + it * nwarps) * HPW + grp; };

    if (my_quads > 0 && j == 0 && item_of(0) < item1) issue(item_of(0), 0);
    bool waited_c = p.full_read != 0;
    bool dead = false;

    auto scalar_gates = [&](int item, float& bt, float& dsc) {
        const int ic = min(item, item1 - 1);
        const int h = ic / B, b = ic - h * B;
        const size_t bh = (size_t)b * H + h;
        bt = p.beta[bh];
        dsc = 1.f;
        if constexpr (KIND != SKETCHSSM_KDA) dsc = reinterpret_cast<const float*>(p.decay)[bh];
    };
    float bt_next = 0.f, dsc_next = 1.f;
    if (my_quads > 0) scalar_gates(item_of(0), bt_next, dsc_next);

    for (int it = 0; it < my_quads; ++it) {
        const int item = item_of(it);
        const bool active = item < item1;
        const int st = stages == 2 ? (it & 1) : 0;
        const uint32_t parity = stages == 2 ? ((it >> 1) & 1) : (it & 1);
        if (stages == 2 && it + 1 < my_quads && j == 0 && item_of(it + 1) < item1) issue(item_of(it + 1), st ^ 1);

        const int item_c = active ? item : item1 - 1;
        const int h = item_c / B, b = item_c - h * B;
        const size_t bh = (size_t)b * H + h;
        const float bt = bt_next, dsc = dsc_next;
        if (it + 1 < my_quads) scalar_gates(item_of(it + 1), bt_next, dsc_next);

        if (active) {
            if (!mbar_wait_bounded(&bars[st], parity)) {
                record_fault(p.status, p.full_read ? kFaultFullReadWait : kFaultDecodeWait, (int)blockIdx.x);
                dead = true;
            }
        }
        dead = __any_sync(0xffffffffu, dead);
        if (dead) break;

        const unsigned char* sb = my_stage + (size_t)st * sl.total;
        const IO* sK = reinterpret_cast<const IO*>(sb + sl.k_off);
        const float* sBeta = reinterpret_cast<const float*>(sb + sl.gate_off);
        const float* sDec = sBeta + L;
        const IO* sG = reinterpret_cast<const IO*>(sb + sl.g_off);

        float q0[EK], x[EK], kk[EK], gg[EK];
        load_row<EK, LPH>(reinterpret_cast<const IO*>(sb + sl.tq_off), j, q0);
        load_row<EK, LPH>(reinterpret_cast<const IO*>(sb + sl.tk_off), j, kk);
        if constexpr (KIND == SKETCHSSM_KDA) load_row<EK, LPH>(reinterpret_cast<const IO*>(sb + sl.tg_off), j, gg);

        if (p.append && active) {
            unsigned char* rh = p.ring + bh * p.rl.head_bytes;
            store_row<EK, LPH>(reinterpret_cast<IO*>(rh) + (size_t)n * K, j, kk);
            if constexpr (KIND == SKETCHSSM_KDA) {
                store_row<EK, LPH>(reinterpret_cast<IO*>(rh + p.rl.decay_off) + (size_t)n * K, j, gg);
                if (j == 0) reinterpret_cast<float*>(rh + p.rl.beta_off)[n] = bt;
            } else if (j == 0) {
                reinterpret_cast<float*>(rh + p.rl.beta_off)[n] = bt;
                reinterpret_cast<float*>(rh + p.rl.decay_off)[n] = dsc;
            }
        }

        // ---- current token, s = t ----
        float dsuf = 1.f;
        {
            float part = 0.f;
#pragma unroll
            for (int e = 0; e < EK; ++e) part = fmaf(kk[e], q0[e], part);
            const float a = bt * group_sum<LPH>(part);
            if (j == 0) sA[n] = a;
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

        if constexpr (KIND == SKETCHSSM_MAMBA2) {
            // all dot products <k_s, q_t> are independent: 16 at a time through the transposing butterfly
            constexpr int NB = 16;
            constexpr int PPL = NB >= LPH ? NB / LPH : 1;
            for (int s0 = 0; s0 < n; s0 += NB) {
                float part[NB];
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    const int s = min(s0 + i, n - 1);
                    float kr[EK];
                    load_row<EK, LPH>(sK + (size_t)s * K, j, kr);
                    float acc = 0.f;
#pragma unroll
                    for (int e = 0; e < EK; ++e) acc = fmaf(kr[e], q0[e], acc);
                    part[i] = acc;
                }
                group_reduce_transpose<LPH, NB>(part, j);
                if (NB >= LPH || (j % (LPH > NB ? LPH / NB : 1)) == 0) {
#pragma unroll
                    for (int i = 0; i < PPL; ++i) {
                        const int idx = NB >= LPH ? PPL * j + i : j / (LPH > NB ? LPH / NB : 1);
                        if (s0 + idx < n) sA[s0 + idx] = part[i];
                    }
                }
            }
            __syncwarp();
            // a_s = beta_s (prod_{j>s} a_j) <k_s, q_t>: lane j finishes slots j, j + LPH, ...; the suffix products
            // are a short serial scan that every lane repeats
            for (int s = n - 1; s >= 0; --s) {
                if ((s % LPH) == j) sA[s] = sBeta[s] * dsuf * sA[s];
                dsuf *= sDec[s];
            }
#pragma unroll
            for (int e = 0; e < EK; ++e) x[e] = dsuf * q0[e];
        } else {
#pragma unroll 2
            for (int s = n - 1; s >= 0; --s) {
                float kr[EK];
                load_row<EK, LPH>(sK + (size_t)s * K, j, kr);
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < EK; ++e) part = fmaf(kr[e], x[e], part);
                const float a = sBeta[s] * group_sum<LPH>(part);
                if (j == 0) sA[s] = a;
                if constexpr (KIND == SKETCHSSM_GDN) {
                    const float d = sDec[s];
#pragma unroll
                    for (int e = 0; e < EK; ++e) x[e] = d * fmaf(-a, kr[e], x[e]);
                } else {
                    float gr[EK];
                    load_row<EK, LPH>(sG + (size_t)s * K, j, gr);
#pragma unroll
                    for (int e = 0; e < EK; ++e) x[e] = gr[e] * fmaf(-a, kr[e], x[e]);
                }
            }
        }

        if (!p.full_read) {
            if (!waited_c) {
                if (!mbar_wait_bounded(cbar, 0)) {
                    record_fault(p.status, kFaultDecodeWait, -1 - (int)blockIdx.x);
                    dead = true;
                }
                dead = __any_sync(0xffffffffu, dead);
                if (dead) break;
                waited_c = true;
            }
            const float* sC = reinterpret_cast<const float*>(smem + (size_t)(h - h_first) * ds.coef_slot_bytes);
            float part[RP];
#pragma unroll
            for (int g = 0; g < RP; ++g) {
                float cw[EK];
                load_row<EK, LPH>(sC + (size_t)g * K, j, cw);
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < EK; ++e) acc = fmaf(cw[e], x[e], acc);
                part[g] = acc;
            }
            group_reduce_transpose<LPH, RP>(part, j);
            if (RP >= LPH) {
#pragma unroll
                for (int i = 0; i < CPL; ++i) sW[CPL * j + i] = part[i];
            } else if ((j % (LPH > RP ? LPH / RP : 1)) == 0) {
                sW[j / (LPH > RP ? LPH / RP : 1)] = part[0];
            }
        } else {
            store_row<EK, LPH>(sW, j, x);
        }
        __syncwarp();

        // ---- output phase: o = sum_r w_r row_r, rows straight from global memory (L2) ----
        {
            float o[EV];
#pragma unroll
            for (int e = 0; e < EV; ++e) o[e] = 0.f;
            float tv[EV];
            load_row<EV, LPH>(reinterpret_cast<const IO*>(p.v) + bh * V, j, tv);
            const int nrows = p.full_read ? K : R;
            const float* rows = p.full_read ? p.state + bh * (size_t)K * V : p.sketch + bh * (size_t)R * V;
            for (int r0 = 0; r0 < nrows; r0 += RB) {
                float t[RB][EV];
#pragma unroll
                for (int i = 0; i < RB; ++i) load_row<EV, LPH>(rows + (size_t)min(r0 + i, nrows - 1) * V, j, t[i]);
#pragma unroll
                for (int i = 0; i < RB; ++i) {
                    const float wt = r0 + i < nrows ? sW[r0 + i] : 0.f;
#pragma unroll
                    for (int e = 0; e < EV; ++e) o[e] = fmaf(wt, t[i][e], o[e]);
                }
            }
            const IO* rv = reinterpret_cast<const IO*>(p.ring + bh * p.rl.head_bytes + p.rl.v_off);
            for (int s0 = 0; s0 < n; s0 += RB) {
                float t[RB][EV];
#pragma unroll
                for (int i = 0; i < RB; ++i) load_row<EV, LPH>(rv + (size_t)min(s0 + i, n - 1) * V, j, t[i]);
#pragma unroll
                for (int i = 0; i < RB; ++i) {
                    const float wt = s0 + i < n ? sA[s0 + i] : 0.f;
#pragma unroll
                    for (int e = 0; e < EV; ++e) o[e] = fmaf(wt, t[i][e], o[e]);
                }
            }
            {
                const float wt = sA[n];
#pragma unroll
                for (int e = 0; e < EV; ++e) o[e] = fmaf(wt, tv[e], o[e]);
            }
            if (active) {
                if (p.append)
                    store_row<EV, LPH>(reinterpret_cast<IO*>(p.ring + bh * p.rl.head_bytes + p.rl.v_off) + (size_t)n * V, j, tv);
                if (p.out_bf16) store_row<EV, LPH>(reinterpret_cast<__nv_bfloat16*>(p.out) + bh * V, j, o);
                else store_row<EV, LPH>(reinterpret_cast<float*>(p.out) + bh * V, j, o);
            }
        }
        __syncwarp();  // all lanes are done with this stage and the weight scratch before either is reused
        if (stages == 1 && it + 1 < my_quads && j == 0 && item_of(it + 1) < item1) issue(item_of(it + 1), 0);
    }

    if (dead) {   // bounded grace period for copies still in flight before the CTA retires
        mbar_wait_bounded(&bars[0], 0, 1u << 16);
        if (stages == 2) mbar_wait_bounded(&bars[1], 0, 1u << 16);
    }
    if (!waited_c && threadIdx.x == 0 && item1 > item0) mbar_wait_bounded(cbar, 0, 1u << 20);
}


// ---------------------------------------------------------------------------------------------
// launch
// ---------------------------------------------------------------------------------------------
template <int KIND, typename IO, int K, int V, int LPH, int RP>
static int launch_fused_t(Ctx* ctx, Params p, cudaStream_t stream) {
    constexpr int HPW = 32 / LPH;
    const WStage sl = make_wstage(KIND, (int)sizeof(IO), K, p.L, p.n_before);
    const uint32_t smem_budget = 227u * 1024u;
    if (ctx->sm_count == 0) {
        int dev = 0, sms = 0;
        if ((ctx->last_cuda_error = cudaGetDevice(&dev)) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
        if ((ctx->last_cuda_error = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return SKETCHSSM_CUDA_ERROR;
        ctx->sm_count = sms;
    }
    // warps per CTA / stages / CTAs per SM: as many warps per SM as shared memory allows, capped at `cap`
    // (the kernel needs about 128 registers per thread, so 16 warps fill the register file)
    const int cap = p.max_warps_per_sm > 0 ? p.max_warps_per_sm : 16;
    int best_nw = 0, best_st = 1, best_ctas = 1, best_score = -1;
    const int want_st = (p.stages == 1 || p.stages == 2) ? p.stages : 0;
    const int want_nw = p.warps_per_cta;
    for (int st = 1; st <= 2; ++st) {
        if (want_st && st != want_st) continue;
        for (int nw = 8; nw >= 1; --nw) {
            if (want_nw && nw != want_nw) continue;
            const WSmem d = make_fsmem(K, RP, nw * HPW, st, p.full_read, sl.total);
            if (d.total > smem_budget) continue;
            int ctas = (int)((228u * 1024u) / (d.total + 1024u));
            if (ctas * nw > cap) ctas = cap / nw;
            if (ctas < 1) continue;
            // prefer more resident warps, then two stages, then fewer CTAs (less coefficient-map staging)
            const int score = ctas * nw * 100 + st * 10 + (8 - ctas);
            if (score > best_score) { best_score = score; best_nw = nw; best_st = st; best_ctas = ctas; }
        }
    }
    if (best_nw == 0) return SKETCHSSM_UNSUPPORTED_SHAPE;
    p.stages = best_st;
    const WSmem d = make_fsmem(K, RP, best_nw * HPW, best_st, p.full_read, sl.total);
    auto kern = decode_fused_kernel<KIND, IO, K, V, LPH, RP>;
    if ((ctx->last_cuda_error = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)d.total)) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    long long grid = (long long)ctx->sm_count * best_ctas;
    const long long total = (long long)p.B * p.H;
    const long long min_items = (long long)best_nw * HPW;       // at least one quad per warp when possible
    if (grid > (total + min_items - 1) / min_items) grid = (total + min_items - 1) / min_items;
    if (grid < p.H) grid = p.H;                                  // a CTA's range then spans at most two head indices
    if (grid > total) grid = total;
    kern<<<dim3((unsigned)grid), best_nw * 32, d.total, stream>>>(p);
    if ((ctx->last_cuda_error = cudaGetLastError()) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

template <int KIND, typename IO, int K, int V>
static int launch_fused_rank(Ctx* ctx, const Params& p, cudaStream_t stream) {
    const int R = p.full_read ? 1 : p.R;     // full-read mode has no coefficient map: smallest instantiation
    if (R <= 8) return launch_fused_t<KIND, IO, K, V, 8, 8>(ctx, p, stream);
    if (R <= 16) return launch_fused_t<KIND, IO, K, V, 8, 16>(ctx, p, stream);
    if (R <= 32) return launch_fused_t<KIND, IO, K, V, 8, 32>(ctx, p, stream);
    return launch_fused_t<KIND, IO, K, V, 8, 64>(ctx, p, stream);
}

template <int KIND, typename IO>
static int launch_fused_shape(Ctx* ctx, const Params& p, cudaStream_t stream) {
    const int K = ctx->cfg.dk, V = ctx->cfg.dv;
    if (K == 128 && V == 128) return launch_fused_rank<KIND, IO, 128, 128>(ctx, p, stream);
    if (K == 128 && V == 64) return launch_fused_rank<KIND, IO, 128, 64>(ctx, p, stream);
    if (K == 64 && V == 64) return launch_fused_rank<KIND, IO, 64, 64>(ctx, p, stream);
    if (K == 64 && V == 128) return launch_fused_rank<KIND, IO, 64, 128>(ctx, p, stream);
    return SKETCHSSM_UNSUPPORTED_SHAPE;
}

// One translation unit per (recurrence kind, I/O type) keeps the builds parallel.
#if !defined(SKETCHSSM_GROUP_KIND) || !defined(SKETCHSSM_GROUP_IO)
#error "compile with -DSKETCHSSM_GROUP_KIND=0|1|2 -DSKETCHSSM_GROUP_IO=0|1"
#endif
#if SKETCHSSM_GROUP_IO == 0
using GroupIO = float;
#define SKETCHSSM_GROUP_FN(kind) launch_decode_group_##kind##_f32
#else
using GroupIO = __nv_bfloat16;
#define SKETCHSSM_GROUP_FN(kind) launch_decode_group_##kind##_bf16
#endif
#if SKETCHSSM_GROUP_KIND == 0
int SKETCHSSM_GROUP_FN(mamba2)(Ctx* ctx, const Params& p, cudaStream_t stream) {
    return launch_fused_shape<SKETCHSSM_MAMBA2, GroupIO>(ctx, p, stream);
}
#elif SKETCHSSM_GROUP_KIND == 1
int SKETCHSSM_GROUP_FN(gdn)(Ctx* ctx, const Params& p, cudaStream_t stream) {
    return launch_fused_shape<SKETCHSSM_GDN, GroupIO>(ctx, p, stream);
}
#else
int SKETCHSSM_GROUP_FN(kda)(Ctx* ctx, const Params& p, cudaStream_t stream) {
    return launch_fused_shape<SKETCHSSM_KDA, GroupIO>(ctx, p, stream);
}
#endif

}  // namespace sketchssm
