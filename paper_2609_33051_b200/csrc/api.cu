// C ABI of the SketchSSM decode hot path: argument checking and kernel dispatch.
#include <new>

#include "internal.cuh"

using namespace sketchssm;

struct sketchssm_ctx : public Ctx {
    int tune_batches_per_cta;
    int tune_stages;
    int tune_warps_per_cta;
    int tune_decode_impl;   // 0: two kernels (weights + output rows), 1: warp-per-head kernel
    int tune_max_warps;
    int tune_update_impl;
    int tune_pdl;
};

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

RingLayout ring_layout(const sketchssm_config& c, int io) {
    RingLayout r;
    r.v_off = (size_t)c.buf_len * c.dk * io;
    r.beta_off = r.v_off + (size_t)c.buf_len * c.dv * io;
    r.decay_off = r.beta_off + (size_t)c.buf_len * 4;
    const size_t decay_bytes = c.kind == SKETCHSSM_KDA ? (size_t)c.buf_len * c.dk * io : (size_t)c.buf_len * 4;
    r.head_bytes = r.decay_off + decay_bytes;
    return r;
}

int check_token_ptrs(const void* q, const void* k, const void* v, const void* beta, const void* decay, const void* out) {
    const void* ps[6] = {q, k, v, beta, decay, out};
    for (const void* p : ps) {
        if (p == nullptr || !aligned16(p)) return SKETCHSSM_INVALID_ARG;
    }
    return SKETCHSSM_OK;
}

Params base_params(const sketchssm_ctx* ctx) {
    Params p{};
    p.state = static_cast<float*>(ctx->bufs.state);
    p.sketch = static_cast<float*>(ctx->bufs.sketch);
    p.ring = static_cast<unsigned char*>(ctx->bufs.ring);
    p.omega = static_cast<const float*>(ctx->bufs.omega);
    p.coef = static_cast<const float*>(ctx->bufs.coef);
    p.status = static_cast<int*>(ctx->bufs.status);
    p.work = static_cast<float*>(ctx->bufs.work);
    p.head_rank = static_cast<const int*>(ctx->bufs.head_rank);
    p.n_dev = nullptr;
    p.n_cap = 0;
    p.wstride = ctx->cfg.dk + ctx->cfg.buf_len;
    p.rl = ctx->ring;
    p.B = ctx->cfg.batch; p.H = ctx->cfg.heads; p.R = ctx->cfg.rank; p.L = ctx->cfg.buf_len;
    p.dk = ctx->cfg.dk; p.dv = ctx->cfg.dv;
    p.out_bf16 = ctx->cfg.out_dtype == SKETCHSSM_BF16;
    p.batches_per_cta = ctx->tune_batches_per_cta;
    p.stages = ctx->tune_stages;
    p.warps_per_cta = ctx->tune_warps_per_cta;
    p.max_warps_per_sm = ctx->tune_max_warps;
    p.update_impl = ctx->tune_update_impl;
    p.pdl = ctx->tune_pdl;
    p.coef_per_seq = ctx->cfg.coef_per_seq;
    p.pivots = ctx->cfg.coef_pivots;
    p.ridge_lambda = ctx->cfg.ridge_lambda;
    p.sketch_bf16 = ctx->cfg.sketch_dtype == SKETCHSSM_BF16;
    p.erase = ctx->cfg.erase_factors ? static_cast<float*>(ctx->bufs.erase) : nullptr;
    return p;
}

int set_device(const sketchssm_ctx* ctx) {
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    if (cur != ctx->cfg.device && cudaSetDevice(ctx->cfg.device) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    return SKETCHSSM_OK;
}

// Argument checks shared by every decode entry point, then the parameter block of a decode launch.
int decode_params(sketchssm_ctx* ctx, int full_read, int n_before, const void* q, const void* k, const void* v,
                  const void* beta, const void* decay, void* out, uint32_t flags, Params* out_p) {
    if (ctx == nullptr) return SKETCHSSM_INVALID_ARG;
    ctx->last_launches = 0;
    if (!ctx->bound) return SKETCHSSM_NOT_BOUND;
    if (n_before < 0 || n_before > ctx->cfg.buf_len - 1) return SKETCHSSM_INVALID_ARG;
    if (flags & ~SKETCHSSM_NO_APPEND) return SKETCHSSM_INVALID_ARG;
    const int rc = check_token_ptrs(q, k, v, beta, decay, out);
    if (rc != SKETCHSSM_OK) return rc;
    Params p = base_params(ctx);
    p.q = q; p.k = k; p.v = v; p.beta = static_cast<const float*>(beta); p.decay = decay; p.out = out;
    p.n_before = n_before;
    p.has_token = 1;
    p.append = (flags & SKETCHSSM_NO_APPEND) ? 0 : 1;
    p.full_read = full_read;
    *out_p = p;
    return SKETCHSSM_OK;
}

// The flush kernel for this configuration: the warp-specialised tensor-core kernels where their shape limits allow,
// the single-group tensor-core kernel for Mamba-2 ranks above 32, CUDA cores otherwise.
int dispatch_update(sketchssm_ctx* ctx, const Params& p, cudaStream_t cs) {
    if (p.update_impl != 1) {
        int rc;
        if (p.update_impl != 3) {
            rc = launch_update_tc_ws(ctx, p, cs);
            if (rc != SKETCHSSM_UNSUPPORTED_SHAPE) return rc;
        }
        rc = launch_update_tc(ctx, p, cs);
        if (rc != SKETCHSSM_UNSUPPORTED_SHAPE) return rc;
        // gated delta rule: warp-specialised tensor-core kernel (up to 64 tokens in blocks of 16, rank <= 16)
        if (p.update_impl == 0) {
            rc = launch_update_tc_ws_gdn(ctx, p, cs);
            if (rc != SKETCHSSM_UNSUPPORTED_SHAPE) return rc;
            // delta rule with per-channel decay: warp-specialised tensor-core kernel (up to 64 tokens in blocks of 32, rank <= 16)
            rc = launch_update_tc_ws_kda(ctx, p, cs);
            if (rc != SKETCHSSM_UNSUPPORTED_SHAPE) return rc;
        }
    }
    return launch_update(ctx, p, cs);
}

int decode_common(sketchssm_ctx* ctx, int full_read, int n_before, const void* q, const void* k, const void* v,
                  const void* beta, const void* decay, void* out, uint32_t flags, void* stream) {
    Params p;
    int rc = decode_params(ctx, full_read, n_before, q, k, v, beta, decay, out, flags, &p);
    if (rc != SKETCHSSM_OK) return rc;
    rc = set_device(ctx);
    if (rc != SKETCHSSM_OK) return rc;
    // Only a state update writes the sketch.  Unless that was the previous call on this context (it may still be running:
    // programmatic dependent launch), a decode step may read U before it waits for its predecessor in the stream.
    // (The projected erase vectors travel with the sketch rows and are written by the previous decode step: no early read.)
    p.early_sketch = (!full_read && !ctx->sketch_fresh && p.erase == nullptr) ? 1 : 0;
    ctx->sketch_fresh = false;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (p.early_sketch) {
        // A step recorded into a stream capture is replayed after whatever the graph's previous launch left running,
        // which may be a state update of this context: the recorded node always waits first.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(cs, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) p.early_sketch = 0;
    }
    const bool bf = ctx->cfg.io_dtype == SKETCHSSM_BF16;
    if (ctx->tune_decode_impl == 1) return launch_decode(ctx, p, cs);
    // the two-kernel decode stages one map per head index, knows one rank and the value widths 64 and 128
    if ((p.coef_per_seq && !full_read) || p.head_rank != nullptr || ctx->cfg.dv == 80 || (p.sketch_bf16 && !full_read) ||
        (p.erase != nullptr && !full_read))
        return SKETCHSSM_UNSUPPORTED_SHAPE;
    switch (ctx->cfg.kind) {
        case SKETCHSSM_MAMBA2:
            return bf ? launch_decode_split_mamba2_bf16(ctx, p, cs) : launch_decode_split_mamba2_f32(ctx, p, cs);
        case SKETCHSSM_GDN:
            return bf ? launch_decode_split_gdn_bf16(ctx, p, cs) : launch_decode_split_gdn_f32(ctx, p, cs);
        default:
            return bf ? launch_decode_split_kda_bf16(ctx, p, cs) : launch_decode_split_kda_f32(ctx, p, cs);
    }
}

}  // namespace

extern "C" {

int sketchssm_create(const sketchssm_config* cfg, sketchssm_ctx** out) {
    if (cfg == nullptr || out == nullptr) return SKETCHSSM_INVALID_ARG;
    *out = nullptr;
    if (cfg->kind < SKETCHSSM_MAMBA2 || cfg->kind > SKETCHSSM_KDA) return SKETCHSSM_INVALID_ARG;
    if (cfg->io_dtype != SKETCHSSM_F32 && cfg->io_dtype != SKETCHSSM_BF16) return SKETCHSSM_INVALID_ARG;
    if (cfg->out_dtype != SKETCHSSM_F32 && cfg->out_dtype != SKETCHSSM_BF16) return SKETCHSSM_INVALID_ARG;
    if (cfg->batch < 1 || cfg->heads < 1 || cfg->device < 0) return SKETCHSSM_INVALID_ARG;
    if (cfg->rank < 1 || cfg->buf_len < 1) return SKETCHSSM_INVALID_ARG;
    if ((cfg->dk != 64 && cfg->dk != 128) || (cfg->dv != 64 && cfg->dv != 128 && !(cfg->dv == 80 && cfg->dk == 128)))
        return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (cfg->rank > kMaxRank) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (cfg->buf_len < 4 || cfg->buf_len > kMaxBufLen || (cfg->buf_len & 3)) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if ((size_t)cfg->batch * cfg->heads > (size_t)1 << 24) return SKETCHSSM_UNSUPPORTED_SHAPE;
    if (cfg->coef_per_seq != 0 && cfg->coef_per_seq != 1) return SKETCHSSM_INVALID_ARG;
    if (cfg->sketch_dtype != SKETCHSSM_F32 && cfg->sketch_dtype != SKETCHSSM_BF16) return SKETCHSSM_INVALID_ARG;
    if (cfg->erase_factors != 0 && cfg->erase_factors != 1) return SKETCHSSM_INVALID_ARG;
    if (cfg->erase_factors) {
        if (cfg->kind == SKETCHSSM_MAMBA2) return SKETCHSSM_INVALID_ARG;            // no erase term: nothing to project
        // rows of r floats travel as bulk copies (16-byte units); the per-slot dot products and the two coefficient
        // vectors share the decode kernel's per-warp scratch
        if ((cfg->rank & 3) || cfg->buf_len > 32 || 2 * ((cfg->rank + 7) & ~7) > cfg->dk) return SKETCHSSM_UNSUPPORTED_SHAPE;
        if (cfg->sketch_dtype == SKETCHSSM_BF16 && (cfg->rank & 7)) return SKETCHSSM_UNSUPPORTED_SHAPE;      // bfloat16 rows of 16-byte units
    }
    if (cfg->coef_per_seq) {
        if (!(cfg->ridge_lambda > 0.f) || cfg->coef_pivots < 0) return SKETCHSSM_INVALID_ARG;
        if (cfg->coef_pivots > 8) return SKETCHSSM_UNSUPPORTED_SHAPE;
    }
    sketchssm_ctx* c = new (std::nothrow) sketchssm_ctx();
    if (c == nullptr) return SKETCHSSM_INVALID_ARG;
    c->cfg = *cfg;
    c->io_size = cfg->io_dtype == SKETCHSSM_BF16 ? 2 : 4;
    c->ring = ring_layout(*cfg, c->io_size);
    c->bound = false;
    c->bufs = sketchssm_buffers{};
    c->last_launches = 0;
    c->sketch_fresh = true;
    c->last_cuda_error = cudaSuccess;
    c->tune_batches_per_cta = 0;
    c->tune_stages = 0;
    c->tune_warps_per_cta = 0;
    c->tune_decode_impl = 1;
    c->tune_max_warps = 0;
    c->tune_update_impl = 0;
    c->tune_pdl = 1;
    *out = c;
    return SKETCHSSM_OK;
}

int sketchssm_destroy(sketchssm_ctx* ctx) {
    if (ctx == nullptr) return SKETCHSSM_INVALID_ARG;
    delete ctx;
    return SKETCHSSM_OK;
}

int sketchssm_query_sizes(const sketchssm_ctx* ctx, sketchssm_sizes* out) {
    if (ctx == nullptr || out == nullptr) return SKETCHSSM_INVALID_ARG;
    const sketchssm_config& c = ctx->cfg;
    const size_t bh = (size_t)c.batch * c.heads;
    out->state_bytes = bh * c.dk * c.dv * 4;
    const size_t su = c.sketch_dtype == SKETCHSSM_BF16 ? 2 : 4;
    out->sketch_bytes = bh * c.rank * c.dv * su;
    out->ring_bytes = bh * ctx->ring.head_bytes;
    out->omega_bytes = (size_t)c.heads * c.dk * c.rank * 4;
    out->coef_bytes = (c.coef_per_seq ? bh : (size_t)c.heads) * c.rank * c.dk * su;
    out->status_bytes = (((size_t)(kStatusInts + 4 + c.heads) * sizeof(int32_t)) + 15) & ~(size_t)15;   // status word + tile scheduler counters
    out->work_bytes = bh * (size_t)(c.dk + c.buf_len) * 4;
    out->ring_head_bytes = ctx->ring.head_bytes;
    out->ring_v_offset = ctx->ring.v_off;
    out->ring_beta_offset = ctx->ring.beta_off;
    out->ring_decay_offset = ctx->ring.decay_off;
    out->alignment = 16;
    out->erase_bytes = c.erase_factors ? bh * (size_t)c.buf_len * c.rank * su : 0;
    return SKETCHSSM_OK;
}

int sketchssm_bind(sketchssm_ctx* ctx, const sketchssm_buffers* b) {
    if (ctx == nullptr || b == nullptr) return SKETCHSSM_INVALID_ARG;
    const void* ps[7] = {b->state, b->sketch, b->ring, b->omega, b->coef, b->status, b->work};
    for (const void* p : ps) {
        if (p == nullptr || !aligned16(p)) return SKETCHSSM_INVALID_ARG;
    }
    if (b->head_rank != nullptr && (reinterpret_cast<uintptr_t>(b->head_rank) & 3u)) return SKETCHSSM_INVALID_ARG;
    if (ctx->cfg.erase_factors && (b->erase == nullptr || !aligned16(b->erase))) return SKETCHSSM_INVALID_ARG;
    ctx->bufs = *b;
    ctx->bound = true;
    ctx->sketch_fresh = true;       // whatever filled the buffers may still be running
    return SKETCHSSM_OK;
}

int sketchssm_state_update(sketchssm_ctx* ctx, int n_before, const void* q, const void* k, const void* v,
                           const void* beta, const void* decay, void* out, uint32_t flags, void* stream) {
    if (ctx == nullptr) return SKETCHSSM_INVALID_ARG;
    ctx->last_launches = 0;
    if (!ctx->bound) return SKETCHSSM_NOT_BOUND;
    if (flags & ~SKETCHSSM_NO_SKETCH) return SKETCHSSM_INVALID_ARG;
    const int n_tok = (k != nullptr) + (v != nullptr) + (beta != nullptr) + (decay != nullptr);
    if (n_tok != 0 && n_tok != 4) return SKETCHSSM_INVALID_ARG;
    const bool has_token = n_tok == 4;
    if ((q == nullptr) != (out == nullptr)) return SKETCHSSM_INVALID_ARG;
    if (n_before < 0 || n_before + (has_token ? 1 : 0) > ctx->cfg.buf_len) return SKETCHSSM_INVALID_ARG;
    const void* ps[6] = {q, k, v, beta, decay, out};
    for (const void* p : ps) {
        if (p != nullptr && !aligned16(p)) return SKETCHSSM_INVALID_ARG;
    }
    const bool sketch = !(flags & SKETCHSSM_NO_SKETCH);
    const int n_tot = n_before + (has_token ? 1 : 0);
    if (n_tot == 0 && !sketch && out == nullptr) return SKETCHSSM_OK;  // nothing to do
    int rc = set_device(ctx);
    if (rc != SKETCHSSM_OK) return rc;
    Params p = base_params(ctx);
    p.q = q; p.k = k; p.v = v; p.beta = static_cast<const float*>(beta); p.decay = decay; p.out = out;
    p.n_before = n_before;
    p.has_token = has_token ? 1 : 0;
    p.write_sketch = sketch ? 1 : 0;
    p.write_state = n_tot > 0 ? 1 : 0;
    ctx->sketch_fresh = true;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    rc = dispatch_update(ctx, p, cs);
    if (rc != SKETCHSSM_OK) return rc;
    if (p.coef_per_seq && sketch) {
        const int launched = ctx->last_launches;
        rc = launch_coef_map(ctx, p, cs);         // C from S_new and U, after the flush kernel has completed
        if (rc != SKETCHSSM_OK) return rc;
        ctx->last_launches = launched + 1;
    }
    return SKETCHSSM_OK;
}

int sketchssm_step_mixed(sketchssm_ctx* ctx, const int32_t* phase, const void* q, const void* k, const void* v,
                         const void* beta, const void* decay, void* out, uint32_t flags, void* stream) {
    if (ctx == nullptr) return SKETCHSSM_INVALID_ARG;
    ctx->last_launches = 0;
    if (!ctx->bound) return SKETCHSSM_NOT_BOUND;
    if (phase == nullptr || (reinterpret_cast<uintptr_t>(phase) & 3u) || flags != 0) return SKETCHSSM_INVALID_ARG;
    const int L = ctx->cfg.buf_len;
    // decode part: the stage has room for the largest fill a decoding sequence may have (L - 1 buffered tokens)
    Params pd;
    int rc = decode_params(ctx, 0, L - 1, q, k, v, beta, decay, out, 0u, &pd);
    if (rc != SKETCHSSM_OK) return rc;
    rc = set_device(ctx);
    if (rc != SKETCHSSM_OK) return rc;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    pd.n_dev = phase;
    pd.early_sketch = 0;
    rc = launch_decode(ctx, pd, cs);
    if (rc != SKETCHSSM_OK) return rc;
    int launched = ctx->last_launches;
    // flush part: every flushing sequence replays its own count of buffered tokens plus the current one
    Params pu = base_params(ctx);
    pu.q = q; pu.k = k; pu.v = v; pu.beta = static_cast<const float*>(beta); pu.decay = decay; pu.out = out;
    pu.n_before = L - 1;
    pu.has_token = 1;
    pu.write_sketch = 1;
    pu.write_state = 1;
    pu.n_dev = phase;
    rc = launch_update(ctx, pu, cs);
    if (rc != SKETCHSSM_OK) return rc;
    launched += ctx->last_launches;
    if (pu.coef_per_seq) {
        rc = launch_coef_map(ctx, pu, cs);
        if (rc != SKETCHSSM_OK) return rc;
        launched += 1;
    }
    ctx->last_launches = launched;
    ctx->sketch_fresh = true;
    return SKETCHSSM_OK;
}

int sketchssm_decode_step(sketchssm_ctx* ctx, int n_before, const void* q, const void* k, const void* v,
                          const void* beta, const void* decay, void* out, uint32_t flags, void* stream) {
    return decode_common(ctx, 0, n_before, q, k, v, beta, decay, out, flags, stream);
}

int sketchssm_full_read_decode(sketchssm_ctx* ctx, int n_before, const void* q, const void* k, const void* v,
                               const void* beta, const void* decay, void* out, uint32_t flags, void* stream) {
    return decode_common(ctx, 1, n_before, q, k, v, beta, decay, out, flags, stream);
}

int sketchssm_decode_step_static(sketchssm_ctx* ctx, int n_before, const void* q, const void* k, const void* v,
                                 const void* beta, const void* decay, void* out, uint32_t flags, void* stream) {
    Params p;
    int rc = decode_params(ctx, 0, n_before, q, k, v, beta, decay, out, flags, &p);
    if (rc != SKETCHSSM_OK) return rc;
    // runs the two-kernel decode (one map per head index, one rank, value widths 64 and 128)
    if (ctx->cfg.coef_per_seq || ctx->bufs.head_rank != nullptr || ctx->cfg.dv == 80 || ctx->cfg.sketch_dtype == SKETCHSSM_BF16 ||
        ctx->cfg.erase_factors)
        return SKETCHSSM_UNSUPPORTED_SHAPE;
    // the size limit of the library's static array is checked (on the host, before any CUDA call) by the launcher
    const sketchssm_config& c = ctx->cfg;
    if ((size_t)c.batch * c.heads * (size_t)(c.dk + c.buf_len) * sizeof(float) > (size_t)SKETCHSSM_STATIC_WORK_BYTES)
        return SKETCHSSM_UNSUPPORTED_SHAPE;
    rc = set_device(ctx);
    if (rc != SKETCHSSM_OK) return rc;
    return launch_decode_static(ctx, p, static_cast<cudaStream_t>(stream));
}

int sketchssm_step_host(sketchssm_ctx* ctx, int op, int n_before, const void* hq, const void* hk, const void* hv,
                        const void* hbeta, const void* hdecay, void* hout, const sketchssm_staging* st,
                        uint32_t flags, void* stream) {
    if (ctx == nullptr || st == nullptr) return SKETCHSSM_INVALID_ARG;
    if (op < SKETCHSSM_OP_DECODE || op > SKETCHSSM_OP_UPDATE) return SKETCHSSM_INVALID_ARG;
    if (hq == nullptr || hk == nullptr || hv == nullptr || hbeta == nullptr || hdecay == nullptr || hout == nullptr)
        return SKETCHSSM_INVALID_ARG;
    if (!ctx->bound) return SKETCHSSM_NOT_BOUND;
    int rc = check_token_ptrs(st->q, st->k, st->v, st->beta, st->decay, st->out);
    if (rc != SKETCHSSM_OK) return rc;
    rc = set_device(ctx);
    if (rc != SKETCHSSM_OK) return rc;
    const sketchssm_config& c = ctx->cfg;
    const size_t bh = (size_t)c.batch * c.heads;
    const size_t qk_bytes = bh * c.dk * ctx->io_size, v_bytes = bh * c.dv * ctx->io_size;
    const size_t dec_bytes = c.kind == SKETCHSSM_KDA ? qk_bytes : bh * 4;
    const size_t out_bytes = bh * c.dv * (c.out_dtype == SKETCHSSM_BF16 ? 2 : 4);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(st->q, hq, qk_bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(st->k, hk, qk_bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(st->v, hv, v_bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(st->beta, hbeta, bh * 4, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(st->decay, hdecay, dec_bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) { ctx->last_cuda_error = e; return SKETCHSSM_CUDA_ERROR; }
    if (op == SKETCHSSM_OP_UPDATE)
        rc = sketchssm_state_update(ctx, n_before, st->q, st->k, st->v, st->beta, st->decay, st->out, flags, stream);
    else
        rc = decode_common(ctx, op == SKETCHSSM_OP_FULL_READ, n_before, st->q, st->k, st->v, st->beta, st->decay,
                           st->out, flags, stream);
    if (rc != SKETCHSSM_OK) return rc;
    e = cudaMemcpyAsync(hout, st->out, out_bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) { ctx->last_cuda_error = e; return SKETCHSSM_CUDA_ERROR; }
    return SKETCHSSM_OK;
}

int sketchssm_read_status(sketchssm_ctx* ctx, int32_t detail[4], void* stream) {
    if (ctx == nullptr) return SKETCHSSM_INVALID_ARG;
    if (!ctx->bound) return SKETCHSSM_NOT_BOUND;
    int rc = set_device(ctx);
    if (rc != SKETCHSSM_OK) return rc;
    int32_t host[kStatusInts] = {0, 0, 0, 0};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(host, ctx->bufs.status, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return SKETCHSSM_CUDA_ERROR;
    if (cudaStreamSynchronize(s) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    if (detail != nullptr) {
        for (int i = 0; i < kStatusInts; ++i) detail[i] = host[i];
    }
    return host[0] == 0 ? SKETCHSSM_OK : SKETCHSSM_DEVICE_TIMEOUT;
}

int sketchssm_selftest_wait_timeout(sketchssm_ctx* ctx, int poll_limit, int where, void* stream) {
    if (ctx == nullptr) return SKETCHSSM_INVALID_ARG;
    ctx->last_launches = 0;
    if (!ctx->bound) return SKETCHSSM_NOT_BOUND;
    if (poll_limit < 1 || poll_limit > (1 << 16)) return SKETCHSSM_INVALID_ARG;
    const int rc = set_device(ctx);
    if (rc != SKETCHSSM_OK) return rc;
    return launch_wait_probe(ctx, poll_limit, where, static_cast<cudaStream_t>(stream));
}

const char* sketchssm_last_cuda_error(const sketchssm_ctx* ctx) {
    return ctx == nullptr ? "no context" : cudaGetErrorString(ctx->last_cuda_error);
}

int sketchssm_last_launch_count(const sketchssm_ctx* ctx) { return ctx == nullptr ? 0 : ctx->last_launches; }

int sketchssm_tune(sketchssm_ctx* ctx, const char* key, int value) {
    if (ctx == nullptr || key == nullptr) return SKETCHSSM_INVALID_ARG;
    auto eq = [](const char* a, const char* b) {
        while (*a && *b && *a == *b) { ++a; ++b; }
        return *a == *b;
    };
    if (eq(key, "decode_batches_per_cta")) { ctx->tune_batches_per_cta = value; return SKETCHSSM_OK; }
    if (eq(key, "decode_stages")) { ctx->tune_stages = value; return SKETCHSSM_OK; }
    if (eq(key, "decode_warps_per_cta")) { ctx->tune_warps_per_cta = value; return SKETCHSSM_OK; }
    if (eq(key, "decode_max_warps_per_sm")) { ctx->tune_max_warps = value; return SKETCHSSM_OK; }
    if (eq(key, "pdl")) { ctx->tune_pdl = value; return SKETCHSSM_OK; }
    if (eq(key, "update_impl")) { ctx->tune_update_impl = value; return SKETCHSSM_OK; }
    if (eq(key, "decode_impl")) { ctx->tune_decode_impl = value; return SKETCHSSM_OK; }
    return SKETCHSSM_INVALID_ARG;
}

const char* sketchssm_status_string(int status) {
    switch (status) {
        case SKETCHSSM_OK: return "ok";
        case SKETCHSSM_INVALID_ARG: return "invalid argument";
        case SKETCHSSM_UNSUPPORTED_SHAPE: return "unsupported shape";
        case SKETCHSSM_NOT_BOUND: return "buffers not bound";
        case SKETCHSSM_CUDA_ERROR: return "CUDA runtime error";
        case SKETCHSSM_DEVICE_TIMEOUT: return "bounded device wait ran out";
    }
    return "unknown status";
}

const char* sketchssm_version(void) { return "sketchssm-b200 0.1"; }

}  // extern "C"
