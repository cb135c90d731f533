// C ABI of libdq (see include/dq.h): argument checks, scratch ownership and the order of kernel launches.
#include <math.h>
#include <string.h>
#include <new>

#include "dq_kernels.cuh"

using namespace dq;

namespace {

bool bits_ok(int b) { return b == 2 || b == 4 || b == 8; }                 // gradient messages
bool model_bits_ok(int b) { return b >= 2 && b <= 11; }                    // the model: every width of Table 1
bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

template <class T>
int dev_alloc(T** p, size_t count)
{
    *p = nullptr;
    if (count == 0) count = 1;
    return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T)) == cudaSuccess ? DQ_OK : DQ_ERR_CUDA;
}

int last_error() { return cudaGetLastError() == cudaSuccess ? DQ_OK : DQ_ERR_CUDA; }

bool sparse_messages(const dq_ctx* ctx) { return ctx->cfg.sparsify && ctx->cfg.msg_format == DQ_MSG_SPARSE; }

int check_msgs(const dq_ctx* ctx, const dq_msgs* m)
{
    if (!m || !m->codes || !m->scale) return DQ_ERR_ARG;
    if (!aligned(m->codes, 16) || (m->stride & 15)) return DQ_ERR_ARG;
    if (sparse_messages(ctx)) {
        if (!m->idx || !m->nnz || m->cap < 1) return DQ_ERR_ARG;
        if (m->stride < dq_packed_bytes(m->cap, ctx->cfg.b)) return DQ_ERR_SHAPE;
    } else if (m->stride < dq_packed_bytes(ctx->cfg.d, ctx->cfg.b)) {
        return DQ_ERR_SHAPE;
    }
    return DQ_OK;
}

int check_state(const dq_ctx* ctx, const dq_state* s)
{
    if (!s || !s->x || !s->g_full || !s->norm_x) return DQ_ERR_ARG;
    if (!aligned(s->x, 16) || !aligned(s->g_full, 16)) return DQ_ERR_ARG;
    if (ctx->cfg.accelerated) {
        if (!s->y || !s->x_sum || !s->x_snap) return DQ_ERR_ARG;
        if (!aligned(s->y, 16) || !aligned(s->x_sum, 16) || !aligned(s->x_snap, 16)) return DQ_ERR_ARG;
    }
    return DQ_OK;
}

}  // namespace

extern "C" {

int64_t dq_packed_bytes(int64_t count, int b)
{
    const int64_t bytes = (count * b + 7) / 8;
    return (bytes + 15) / 16 * 16;
}

const char* dq_strerror(int status)
{
    switch (status) {
        case DQ_OK: return "ok";
        case DQ_ERR_ARG: return "bad argument (null, non-positive or misaligned)";
        case DQ_ERR_SHAPE: return "sizes inconsistent with the context";
        case DQ_ERR_BITS: return "bit width: the gradient takes 2, 4 or 8 bits, the model 2..11";
        case DQ_ERR_NONFINITE: return "vector to quantise holds NaN or Inf";
        case DQ_ERR_CAPACITY: return "sparse message exceeds its capacity";
        case DQ_ERR_CUDA: return "CUDA runtime error";
        case DQ_ERR_TIMEOUT: return "timeout";
        default: return "unknown status";
    }
}

int dq_create(dq_ctx** out, const dq_config* cfg, const dq_data* data)
{
    if (!out || !cfg) return DQ_ERR_ARG;
    *out = nullptr;
    if (cfg->d < 1 || cfg->d > ((int64_t)1 << 32) || cfg->M < 1 || cfg->M > 4096 || cfg->B < 1) return DQ_ERR_ARG;
    if (!bits_ok(cfg->b) || !model_bits_ok(cfg->bx)) return DQ_ERR_BITS;
    if (cfg->msg_format == DQ_MSG_SPARSE && !cfg->sparsify) return DQ_ERR_ARG;
    if (cfg->msg_format != DQ_MSG_SPARSE && cfg->msg_format != DQ_MSG_DENSE) return DQ_ERR_ARG;
    if (!(cfg->box_lo <= cfg->box_hi) || cfg->lambda1 < 0 || cfg->lambda2 < 0) return DQ_ERR_ARG;
    if (cfg->sparse_cap < 0 || cfg->sparse_cap > cfg->d) return DQ_ERR_ARG;
    if (!(cfg->mu >= 0.0f)) return DQ_ERR_ARG;
    if (cfg->max_delay < 0 || cfg->max_delay > 64 || (cfg->max_delay > 0 && !data)) return DQ_ERR_ARG;
    if (cfg->delay_across_epochs && (cfg->max_delay <= 0 || cfg->mu > 0.0f)) return DQ_ERR_ARG;   // needs a ring, and a fixed model width to re-read it
    if (data) {
        if (data->n < 1 || !data->values || !data->labels) return DQ_ERR_SHAPE;
        if (cfg->model == DQ_MODEL_MLP) {
            if (data->format != DQ_DENSE_F32 || cfg->hidden < 1 || cfg->classes < 2 || data->d < 1) return DQ_ERR_ARG;
            if (cfg->hidden + 3 * (int64_t)cfg->classes > 3072) return DQ_ERR_ARG;   // the output layer's row fits 48 KB of shared memory
            if (cfg->d != (int64_t)cfg->hidden * (data->d + 1) + (int64_t)cfg->classes * (cfg->hidden + 1)) return DQ_ERR_SHAPE;
        } else if (cfg->model != DQ_MODEL_LOGISTIC || data->d != cfg->d) {
            return DQ_ERR_SHAPE;
        }
        if (data->format == DQ_CSR_F32 && (!data->col_idx || !data->row_ptr)) return DQ_ERR_ARG;
        if (data->format < DQ_DENSE_F32 || data->format > DQ_DENSE_BF16) return DQ_ERR_ARG;
        if (!aligned(data->values, 16)) return DQ_ERR_ARG;
        if (data->n < cfg->M) return DQ_ERR_SHAPE;
    }
    dq_ctx* c = new (std::nothrow) dq_ctx();
    if (!c) return DQ_ERR_CUDA;
    c->cfg = *cfg;
    c->has_data = data != nullptr;
    if (data) c->data = *data;
    c->keys = expand_keys(cfg->seed);
    int dev = 0; cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { delete c; return DQ_ERR_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    const int64_t d = cfg->d; const int M = cfg->M;
    c->nchunks = (d + kChunk - 1) / kChunk;
    const bool sparse = cfg->sparsify && cfg->msg_format == DQ_MSG_SPARSE;
    int rc = DQ_OK;
    rc |= dev_alloc(&c->norm_bits, M);
    // offset table of the sparsifier: one entry per chunk; list mode uses chunks of 32 groups (256 coordinates)
    const int64_t chunk_slots = (d + 255) / 256 + 1;
    rc |= dev_alloc(&c->chunk_off, cfg->sparsify ? (size_t)M * chunk_slots : 1);
    rc |= dev_alloc(&c->tile_ptr, sparse ? (size_t)M * (c->nchunks + 1) : 1);
    // staging area for the survivors of the mask pass: kStash entries per chunk, i.e. room for a density of 1/16,
    // beyond which the sparsifier falls back to re-reading the vector
    rc |= dev_alloc(&c->stage_idx, cfg->sparsify ? (size_t)M * c->nchunks * kStash : 1);
    rc |= dev_alloc(&c->stage_val, cfg->sparsify ? (size_t)M * c->nchunks * kStash : 1);
    rc |= dev_alloc(&c->stage_ctrl, (size_t)M + 1);
    rc |= dev_alloc(&c->xnorm_bits, 2);
    rc |= dev_alloc(&c->status, 1);
    rc |= dev_alloc(&c->bits, 2);
    rc |= dev_alloc(&c->rp_dev, 1);
    // message buffers of dq_round / dq_codec_round
    c->msgs.cap = sparse ? (cfg->sparse_cap > 0 ? cfg->sparse_cap : d) : 0;
    c->msgs.stride = sparse ? dq_packed_bytes(c->msgs.cap, cfg->b) : dq_packed_bytes(d, cfg->b);
    rc |= dev_alloc(&c->msgs.codes, (size_t)c->msgs.stride * M);
    rc |= dev_alloc(&c->msgs.scale, M);
    rc |= dev_alloc(&c->msgs.idx, sparse ? (size_t)c->msgs.cap * M : 1);
    rc |= dev_alloc(&c->msgs.nnz, M);
    rc |= dev_alloc(&c->codes_x, (size_t)dq_packed_bytes(d, cfg->mu > 0.0f ? 11 : cfg->bx));
    rc |= dev_alloc(&c->bx_dev, 1);
    rc |= dev_alloc(&c->prec_stats, 11);
    rc |= dev_alloc(&c->delta_x, 1);
    // ||alpha_w||_inf, ||beta_w||_inf and the fixed-point ||alpha_w||_1 sit in one block so that one kernel of a round
    // can clear all three: [M] float | [M] u32 | [M] u64
    rc |= dev_alloc(&c->norm_block, (size_t)4 * M);
    if (c->norm_block) {
        c->ninf = reinterpret_cast<float*>(c->norm_block);
        c->beta_norm_bits = c->norm_block + M;
        c->l1_sum = reinterpret_cast<unsigned long long*>(c->norm_block + 2 * (size_t)M);
    }
    if (data) {
        rc |= dev_alloc(&c->alpha, (size_t)M * d);
        rc |= dev_alloc(&c->rows, (size_t)M * cfg->B);
        rc |= dev_alloc(&c->xhat_diff, (size_t)d * (cfg->max_delay + 1));     // a ring of broadcasts when workers may lag
        if (cfg->max_delay > 0 && cfg->delay_across_epochs && cfg->model == DQ_MODEL_LOGISTIC) {
            rc |= dev_alloc(&c->xhat_ring, (size_t)d * (cfg->max_delay + 1));
            if (rc == DQ_OK && cudaMemset(c->xhat_ring, 0, sizeof(float) * (size_t)d * (cfg->max_delay + 1)) != cudaSuccess) rc = DQ_ERR_CUDA;
        }
        rc |= dev_alloc(&c->delays_dev, M);
        rc |= dev_alloc(&c->slots_dev, M);
        if (rc == DQ_OK && cudaMemset(c->delays_dev, 0, sizeof(int32_t) * M) != cudaSuccess) rc = DQ_ERR_CUDA;
        rc |= dev_alloc(&c->g64, (size_t)d);
        rc |= dev_alloc(&c->rbuf, (size_t)M * cfg->B);
        if (cfg->model == DQ_MODEL_MLP) {
            const size_t rmax = (size_t)((int64_t)M * cfg->B > data->n ? (int64_t)M * cfg->B : data->n);
            rc |= dev_alloc(&c->mlp_rows, rmax);
            for (int k = 0; k < 2; ++k) {
                rc |= dev_alloc(&c->mlp_act[k], rmax * cfg->hidden);
                rc |= dev_alloc(&c->mlp_dh[k], rmax * cfg->hidden);
                rc |= dev_alloc(&c->mlp_dz[k], rmax * cfg->classes);
            }
        }
        if (data->format == DQ_CSR_F32) {
            // integer grid of the CSR gradient accumulator: a minibatch sum is at most max |a_ij| in magnitude (B terms
            // of at most max |a_ij| / B), so with max |a_ij| < 2^e one unit of 2^(e-61) keeps every sum below 2^61
            rc |= dev_alloc(&c->acc64, (size_t)M * d);
            int64_t nnz = 0; uint32_t vbits = 0;
            if (rc == DQ_OK && (cudaMemset(c->acc64, 0, sizeof(long long) * M * d) != cudaSuccess ||
                                cudaMemcpy(&nnz, data->row_ptr + data->n, sizeof(int64_t), cudaMemcpyDeviceToHost) != cudaSuccess)) rc = DQ_ERR_CUDA;
            if (rc == DQ_OK && nnz > 0) {
                launch_norm_inf(c, static_cast<const float*>(data->values), nnz, 1, c->xnorm_bits, nullptr);
                if (cudaMemcpy(&vbits, c->xnorm_bits, sizeof(uint32_t), cudaMemcpyDeviceToHost) != cudaSuccess) rc = DQ_ERR_CUDA;
            }
            float vmax; memcpy(&vmax, &vbits, sizeof(float));
            int e = 0;
            if (vbits != 0u && vbits < 0x7F800000u) (void)frexpf(vmax, &e);
            c->acc_scale = ldexp(1.0, 61 - e); c->acc_inv = ldexp(1.0, e - 61);
        }
        c->list_mode = sparse && data->format == DQ_CSR_F32;
        if (c->list_mode) {
            c->glist_cap = (d + 7) / 8;
            c->bm_words = (c->glist_cap + 31) / 32;
            rc |= dev_alloc(&c->touched, (size_t)M * c->bm_words);
            rc |= dev_alloc(&c->glist, (size_t)M * c->glist_cap);
            rc |= dev_alloc(&c->gcount, M);
            rc |= dev_alloc(&c->seg_count, (size_t)M * ((c->bm_words + kThreads - 1) / kThreads));
            if (rc == DQ_OK && (cudaMemset(c->touched, 0, sizeof(uint32_t) * M * c->bm_words) != cudaSuccess ||
                                cudaMemset(c->gcount, 0, sizeof(uint32_t) * M) != cudaSuccess ||
                                cudaMemset(c->alpha, 0, sizeof(float) * M * d) != cudaSuccess)) rc = DQ_ERR_CUDA;
        }
    }
    if (rc == DQ_OK && cudaMemset(c->status, 0, sizeof(int)) != cudaSuccess) rc = DQ_ERR_CUDA;
    if (rc == DQ_OK && cudaMemset(c->bx_dev, 0, sizeof(int32_t)) != cudaSuccess) rc = DQ_ERR_CUDA;
    if (rc != DQ_OK) { dq_destroy(c); cudaGetLastError(); return DQ_ERR_CUDA; }
    c->epoch = -1;
    if (fused_grad_setup(c) != DQ_OK) { dq_destroy(c); cudaGetLastError(); return DQ_ERR_CUDA; }
    small_round_setup(c);
    sparse_message_setup(c);
    *out = c;
    return DQ_OK;
}

int dq_destroy(dq_ctx* c)
{
    if (!c) return DQ_ERR_ARG;
    void* ptrs[] = {c->norm_bits, c->norm_block, c->chunk_off, c->tile_ptr, c->stage_idx, c->stage_val, c->stage_ctrl, c->delays_dev, c->slots_dev, c->xnorm_bits, c->status, c->bits,
                    c->msgs.codes, c->msgs.scale, c->msgs.idx, c->msgs.nnz, c->codes_x, c->delta_x, c->alpha,
                    c->rows, c->xhat_diff, c->g64, c->acc64, c->rbuf, c->fused_part, c->fused_cnt, c->ptouched, c->gtmp, c->xhat_ring, c->rp_dev, c->touched, c->glist, c->gcount, c->seg_count, c->bx_dev, c->prec_stats, c->mlp_rows, c->mlp_act[0], c->mlp_act[1], c->mlp_dz[0], c->mlp_dz[1], c->mlp_dh[0], c->mlp_dh[1], c->hx, c->hg, c->hv, c->hnorm};
    if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
    if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
    for (void* p : ptrs) if (p) cudaFree(p);
    delete c;
    return DQ_OK;
}

int dq_quantize_model(dq_ctx* ctx, const float* x, const float* norm_x, uint32_t round, uint8_t* codes_x, float* delta_x,
                      void* stream)
{
    if (!ctx || !x || !codes_x || !delta_x) return DQ_ERR_ARG;
    if (!aligned(codes_x, 16) || !aligned(x, 4)) return DQ_ERR_ARG;
    cudaStream_t st = as_stream(stream);
    const uint32_t* nb = reinterpret_cast<const uint32_t*>(norm_x);
    if (!nb) { launch_norm_inf(ctx, x, ctx->cfg.d, 1, ctx->xnorm_bits, st); nb = ctx->xnorm_bits; }
    launch_quantize_pack(ctx, x, ctx->cfg.d, 1, ctx->cfg.bx, nb, codes_x, dq_packed_bytes(ctx->cfg.d, ctx->cfg.bx), delta_x,
                         round, kMaster, kStreamModel, st);
    return last_error();
}

int dq_norm_inf(dq_ctx* ctx, const float* v, int M, float* norm_inf, void* stream)
{
    if (!ctx || !v || !norm_inf || M < 1 || !aligned(v, 4)) return DQ_ERR_ARG;
    launch_norm_inf(ctx, v, ctx->cfg.d, M, reinterpret_cast<uint32_t*>(norm_inf), as_stream(stream));
    return last_error();
}

int dq_quantize_sparsify_pack(dq_ctx* ctx, const float* v, const float* norm_inf, uint32_t round, dq_msgs* out, void* stream)
{
    if (!ctx || !v) return DQ_ERR_ARG;
    if (!aligned(v, 4)) return DQ_ERR_ARG;
    int rc = check_msgs(ctx, out);
    if (rc != DQ_OK) return rc;
    cudaStream_t st = as_stream(stream);
    const dq_config& c = ctx->cfg;
    const uint32_t* nb = reinterpret_cast<const uint32_t*>(norm_inf);
    if (!nb) { launch_norm_inf(ctx, v, c.d, c.M, ctx->norm_bits, st); nb = ctx->norm_bits; }
    if (!c.sparsify)
        launch_quantize_pack(ctx, v, c.d, c.M, c.b, nb, out->codes, out->stride, out->scale, round, 0u, kStreamGrad, st);
    else
        launch_sparsify_pack(ctx, v, c.d, c.M, c.b, nb, round, out, sparse_messages(ctx), st);
    return last_error();
}

int dq_master_unpack_aggregate_prox(dq_ctx* ctx, const dq_msgs* msgs, dq_state* s, float eta, float theta, void* stream)
{
    if (!ctx) return DQ_ERR_ARG;
    int rc = check_msgs(ctx, msgs);
    if (rc == DQ_OK) rc = check_state(ctx, s);
    if (rc != DQ_OK) return rc;
    if (!(eta > 0.0f) || !isfinite(eta)) return DQ_ERR_ARG;
    launch_master(ctx, msgs, sparse_messages(ctx), s, eta, theta, as_stream(stream));
    return last_error();
}

int dq_unpack(dq_ctx* ctx, const dq_msgs* msgs, int w, float* out, void* stream)
{
    if (!ctx || !out) return DQ_ERR_ARG;
    int rc = check_msgs(ctx, msgs);
    if (rc != DQ_OK) return rc;
    if (w < 0 || w >= ctx->cfg.M) return DQ_ERR_SHAPE;
    launch_unpack(ctx, msgs, sparse_messages(ctx), w, out, as_stream(stream));
    return last_error();
}

int dq_codec_round(dq_ctx* ctx, const float* v, dq_state* s, uint32_t round, float eta, float theta, uint8_t* codes_x,
                   float* delta_x, void* stream)
{
    if (!ctx || !v || !codes_x || !delta_x) return DQ_ERR_ARG;
    int rc = check_state(ctx, s);
    if (rc != DQ_OK) return rc;
    rc = dq_quantize_sparsify_pack(ctx, v, nullptr, round, &ctx->msgs, stream);
    if (rc == DQ_OK) rc = dq_master_unpack_aggregate_prox(ctx, &ctx->msgs, s, eta, theta, stream);
    if (rc == DQ_OK) rc = dq_quantize_model(ctx, s->x, s->norm_x, round, codes_x, delta_x, stream);
    return rc;
}

int dq_codec_host_setup(dq_ctx* ctx, const float* x_host, const float* g_full_host)
{
    if (!ctx || !x_host || !g_full_host || ctx->cfg.accelerated) return DQ_ERR_ARG;
    const size_t d = (size_t)ctx->cfg.d;
    int rc = DQ_OK;
    if (!ctx->hx) {
        rc |= dev_alloc(&ctx->hx, d); rc |= dev_alloc(&ctx->hg, d); rc |= dev_alloc(&ctx->hnorm, 1);
        rc |= dev_alloc(&ctx->hv, d * ctx->cfg.M);
    }
    if (rc != DQ_OK) return DQ_ERR_CUDA;
    if (cudaMemcpy(ctx->hx, x_host, d * 4, cudaMemcpyHostToDevice) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaMemcpy(ctx->hg, g_full_host, d * 4, cudaMemcpyHostToDevice) != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_codec_round_host(dq_ctx* ctx, const float* v_host, uint32_t round, float eta, uint8_t* codes_x_host, float* delta_x_host,
                        void* stream)
{
    if (!ctx || !ctx->hx || !v_host || !codes_x_host || !delta_x_host) return DQ_ERR_ARG;
    cudaStream_t st = as_stream(stream);
    const size_t d = (size_t)ctx->cfg.d;
    if (cudaMemcpyAsync(ctx->hv, v_host, d * ctx->cfg.M * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return DQ_ERR_CUDA;
    dq_state s = {ctx->hx, nullptr, ctx->hg, nullptr, nullptr, ctx->hnorm, nullptr};
    int rc = dq_codec_round(ctx, ctx->hv, &s, round, eta, 0.0f, ctx->codes_x, ctx->delta_x, stream);
    if (rc != DQ_OK) return rc;
    if (cudaMemcpyAsync(codes_x_host, ctx->codes_x, (size_t)dq_packed_bytes(ctx->cfg.d, ctx->cfg.bx), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaMemcpyAsync(delta_x_host, ctx->delta_x, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DQ_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? DQ_OK : DQ_ERR_CUDA;
}

int dq_epoch_begin(dq_ctx* ctx, dq_state* s, float theta, void* stream)
{
    if (!ctx || !ctx->has_data) return DQ_ERR_ARG;
    int rc = check_state(ctx, s);
    if (rc != DQ_OK) return rc;
    if (!s->x_snap || !s->z_snap || !aligned(s->x_snap, 16)) return DQ_ERR_ARG;
    launch_epoch_begin(ctx, s, theta, as_stream(stream));
    const bool across = ctx->cfg.max_delay > 0 && ctx->cfg.delay_across_epochs;
    if (across && ctx->xhat_ring && ctx->ring_rounds > 0)    // the kept broadcasts against the new snapshot
        launch_rediff_ring(ctx, s->x_snap, as_stream(stream));
    if (!across) ctx->ring_rounds = 0;
    ctx->rounds_in_epoch = 0;
    ctx->ticks_in_epoch = 0;
    ctx->epoch += 1;
    return last_error();
}

int dq_worker_grad(dq_ctx* ctx, const uint8_t* codes_x, const float* delta_x, int is_snapshot, const dq_state* s,
                   uint32_t round, const int32_t* batch_idx, float* alpha, float* norm_inf, void* stream)
{
    if (!ctx || !ctx->has_data || !s || !s->x_snap || !s->z_snap || !alpha || !norm_inf) return DQ_ERR_ARG;
    if (!is_snapshot && (!codes_x || !delta_x)) return DQ_ERR_ARG;
    if (!aligned(alpha, 16) || (codes_x && !aligned(codes_x, 16))) return DQ_ERR_ARG;
    launch_worker_grad(ctx, codes_x, delta_x, is_snapshot, s, round, batch_idx, alpha, norm_inf, as_stream(stream));
    return last_error();
}

// The stages of one round, enqueued on `st` (directly, or into a stream capture).
static int enqueue_round(dq_ctx* ctx, dq_state* s, uint32_t round, int flag, float eta, float theta, uint64_t* bits_down,
                         uint64_t* bits_up, void* st)
{
    int rc = DQ_OK;
    if (!flag && fused_round_applies(ctx)) {                 // large dense minibatches: model and message quantisers ride in the gradient kernel
        const BitsArgs ba0 = {bits_down ? bits_down : ctx->bits, bits_up ? bits_up : ctx->bits + 1, ctx->msgs.nnz, 0, 0, ctx->cfg.bx, ctx->cfg.b, nullptr};
        launch_fused_round(ctx, s, round, as_stream(st));
        ctx->normx_zeroed = true;                            // the gradient kernel's last block cleared ||x||_inf for the master's maximum
        launch_master(ctx, &ctx->msgs, false, s, eta, theta, as_stream(st), (bits_down || bits_up) ? &ba0 : nullptr);
        ctx->normx_zeroed = false;
        return last_error();
    }
    const bool adaptive = ctx->cfg.mu > 0.0f;
    // delayed workers: this round's xhat - xsnap goes to its slot of the ring, and every worker is pointed at the
    // slot of the broadcast it lags behind to
    const int tau = ctx->cfg.max_delay;
    float* const ring = ctx->xhat_diff;
    if (tau > 0) {
        const int t = (int)ctx->ring_rounds;
        // while a round is captured for replay the kernels take the epoch's round counter from the device instead
        if (ctx->rp_active) ctx->diff_ring = tau + 1;
        else ctx->xhat_diff = ring + (int64_t)(t % (tau + 1)) * ctx->cfg.d;
        if (flag) {                                          // xhat = xsnap: a zero difference; the network's ring holds xhat itself
            if (ctx->cfg.model == DQ_MODEL_MLP) cudaMemcpyAsync(ctx->xhat_diff, s->x_snap, sizeof(float) * ctx->cfg.d, cudaMemcpyDeviceToDevice, as_stream(st));
            else cudaMemsetAsync(ctx->xhat_diff, 0, sizeof(float) * ctx->cfg.d, as_stream(st));
            if (ctx->xhat_ring)
                cudaMemcpyAsync(ctx->xhat_ring + (int64_t)(t % (tau + 1)) * ctx->cfg.d, s->x_snap, sizeof(float) * ctx->cfg.d, cudaMemcpyDeviceToDevice, as_stream(st));
        }
        launch_set_slots(ctx, t, as_stream(st));
    }
    if (!flag) {     // model quantisation that also emits xhat - xsnap for the workers
        const uint32_t* nx = reinterpret_cast<const uint32_t*>(s->norm_x);
        float* zf = worker_accumulates(ctx) ? ctx->alpha : nullptr;
        const int64_t zn = worker_accumulates(ctx) ? (int64_t)ctx->cfg.M * ctx->cfg.d : 0;
        const float* ref = ctx->cfg.model == DQ_MODEL_MLP ? nullptr : s->x_snap;    // the network wants xhat itself
        if (!adaptive) {
            launch_quantize_pack(ctx, s->x, ctx->cfg.d, 1, ctx->cfg.bx, nx, ctx->codes_x, dq_packed_bytes(ctx->cfg.d, ctx->cfg.bx),
                                 ctx->delta_x, round, kMaster, kStreamModel, as_stream(st), ref, ctx->xhat_diff, zf, zn,
                                 reinterpret_cast<uint32_t*>(ctx->ninf), ctx->cfg.sparsify ? 4 * ctx->cfg.M : ctx->cfg.M);
        } else {     // condition (3): pick the width on the device, then launch the three specialised widths and the general kernel; all but one return at once
            launch_select_bits(ctx, s->x, s->x_snap, nx, ctx->cfg.mu, ctx->cfg.accelerated, theta, ctx->bx_dev, ctx->prec_stats, as_stream(st));
            for (int bits : {2, 4, 8, 3})                      // 3 stands for "any other width": the general kernel reads it from the device
                launch_quantize_pack(ctx, s->x, ctx->cfg.d, 1, bits, nx, ctx->codes_x, dq_packed_bytes(ctx->cfg.d, bits), ctx->delta_x,
                                     round, kMaster, kStreamModel, as_stream(st), ref, ctx->xhat_diff, zf, zn,
                                     reinterpret_cast<uint32_t*>(ctx->ninf), ctx->cfg.sparsify ? 4 * ctx->cfg.M : ctx->cfg.M, ctx->bx_dev);
        }
        ctx->diff_ready = ctx->alpha_zeroed = ctx->ninf_zeroed = ctx->normx_zeroed = true;
        ctx->sp_norms_zeroed = ctx->cfg.sparsify != 0;          // the same kernel cleared ||beta||_inf and ||alpha||_1
        if (ctx->xhat_ring)                                  // delays across epochs: keep the broadcast itself as well
            launch_dequant_xhat(ctx, ctx->codes_x, ctx->delta_x, ctx->xhat_ring + (int64_t)((int)ctx->ring_rounds % (tau + 1)) * ctx->cfg.d, as_stream(st));
    } else if (adaptive) {
        cudaMemsetAsync(ctx->bx_dev, 0, sizeof(int32_t), as_stream(st));
    }
    ctx->xhat_diff = ring;                                   // the workers index the ring themselves
    ctx->diff_ring = 0;
    ctx->use_slots = tau > 0;
    // sparse gradients into sparse messages: one cluster kernel takes over from the worker kernel's accumulator
    const bool msg_kernel = !flag && sparse_message_applies(ctx);
    ctx->defer_list = msg_kernel;
    // a snapshot round's gradient differences are zero, unless a worker still works on a model of the previous epoch
    const bool across = tau > 0 && ctx->cfg.delay_across_epochs;
    if (flag && across) ctx->diff_ready = true;              // (this round's slot of the ring holds the zero difference)
    rc = dq_worker_grad(ctx, ctx->codes_x, ctx->delta_x, (flag && !across) ? 1 : 0, s, round, nullptr, ctx->alpha, ctx->ninf, st);
    ctx->defer_list = false;
    ctx->use_slots = false;
    ctx->diff_ready = ctx->alpha_zeroed = ctx->ninf_zeroed = false;
    if (msg_kernel && rc == DQ_OK) {
        const BitsArgs bam = {bits_down ? bits_down : ctx->bits, bits_up ? bits_up : ctx->bits + 1, ctx->msgs.nnz, flag, 1, ctx->cfg.bx, ctx->cfg.b,
                              (adaptive && !flag) ? ctx->bx_dev : nullptr};
        launch_sparse_message(ctx, round, &ctx->msgs, as_stream(st));
        ctx->sp_norms_zeroed = false;
        ctx->tile_ptr_ready = true;
        launch_master(ctx, &ctx->msgs, true, s, eta, theta, as_stream(st), (bits_down || bits_up) ? &bam : nullptr);
        ctx->tile_ptr_ready = false;
        ctx->list_ready = false; ctx->normx_zeroed = false;
        return last_error();
    }
    const BitsArgs ba = {bits_down ? bits_down : ctx->bits, bits_up ? bits_up : ctx->bits + 1, ctx->msgs.nnz, flag,
                         sparse_messages(ctx) ? 1 : 0, ctx->cfg.bx, ctx->cfg.b, (adaptive && !flag) ? ctx->bx_dev : nullptr};
    // dense messages and an averaged master: quantiser and master step share one kernel (the codes would only travel
    // to memory and back between them)
    const bool merged = rc == DQ_OK && quantize_master_applies(ctx);
    if (merged) {
        launch_quantize_master(ctx, ctx->alpha, reinterpret_cast<const uint32_t*>(ctx->ninf), round, &ctx->msgs, s, eta, theta,
                               as_stream(st), (bits_down || bits_up) ? &ba : nullptr);
        ctx->list_ready = false; ctx->normx_zeroed = false;
        return last_error();
    }
    if (rc == DQ_OK) rc = dq_quantize_sparsify_pack(ctx, ctx->alpha, ctx->ninf, round, &ctx->msgs, st);
    ctx->list_ready = false;
    if (rc != DQ_OK) { ctx->normx_zeroed = false; return rc; }
    launch_master(ctx, &ctx->msgs, sparse_messages(ctx), s, eta, theta, as_stream(st), (bits_down || bits_up) ? &ba : nullptr);
    ctx->normx_zeroed = false;
    return last_error();
}

// Captures the kernel sequence of a non-flag round into a graph whose kernels read (round, eta, theta) from
// device memory, so that the same executable graph serves every later round on the same buffers.
static int capture_round(dq_ctx* ctx, dq_state* s, uint64_t* bits_down, uint64_t* bits_up)
{
    if (ctx->graph_exec) { cudaGraphExecDestroy(ctx->graph_exec); ctx->graph_exec = nullptr; }
    if (!ctx->cap_stream && cudaStreamCreateWithFlags(&ctx->cap_stream, cudaStreamNonBlocking) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return DQ_ERR_CUDA;
    const int64_t before = ctx->launches;
    ctx->rp_active = ctx->rp_dev;
    int rc = enqueue_round(ctx, s, 0u, 0, 1.0f, 0.0f, bits_down, bits_up, ctx->cap_stream);
    ctx->rp_active = nullptr;
    ctx->graph_launches = ctx->launches - before;
    ctx->launches = before;
    cudaGraph_t graph = nullptr;
    if (cudaStreamEndCapture(ctx->cap_stream, &graph) != cudaSuccess || !graph) rc = DQ_ERR_CUDA;
    if (rc == DQ_OK && cudaGraphInstantiate(&ctx->graph_exec, graph, 0) != cudaSuccess) rc = DQ_ERR_CUDA;
    if (graph) cudaGraphDestroy(graph);
    if (rc != DQ_OK) { cudaGetLastError(); ctx->graph_exec = nullptr; return rc; }
    ctx->graph_state = *s; ctx->graph_bits[0] = bits_down; ctx->graph_bits[1] = bits_up;
    return DQ_OK;
}

int dq_round(dq_ctx* ctx, dq_state* s, uint32_t round, float eta, float theta, uint64_t* bits_down, uint64_t* bits_up,
             void* stream)
{
    if (!ctx || !ctx->has_data) return DQ_ERR_ARG;
    int rc = check_state(ctx, s);
    if (rc != DQ_OK) return rc;
    if (!s->x_snap || !s->z_snap) return DQ_ERR_ARG;
    if (!(eta > 0.0f) || !isfinite(eta)) return DQ_ERR_ARG;
    if (ctx->epoch < 0) return DQ_ERR_ARG;                     // dq_epoch_begin has not run
    const dq_config& c = ctx->cfg;
    const int flag = c.snapshot_flag && ctx->rounds_in_epoch == 0 && (!c.accelerated || ctx->epoch == 0);
    if (!flag && ctx->cluster_blocks > 0) {                  // small problem: the whole round in one cluster kernel
        launch_round_cluster(ctx, s, round, 1, eta, theta, bits_down, bits_up, as_stream(stream));
        ctx->rounds_in_epoch += 1; ctx->ring_rounds += 1;
        ctx->ticks_in_epoch += 1;
        return last_error();
    }
    bool replayed = false;
    if (!flag && !ctx->graph_off && !c.no_graph && !(c.max_delay > 0 && c.delay_across_epochs)) {
        const dq_state& g = ctx->graph_state;
        const bool same = ctx->graph_exec && g.x == s->x && g.x_snap == s->x_snap && g.g_full == s->g_full && g.y == s->y &&
                          g.x_sum == s->x_sum && g.norm_x == s->norm_x && g.z_snap == s->z_snap &&
                          ctx->graph_bits[0] == bits_down && ctx->graph_bits[1] == bits_up;
        if (!same && capture_round(ctx, s, bits_down, bits_up) != DQ_OK) ctx->graph_off = true;   // fall back to direct launches
        if (!ctx->graph_off) {
            cudaStream_t st = as_stream(stream);
            // the round's last kernel advances the round number on the device: only a jump in the numbering or new
            // step sizes need the launch that sets them (scalars travel as kernel arguments: no host buffer to keep alive)
            const uint32_t t_epoch = (uint32_t)ctx->ring_rounds;
            if (!(ctx->rp_host_valid && ctx->rp_host.round == round && ctx->rp_host.eta == eta && ctx->rp_host.theta == theta &&
                  ctx->rp_host.t_epoch == t_epoch))
                launch_set_round_params(ctx, round, eta, theta, t_epoch, st);
            if (cudaGraphLaunch(ctx->graph_exec, st) != cudaSuccess) return DQ_ERR_CUDA;
            ctx->rp_host = dq::RoundParams{round + 1u, eta, theta, 0u, t_epoch + 1u, {0u, 0u, 0u}}; ctx->rp_host_valid = true;
            ctx->launches += ctx->graph_launches;
            replayed = true;
        }
    }
    if (!replayed) {
        rc = enqueue_round(ctx, s, round, flag, eta, theta, bits_down, bits_up, stream);
        if (rc != DQ_OK) return rc;
    }
    ctx->rounds_in_epoch += 1; ctx->ring_rounds += 1;
    ctx->ticks_in_epoch += ctx->cfg.sequential ? ctx->cfg.M : 1;
    return last_error();
}

int dq_set_delays(dq_ctx* ctx, const int32_t* delays)
{
    if (!ctx || !ctx->has_data || ctx->cfg.max_delay <= 0) return DQ_ERR_ARG;
    const int M = ctx->cfg.M;
    if (!delays) return cudaMemset(ctx->delays_dev, 0, sizeof(int32_t) * M) == cudaSuccess ? DQ_OK : DQ_ERR_CUDA;
    for (int w = 0; w < M; ++w) if (delays[w] < 0 || delays[w] > ctx->cfg.max_delay) return DQ_ERR_ARG;
    return cudaMemcpy(ctx->delays_dev, delays, sizeof(int32_t) * M, cudaMemcpyHostToDevice) == cudaSuccess ? DQ_OK : DQ_ERR_CUDA;
}

int dq_rounds(dq_ctx* ctx, dq_state* s, uint32_t round0, int32_t nrounds, float eta, float theta, uint64_t* bits_down,
              uint64_t* bits_up, void* stream)
{
    if (!ctx || nrounds < 0) return DQ_ERR_ARG;
    int32_t i = 0;
    while (i < nrounds) {
        const dq_config& c = ctx->cfg;
        const bool flag = c.snapshot_flag && ctx->rounds_in_epoch == 0 && (!c.accelerated || ctx->epoch == 0);
        if (flag || ctx->cluster_blocks == 0) {                // one round by the general path (it checks the arguments)
            const int rc = dq_round(ctx, s, round0 + (uint32_t)i, eta, theta, bits_down, bits_up, stream);
            if (rc != DQ_OK) return rc;
            i += 1;
            continue;
        }
        int rc = check_state(ctx, s);
        if (rc != DQ_OK) return rc;
        if (!ctx->has_data || !s->x_snap || !s->z_snap || !(eta > 0.0f) || !isfinite(eta) || ctx->epoch < 0) return DQ_ERR_ARG;
        launch_round_cluster(ctx, s, round0 + (uint32_t)i, nrounds - i, eta, theta, bits_down, bits_up, as_stream(stream));
        ctx->rounds_in_epoch += nrounds - i; ctx->ring_rounds += nrounds - i;
        ctx->ticks_in_epoch += nrounds - i;
        i = nrounds;
    }
    return last_error();
}

int dq_select_model_bits(dq_ctx* ctx, const float* x, const float* x_snap, const float* norm_x, float mu, int32_t* bits,
                         double* stats, void* stream)
{
    if (!ctx || !x || !x_snap || !bits || !(mu >= 0.0f)) return DQ_ERR_ARG;
    cudaStream_t st = as_stream(stream);
    const uint32_t* nb = reinterpret_cast<const uint32_t*>(norm_x);
    if (!nb) { launch_norm_inf(ctx, x, ctx->cfg.d, 1, ctx->xnorm_bits, st); nb = ctx->xnorm_bits; }
    // theta is folded into mu by the caller here, so the kernel is told "not accelerated"
    launch_select_bits(ctx, x, x_snap, nb, mu, 0, 0.0f, bits, stats ? stats : ctx->prec_stats, st);
    return last_error();
}

int dq_last_model_bits(dq_ctx* ctx, int32_t* bits_host, void* stream)
{
    if (!ctx || !bits_host) return DQ_ERR_ARG;
    cudaStream_t st = as_stream(stream);
    if (cudaMemcpyAsync(bits_host, ctx->bx_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DQ_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? DQ_OK : DQ_ERR_CUDA;
}

int dq_objective(dq_ctx* ctx, const float* x, double* P, void* stream)
{
    if (!ctx || !ctx->has_data || !x || !P) return DQ_ERR_ARG;
    launch_objective(ctx, x, P, as_stream(stream));
    return last_error();
}

int dq_round_buffers(dq_ctx* ctx, dq_msgs* msgs, const float** alpha, const float** norm_inf, const int32_t** batch_idx,
                     const uint8_t** codes_x, const float** delta_x)
{
    if (!ctx) return DQ_ERR_ARG;
    if (msgs) *msgs = ctx->msgs;
    if (alpha) *alpha = ctx->alpha;
    if (norm_inf) *norm_inf = ctx->ninf;
    if (batch_idx) *batch_idx = ctx->rows;
    if (codes_x) *codes_x = ctx->codes_x;
    if (delta_x) *delta_x = ctx->delta_x;
    return DQ_OK;
}

int dq_poll_status(dq_ctx* ctx, int* status, void* stream)
{
    if (!ctx || !status) return DQ_ERR_ARG;
    cudaStream_t st = as_stream(stream);
    if (cudaMemcpyAsync(status, ctx->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DQ_ERR_CUDA;
    if (*status != 0 && cudaMemsetAsync(ctx->status, 0, sizeof(int), st) != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int64_t dq_launch_count(const dq_ctx* ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
