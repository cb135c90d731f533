// Host-side launchers shared between the translation units of libdq.
#pragma once
#include "dq_common.cuh"

namespace dq {

// codec (dq_codec.cu)
void launch_norm_inf(dq_ctx* ctx, const float* v, int64_t d, int M, uint32_t* norm_bits, cudaStream_t st);
void launch_quantize_pack(dq_ctx* ctx, const float* v, int64_t d, int M, int bits, const uint32_t* norm_bits,
                          uint8_t* codes, int64_t stride, float* scale, uint32_t round, uint32_t worker_base,
                          uint32_t stream_id, cudaStream_t st, const float* ref = nullptr, float* diff = nullptr,
                          float* zero_f = nullptr, int64_t zero_n = 0, uint32_t* zero_u = nullptr, int zero_un = 0,
                          const int32_t* bits_gate = nullptr);
void launch_select_bits(dq_ctx* ctx, const float* x, const float* xsnap, const uint32_t* norm_bits, float mu, int accelerated,
                        float theta, int32_t* bits, double* stats, cudaStream_t st);
void launch_sparsify_pack(dq_ctx* ctx, const float* v, int64_t d, int M, int bits, const uint32_t* norm_bits,
                          uint32_t round, const dq_msgs* out, bool sparse_out, cudaStream_t st);
void launch_dequant_diff_any(dq_ctx* ctx, const uint8_t* codes, const float* delta_x, const float* ref, float* diff, int bits, cudaStream_t st);
void launch_clear_listed(dq_ctx* ctx, cudaStream_t st);
void launch_build_group_list(dq_ctx* ctx, uint32_t* norm_bits, cudaStream_t st);
void launch_master(dq_ctx* ctx, const dq_msgs* msgs, bool sparse_msgs, dq_state* s, float eta, float theta, cudaStream_t st,
                   const BitsArgs* bits = nullptr);
bool quantize_master_applies(const dq_ctx* ctx);
void launch_quantize_master(dq_ctx* ctx, const float* v, const uint32_t* norm_bits, uint32_t round, const dq_msgs* msgs, dq_state* s,
                            float eta, float theta, cudaStream_t st, const BitsArgs* bits = nullptr);
void launch_unpack(dq_ctx* ctx, const dq_msgs* msgs, bool sparse_msgs, int w, float* out, cudaStream_t st);

// gradients (dq_grad.cu)
void launch_epoch_begin(dq_ctx* ctx, dq_state* s, float theta, cudaStream_t st);
void launch_worker_grad(dq_ctx* ctx, const uint8_t* codes_x, const float* delta_x, int is_snapshot, const dq_state* s,
                        uint32_t round, const int32_t* batch_idx, float* alpha, float* norm_inf, cudaStream_t st);
bool worker_accumulates(const dq_ctx* ctx);
int fused_grad_setup(dq_ctx* ctx);
void sparse_message_setup(dq_ctx* ctx);
bool sparse_message_applies(const dq_ctx* ctx);
void launch_sparse_message(dq_ctx* ctx, uint32_t round, const dq_msgs* out, cudaStream_t st);
bool fused_grad_applies(const dq_ctx* ctx);
bool fused_round_applies(const dq_ctx* ctx);
void launch_fused_round(dq_ctx* ctx, dq_state* s, uint32_t round, cudaStream_t st);
void small_round_setup(dq_ctx* ctx);
void launch_set_slots(dq_ctx* ctx, int round_in_epoch, cudaStream_t st);
void launch_rediff_ring(dq_ctx* ctx, const float* x_snap, cudaStream_t st);
void launch_dequant_xhat(dq_ctx* ctx, const uint8_t* codes_x, const float* delta_x, float* xhat, cudaStream_t st);
void launch_round_cluster(dq_ctx* ctx, dq_state* s, uint32_t round0, int nrounds, float eta, float theta, uint64_t* bits_down,
                          uint64_t* bits_up, cudaStream_t st);
void launch_objective(dq_ctx* ctx, const float* x, double* P, cudaStream_t st);
void launch_set_round_params(dq_ctx* ctx, uint32_t round, float eta, float theta, uint32_t t_epoch, cudaStream_t st);

}  // namespace dq
