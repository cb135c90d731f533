// Shared device helpers for the double-quantization kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "dq.h"

namespace dq {

constexpr uint32_t kMaster = 0xFFFFFFFFu;
enum : uint32_t { kStreamModel = 0, kStreamGrad = 1, kStreamMask = 2, kStreamBatch = 3 };
constexpr int kThreads = 256;
constexpr int kChunk = 2048;   // coordinates one warp owns per step of the sparsifier (32 lanes x 8 x 8)
constexpr int kStash = 128;    // staged survivors per chunk (a density of 1/16); fuller chunks are redone from the vector

// Staging area of the sparsifier (see sparsify_stage_kernel): slot c of worker w starts at entry
// (w * nchunks + c) * kStash; flags [M + 1] = some chunk of worker w (entry M: of any worker) exceeded its slot.
struct StageBufs { uint32_t* idx; float* val; uint32_t* flags; };

// The ten round keys of Philox4x32-10 depend on the seed only; the host expands them once so that the
// kernels read them from the constant bank.
struct PhiloxKeys { uint32_t k0[10]; uint32_t k1[10]; };

inline PhiloxKeys expand_keys(uint64_t seed)
{
    PhiloxKeys K;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) { K.k0[r] = a; K.k1[r] = b; a += 0x9E3779B9u; b += 0xBB67AE85u; }
    return K;
}

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and a word shuffle.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxKeys& K, uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[r];
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k1[r];
        c1 = (uint32_t)p1; c3 = (uint32_t)p0; c0 = n0; c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// 16-bit draw of coordinate lane j (0..7) of a Philox call: low / high half of word j >> 1.
__device__ __forceinline__ uint32_t half16(const uint32_t (&w)[4], int j)
{
    return (j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xFFFFu);
}

constexpr __host__ __device__ int levels(int bits) { return (1 << (bits - 1)) - 1; }

// Fixed-point stochastic rounding of one coordinate.  r = fl(v*inv + 384) lies in [256,512) where the
// fp32 spacing is 2^-15, so bits(r) is (v*inv + 128) * 2^15 plus a constant.  Doubling it and adding the
// raw 16-bit draw h = 2u + c puts floor(((v*inv + 128) * 2^15 + u) / 2^15) into byte 2 of the result;
// the constant only touches bits above byte 2.  Returns that word; byte 2 is the code plus 128.
// No clamp is needed: inv is 1/delta rounded toward zero and |v| <= ||v||_inf, so |v*inv| <= 2^(b-1)-1 and
// Section 3.1's rule (ii) (values outside the hull) cannot fire.  A caller-supplied norm below the true
// maximum breaks that premise and gives unspecified (but in-range, memory-safe) codes for the offending
// coordinates.
template <int BITS>
__device__ __forceinline__ uint32_t round_fixed(float v, float inv, uint32_t h16)
{
    return (__float_as_uint(__fmaf_rn(v, inv, 384.0f)) << 1) + h16;
}

// Packs the codes held in byte 2 of s[0..7] into BITS-bit two's complement, coordinate 0 lowest.
// (code + 128) mod 2^BITS equals the two's complement field for BITS < 8; for BITS = 8 flip bit 7.
template <int BITS>
__device__ __forceinline__ uint64_t pack8(const uint32_t (&s)[8])
{
    uint32_t a = __byte_perm(__byte_perm(s[0], s[1], 0x0062), __byte_perm(s[2], s[3], 0x0062), 0x5410);
    uint32_t b = __byte_perm(__byte_perm(s[4], s[5], 0x0062), __byte_perm(s[6], s[7], 0x0062), 0x5410);
    if (BITS == 8) return ((uint64_t)(b ^ 0x80808080u) << 32) | (uint64_t)(a ^ 0x80808080u);
    if (BITS == 4) {
        a &= 0x0F0F0F0Fu; b &= 0x0F0F0F0Fu;
        a |= a >> 4; b |= b >> 4;                       // bytes 0 and 2 now hold two codes each
        return (uint64_t)__byte_perm(a, b, 0x6420);
    }
    a &= 0x03030303u; b &= 0x03030303u;                 // BITS == 2
    a |= a >> 6; b |= b >> 6;                           // bytes 0 and 2 hold two codes in bits 0..3
    a = (a & 0xFu) | ((a >> 12) & 0xF0u);
    b = (b & 0xFu) | ((b >> 12) & 0xF0u);
    return (uint64_t)(a | (b << 8));
}

template <int BITS>
__device__ __forceinline__ void store_group(uint8_t* dst, uint64_t word)
{
    if (BITS == 8) *reinterpret_cast<uint2*>(dst) = make_uint2((uint32_t)word, (uint32_t)(word >> 32));
    else if (BITS == 4) *reinterpret_cast<uint32_t*>(dst) = (uint32_t)word;
    else *reinterpret_cast<uint16_t*>(dst) = (uint16_t)word;
}

// Sign-extended code j of a 32-bit word of packed BITS-bit codes.
template <int BITS>
__device__ __forceinline__ int code_of(uint32_t word, int j)
{
    return ((int)(word << (32 - BITS * (j + 1)))) >> (32 - BITS);
}

// Eight consecutive floats with one 256-bit read-only load (pointer 32-byte aligned).
__device__ __forceinline__ void load8(const float* p, float (&v)[8])
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
}

// Eight consecutive floats of a buffer that the same kernel also writes (no read-only path), and the store.
__device__ __forceinline__ void load8_rw(const float* p, float (&v)[8])
{
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p) : "memory");
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8])
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
}

// Eight floats starting at coordinate i0 of a row of length d, zero beyond the end; any alignment.
__device__ __forceinline__ void load8_guarded(const float* row, int64_t i0, int64_t d, float (&v)[8])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = (i0 + j < d) ? __ldg(row + i0 + j) : 0.0f;
}

__device__ __forceinline__ void set_status(int* status, int code)
{
    if (*reinterpret_cast<volatile int*>(status) == 0) atomicCAS(status, 0, code);
}

__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) { return __reduce_max_sync(0xFFFFFFFFu, v); }

// Block-wide maximum of unsigned values folded into *dst with one atomic per block.
__device__ __forceinline__ void block_atomic_max(uint32_t v, uint32_t* dst)
{
    __shared__ uint32_t s_max[kThreads / 32];
    v = warp_max_u32(v);
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        uint32_t t = (threadIdx.x < (blockDim.x >> 5)) ? s_max[threadIdx.x] : 0u;
        t = warp_max_u32(t);
        if (threadIdx.x == 0 && t != 0u) atomicMax(dst, t);
    }
}

// Programmatic dependent launch.  Every launch of the library carries the programmatic-serialization attribute and
// every kernel begins with pdl_prologue(), which waits until the kernel before it has completed and its writes are
// visible; nothing before the wait may touch global memory.  No kernel signals its dependents early
// (griddepcontrol.launch_dependents): a dependent's wait is released by that signal, not by the end of the grid, so
// whatever a kernel wrote after signalling was read stale by its successor (seen with a small scan kernel between
// two larger ones).  Without the signal the successor is released when the last block of this grid exits.
// In a kernel launched without the attribute the instruction does nothing.
__device__ __forceinline__ void pdl_prologue()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Launch with the programmatic-serialization attribute: the gap between dependent kernels (drain, then launch)
// is what bounds the small configurations, whose rounds are chains of microsecond kernels.
template <class... P, class... A>
inline cudaError_t launch_k(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args)
{
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<A&&>(args)...);
}

struct ProxParams { float lambda1, lambda2, lo, hi; };

// prox of h = lambda1 |x|_1 + (lambda2/2) |x|^2 + indicator of [lo, hi] at v with step eta: thr = eta lambda1,
// den = 1 + eta lambda2 (soft threshold, shrink, clip), and the master's update of one coordinate built on it
// (Algorithm 1 step 9; Algorithm 3 step 9 with the momentum combination).
__device__ __forceinline__ float prox_h(float v, float thr, float den, float lo, float hi)
{
    const float a = __fsub_rn(fabsf(v), thr);
    float r = (a > 0.0f) ? copysignf(a, v) : 0.0f;
    if (den != 1.0f) r = __fdiv_rn(r, den);
    return fminf(fmaxf(r, lo), hi);
}

template <bool ACC>
__device__ __forceinline__ float master_update(float acc, float inv_m, float eta, float theta, float thr, float den,
                                               const ProxParams& pp, float g_full, float x_or_y, float xsnap,
                                               float& y_out, float& xsum_io)
{
    const float u = __fadd_rn(__fmul_rn(acc, inv_m), g_full);
    const float p = prox_h(__fmaf_rn(-eta, u, x_or_y), thr, den, pp.lo, pp.hi);
    if (!ACC) return p;
    y_out = p;
    const float x = __fmaf_rn(theta, __fsub_rn(p, xsnap), xsnap);
    xsum_io = __fadd_rn(xsum_io, x);
    return x;
}

// Where the sparsifier finds its groups of eight coordinates: every group of the vector (groups == NULL), or
// an ascending list of the groups that can hold a nonzero (groups [M][cap], count [M]).
struct GroupList { const uint32_t* groups; const uint32_t* count; int64_t cap; };

// Group at position p of worker w, or -1 past the end.
__device__ __forceinline__ int64_t group_at(const GroupList& gl, int w, int64_t p, int64_t d)
{
    if (!gl.groups) return ((p << 3) < d) ? p : -1;
    return (p < (int64_t)gl.count[w]) ? (int64_t)gl.groups[(int64_t)w * gl.cap + p] : -1;
}

// Integer accumulator of the CSR worker gradients: acc [M][d], one unit = 1 / scale (scale a power of two).
struct FixedAcc { long long* acc; double scale; double inv_scale; };

// Transmitted-bit counters of a round, written by the master kernel when `down` is set (Section 3.1 message sizes).
struct BitsArgs { uint64_t* down; uint64_t* up; const uint32_t* nnz; int flag_round, sparse_msgs, bx, b;
                  const int32_t* bx_dev; /* width chosen on the device this round, overrides bx when set */ };

__device__ __forceinline__ void write_round_bits(const BitsArgs& ba, int M, int64_t d)
{
    const int bx = ba.bx_dev ? *ba.bx_dev : ba.bx;
    *ba.down = ba.flag_round ? (uint64_t)M : (uint64_t)M * (32ull + (uint64_t)bx * (uint64_t)d);
    int logd = 0; while (((int64_t)1 << logd) < d) ++logd;
    uint64_t up = 0;
    for (int w = 0; w < M; ++w)
        up += ba.sparse_msgs ? 32ull + (uint64_t)ba.nnz[w] * (uint64_t)(logd + ba.b) : 32ull + (uint64_t)ba.b * (uint64_t)d;
    *ba.up = up;
}

// Per-round scalars kept in device memory so that a captured graph of a round can be replayed unchanged.
struct RoundParams { uint32_t round; float eta; float theta; uint32_t pad; uint32_t t_epoch; uint32_t unused[3]; };   // t_epoch: rounds since the epoch began

// Last statement of the kernel that ends a replayed round: the block that finishes last advances the round number
// held on the device (no block reads it afterwards), so that consecutive rounds need no launch that sets it.
// pad counts the blocks that have finished.
__device__ __forceinline__ void finish_round(const RoundParams* rp)
{
    if (rp && threadIdx.x == 0) {
        RoundParams* p = const_cast<RoundParams*>(rp);
        __threadfence();
        if (atomicAdd(&p->pad, 1u) == gridDim.x * gridDim.y * gridDim.z - 1u) { p->pad = 0u; p->round += 1u; p->t_epoch += 1u; }
    }
}

#define DQ_DISPATCH_BITS(bits, CALL)                 \
    switch (bits) {                                  \
        case 2: { constexpr int BITS_ = 2; CALL; } break; \
        case 4: { constexpr int BITS_ = 4; CALL; } break; \
        default: { constexpr int BITS_ = 8; CALL; } break; \
    }

}  // namespace dq

// Host-side context behind the opaque dq_ctx.
struct dq_ctx {
    dq_config cfg;
    dq_data data;
    bool has_data;
    dq::PhiloxKeys keys;
    int sm_count;
    // scratch owned by the context
    uint32_t* norm_bits;        // [M]   ||v_w||_inf bit patterns when the caller supplies none
    uint32_t* norm_block;       // owner of ninf, beta_norm_bits and l1_sum (contiguous)
    bool sp_norms_zeroed;       // an earlier kernel of this round already cleared beta_norm_bits and l1_sum
    uint32_t* beta_norm_bits;   // [M]   ||beta_w||_inf over survivors
    unsigned long long* l1_sum; // [M]   fixed-point ||alpha_w||_1
    uint32_t* chunk_off;        // [M][nchunks + 1] survivors per chunk, then their exclusive prefix
    uint32_t* tile_ptr;         // [M][nchunks + 1] first list entry of each coordinate tile (sparse master)
    // survivors staged by the sparsifier's mask pass, so that no later pass re-reads the vector
    uint32_t* stage_idx;        // [M][nchunks][kStash] coordinates of the staged survivors of each chunk, ascending
    float* stage_val;           // [M][nchunks][kStash] their rescaled values beta_i
    uint32_t* stage_ctrl;       // [M + 1] fallback flags (per worker, any)
    uint32_t* xnorm_bits;       // [1]   ||x||_inf when the caller supplies none
    int* status;                // sticky device status word
    int64_t nchunks;
    // buffers of dq_round / dq_codec_round
    float* alpha;               // [M][d]
    float* ninf;                // [M]
    int32_t* rows;              // [M][B]
    uint8_t* codes_x;           // packed model
    float* delta_x;
    float* xhat_diff;           // [d] dequantised model minus snapshot
    double* g64;                // [d] full-gradient accumulator
    long long* acc64;           // [M][d] CSR data: integer accumulator of the worker gradients, all-zero between rounds
    double acc_scale, acc_inv;  // its grid: one unit is 2^-shift, shift from max |a_ij| so that a minibatch sum cannot overflow
    float* rbuf;                // [M][B] slope differences of the sampled rows
    float* fused_part;          // [SMs + M][d] column sums per (block, worker) of the one-pass dense gradient kernel; NULL: not in use
    uint32_t* fused_cnt;        // [M] blocks that have handed in their sums for a worker (zero between launches)
    uint32_t* fused_done;       // [1] workers whose message is complete, when the kernel carries the whole round
    int32_t* bx_dev;            // model width chosen by condition (3) this round
    // network workload: sampled-row indices and per-row activations / derivatives of the two parameter vectors
    int32_t* mlp_rows; double* mlp_act[2]; float* mlp_dz[2]; float* mlp_dh[2];
    double* prec_stats;         // [4] expected errors at 2/4/8 bits and ||x - xsnap||^2
    dq_msgs msgs;
    uint64_t* bits;             // [2] device counters
    // device-resident state for the host-buffer entry point
    float *hx, *hg, *hv, *hnorm;
    // replay of whole rounds: per-round scalars on the device and the captured graph of a non-flag round
    dq::RoundParams* rp_dev;
    const dq::RoundParams* rp_active;   // non-null while a round is being captured
    dq::RoundParams rp_host; bool rp_host_valid;   // what rp_dev holds once the work enqueued so far has run
    cudaStream_t cap_stream;
    cudaGraphExec_t graph_exec;
    dq_state graph_state;
    uint64_t* graph_bits[2];
    int64_t graph_launches;
    bool graph_off;
    // sparse gradients (CSR data, sparse messages): bitmap of touched groups, their ascending list, its length
    uint32_t* touched; uint32_t* glist; uint32_t* gcount; uint32_t* seg_count; int64_t bm_words; int64_t glist_cap;
    // delayed workers: xhat_diff is a ring of max_delay + 1 vectors (slot = round in epoch mod ring size)
    int32_t* delays_dev;        // [M] rounds each worker lags behind
    int32_t* slots_dev;         // [M] ring slot each worker reads this round
    bool use_slots;             // set while dq_round enqueues a round of a context with max_delay > 0
    float* xhat_ring;           // delays across epochs (logistic model): the broadcasts themselves, [max_delay + 1][d], from which the ring of
                                // differences is formed again when the snapshot changes
    int64_t ring_rounds;        // rounds the ring has seen (since the epoch began, or since the first epoch with delays across epochs)
    int diff_ring;              // set while such a round is captured: slots of the ring, the kernels pick this round's from the device's round counter
    int cluster_blocks;         // blocks of the one-cluster round kernel for small problems; 0: rounds run as separate kernels
    bool list_mode;             // dq_round keeps alpha zero outside the listed groups and works on the list only
    bool list_ready;            // the list of this round has been built (consumed by the sparsifier launch)
    bool msg_cluster;           // sparse gradients become sparse messages in one cluster kernel (sparse_message_kernel)
    bool defer_list;            // set while dq_round enqueues such a round: the worker kernel leaves list, alpha and norm to it
    bool tile_ptr_ready;        // set while dq_round enqueues such a round: the master's tile pointers are already written
    uint32_t* ptouched;         // [M][bm_words] the previous round's bitmap (the groups of alpha that are not zero)
    uint32_t* gtmp;             // [M][glist_cap] per-block scratch lists of that kernel
    bool alpha_zeroed, ninf_zeroed, normx_zeroed;   // an earlier kernel of this round already cleared these
    bool diff_ready;            // the model-quantise kernel of this round already wrote xhat - xsnap
    // bookkeeping
    int64_t launches;
    int64_t rounds_in_epoch;
    int64_t ticks_in_epoch;     // master steps since the epoch began (M per round in sequential mode)
    int64_t epoch;
};
