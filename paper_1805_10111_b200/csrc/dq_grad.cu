// Gradient kernels: the worker's variance-reduced minibatch gradient (Algorithm 1 step 11), the epoch's
// full gradient (step 5), the epoch-boundary state update (steps 3/14, Algorithm 3 steps 3/15), the
// objective of eq. (1).  f_a(x) = log(1 + exp(-y_a <a_a, x>)).
#include <cuda_bf16.h>
#include <type_traits>

#include "dq_common.cuh"
#include "dq_kernels.cuh"

namespace dq {

constexpr int kRowsPerBlock = 16;   // rows of one worker handled by one block of the dense kernels

__device__ __forceinline__ float sigmoidf_(float t) { return __fdiv_rn(1.0f, 1.0f + expf(-t)); }

// slope(z) = d/dz log(1+exp(-y z)) = -y sigma(-y z).  The worker needs slope(zs + dz) - slope(zs)
// = y (sigma(-u) - sigma(-(u+t))) with u = y zs, t = y dz.  Written as y sigma(-(u+t)) sigma(u) expm1(t) it has no
// cancellation when dz is small.  Outside the range where every factor of that product is an ordinary fp32 number:
//   t > 16: the two sigmoids differ by a factor of exp(16) or more, so their plain difference is accurate; it is taken
//           on the side where both are small (sigma(-a) = 1 - sigma(a)), so nothing is lost against a value near 1;
//   0 < t <= 16 and u + t > 80: sigma(-(u+t)) would underflow; sigma(-(u+t)) expm1(t) = -expm1(-t) / (exp(-t) + exp(u))
//           keeps every factor finite (an infinite exp(u) gives the correct limit 0).
__device__ __forceinline__ float slope_difference(float y, float zs, float dz)
{
    const float t = y * dz, u = y * zs;
    if (t > 16.0f)
        return y * (u + 0.5f * t >= 0.0f ? sigmoidf_(-u) - sigmoidf_(-(u + t)) : sigmoidf_(u + t) - sigmoidf_(u));
    if (t > 0.0f && u + t > 80.0f) return y * sigmoidf_(u) * __fdiv_rn(-expm1f(-t), expf(-t) + expf(u));
    return y * sigmoidf_(-y * (zs + dz)) * sigmoidf_(u) * expm1f(t);
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// <a_row, vec> for one dense row, computed by one warp (fp32 partial sums per lane, double across lanes).
template <class T>
__device__ __forceinline__ double warp_dot_dense(const T* __restrict__ row, const float* __restrict__ vec, int64_t d, int lane)
{
    float s0 = 0.0f, s1 = 0.0f;
    int64_t i = lane;
    for (; i + 32 < d; i += 64) { s0 = fmaf(to_float(row[i]), vec[i], s0); s1 = fmaf(to_float(row[i + 32]), vec[i + 32], s1); }
    if (i < d) s0 = fmaf(to_float(row[i]), vec[i], s0);
    return warp_sum((double)s0 + (double)s1);
}

__device__ __forceinline__ double warp_dot_csr(const float* __restrict__ val, const int32_t* __restrict__ col, int64_t k0, int64_t k1,
                                                const float* __restrict__ vec, int lane)
{
    double s = 0.0;
    for (int64_t k = k0 + lane; k < k1; k += 32) s += (double)__ldg(val + k) * (double)__ldg(vec + __ldg(col + k));
    return warp_sum(s);
}

// ---------------------------------------------------------------------------------------------------
// Minibatch rows: worker w draws slot j from its partition [floor(w n/M), floor((w+1) n/M)) with word
// (j & 3) of Philox counter (j >> 2, round, w, batch stream).
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ int64_t sample_row(const PhiloxKeys& K, uint32_t round, int w, int j, int M, int64_t n)
{
    const int64_t lo = ((int64_t)w * n) / M, hi = ((int64_t)(w + 1) * n) / M;
    uint32_t r[4];
    philox4x32_10((uint32_t)(j >> 2), round, (uint32_t)w, kStreamBatch, K, r);
    const uint32_t word = (j & 3) == 0 ? r[0] : (j & 3) == 1 ? r[1] : (j & 3) == 2 ? r[2] : r[3];
    return lo + (int64_t)(((uint64_t)word * (uint64_t)(hi - lo)) >> 32);
}

// Where a worker's minibatch comes from: explicit indices, or the batch stream (then also recorded in rows_out).
struct BatchSource {
    const int32_t* rows_in; int32_t* rows_out; uint32_t round; const RoundParams* rp; int M; int64_t n;
    uint32_t* zero_word;   // cleared by the first thread of the grid (the next stage's maximum), may be NULL
    const int32_t* diff_slot; int64_t diff_stride;   // delayed workers: worker w reads xhat - xsnap at slot diff_slot[w]; NULL: slot 0
};

// xhat - xsnap as worker w sees it (the current broadcast, or an earlier one of the epoch when the worker lags).
__device__ __forceinline__ const float* diff_of_worker(const BatchSource& bs, const float* diff, int w)
{
    return bs.diff_slot ? diff + (int64_t)bs.diff_slot[w] * bs.diff_stride : diff;
}

__device__ __forceinline__ void clear_word(const BatchSource& bs)
{
    if (bs.zero_word && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *bs.zero_word = 0u;
}

__device__ __forceinline__ int64_t batch_row(const BatchSource& bs, const PhiloxKeys& K, int w, int j, int B, bool writer)
{
    const int64_t slot = (int64_t)w * B + j;
    if (bs.rows_in) return bs.rows_in[slot];
    const int64_t a = sample_row(K, bs.rp ? bs.rp->round : bs.round, w, j, bs.M, bs.n);
    if (writer && bs.rows_out) bs.rows_out[slot] = (int32_t)a;
    return a;
}

// xhat - xsnap with xhat_i = code_i * delta_x (the transmitted low-precision model).
template <int BITS>
__global__ void dequant_diff_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ delta_x,
                                    const float* __restrict__ xsnap, int64_t d, float* __restrict__ diff)
{
    pdl_prologue();
    const float dl = *delta_x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t bit = i * BITS;
        const int k = code_of<BITS>(reinterpret_cast<const uint32_t*>(codes)[bit >> 5], (int)((bit & 31) / BITS));
        diff[i] = __fsub_rn(__fmul_rn((float)k, dl), xsnap ? xsnap[i] : 0.0f);
    }
}

// ---------------------------------------------------------------------------------------------------
// CSR worker gradient: one warp per sampled row.  dz = <a, xhat - xsnap>, slope difference, then the
// row is scattered into the worker's accumulator.  The scatter meets other rows of the minibatch in any order,
// so the accumulator is an integer grid on which addition is exact: every term r_a a_ai (the product is exact in
// double) is rounded once to a multiple of 2^-shift and added as a 64-bit integer.  shift is chosen by the host
// from max |a_ai| so that the sum of a minibatch cannot overflow (|r_a| <= 1/B).  Equal inputs therefore give
// equal bits whatever the order of the atomics; acc_to_alpha_kernel / build_group_list_kernel turn the integers
// into alpha_w (one rounding to fp32) and put the zeros back.  acc must be zero on entry.
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ void fixed_add(long long* dst, float r, float a, double scale)
{
    atomicAdd(reinterpret_cast<unsigned long long*>(dst), (unsigned long long)__double2ll_rn((double)r * (double)a * scale));
}

__global__ void __launch_bounds__(kThreads)
worker_grad_csr_kernel(const float* __restrict__ val, const int32_t* __restrict__ col, const int64_t* __restrict__ row_ptr,
                       const float* __restrict__ labels, const float* __restrict__ diff, const float* __restrict__ z_snap,
                       const __grid_constant__ PhiloxKeys K, BatchSource bs, int M, int B, int64_t d, FixedAcc fa,
                       uint32_t* __restrict__ touched /* bitmap of groups of eight coordinates, may be NULL */, int64_t bm_words)
{
    pdl_prologue();
    clear_word(bs);
    const int lane = threadIdx.x & 31;
    const int64_t slot = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (slot >= (int64_t)M * B) return;
    const int w = (int)(slot / B);
    const int64_t a = batch_row(bs, K, w, (int)(slot % B), B, lane == 0);
    const int64_t k0 = row_ptr[a], k1 = row_ptr[a + 1];
    const float dz = (float)warp_dot_csr(val, col, k0, k1, diff_of_worker(bs, diff, w), lane);
    const float r = slope_difference(labels[a], z_snap[a], dz) / (float)B;
    long long* out = fa.acc + (int64_t)w * d;
    uint32_t* bm = touched ? touched + (int64_t)w * bm_words : nullptr;
    for (int64_t k = k0 + lane; k < k1; k += 32) {
        const int32_t c = __ldg(col + k);
        fixed_add(out + c, r, __ldg(val + k), fa.scale);
        if (bm) {
            const uint32_t bit = 1u << ((c >> 3) & 31);
            uint32_t* word = bm + (c >> 8);
            if (!(*reinterpret_cast<volatile uint32_t*>(word) & bit)) atomicOr(word, bit);
        }
    }
}

// alpha_w = the accumulated integers scaled back (one rounding to fp32), ||alpha_w||_inf, and the accumulator is
// left all-zero for the next round.  grid (blocks, M); norm_bits must be zero on entry.
__global__ void __launch_bounds__(kThreads)
acc_to_alpha_kernel(FixedAcc fa, int64_t d, float* __restrict__ alpha, uint32_t* __restrict__ norm_bits)
{
    pdl_prologue();
    const int w = blockIdx.y;
    long long* acc = fa.acc + (int64_t)w * d;
    float* out = alpha + (int64_t)w * d;
    uint32_t nmax = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
        const long long q = acc[i];
        if (q != 0) acc[i] = 0;
        const float a = (float)((double)q * fa.inv_scale);
        out[i] = a;
        nmax = max(nmax, __float_as_uint(a) & 0x7FFFFFFFu);
    }
    block_atomic_max(nmax, norm_bits + w);
}

// ---------------------------------------------------------------------------------------------------
// Dense worker gradient (fp32 or bf16 features) for small minibatches and for rows off the 16-byte grid.
// grid (1, M): one block per worker takes the minibatch in chunks of kRowsPerBlock rows.  Phase A: one warp
// per row computes the slope difference; phase B: threads own columns and add the chunk's rows in slot order,
// so alpha_w is the same bit pattern on every run (no atomics).
// ---------------------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(kThreads)
worker_grad_dense_kernel(const T* __restrict__ X, const float* __restrict__ labels, const float* __restrict__ diff,
                         const float* __restrict__ z_snap, const __grid_constant__ PhiloxKeys K, BatchSource bs, int B, int64_t d,
                         float* __restrict__ alpha)
{
    pdl_prologue();
    __shared__ float s_r[kRowsPerBlock];
    __shared__ int64_t s_row[kRowsPerBlock];
    clear_word(bs);
    const int w = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* out = alpha + (int64_t)w * d;
    for (int j0 = 0; j0 < B; j0 += kRowsPerBlock) {
        const int nrows = min(kRowsPerBlock, B - j0);
        for (int j = warp; j < nrows; j += kThreads / 32) {
            const int64_t a = batch_row(bs, K, w, j0 + j, B, lane == 0);
            const float dz = (float)warp_dot_dense(X + a * d, diff_of_worker(bs, diff, w), d, lane);
            if (lane == 0) { s_r[j] = slope_difference(labels[a], z_snap[a], dz) / (float)B; s_row[j] = a; }
        }
        __syncthreads();
        for (int64_t i = threadIdx.x; i < d; i += blockDim.x) {
            float s = j0 == 0 ? 0.0f : out[i];                   // the same thread wrote it one chunk ago
            for (int j = 0; j < nrows; ++j) s = fmaf(s_r[j], to_float(X[s_row[j] * d + i]), s);
            out[i] = s;
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------------
// 16-byte vector access to a row of features: 4 floats or 8 bfloat16 per load.
// ---------------------------------------------------------------------------------------------------
template <class T> struct RowVec;
template <> struct RowVec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void unpack(const uint4& u, float (&f)[4])
    { f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w); }
};
template <> struct RowVec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void unpack(const uint4& u, float (&f)[8])
    {   // a bfloat16 is the upper half of an fp32
        f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xFFFF0000u);
        f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xFFFF0000u);
        f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xFFFF0000u);
        f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xFFFF0000u);
    }
};

// <a_row, vec> by one warp with 16-byte loads (d a multiple of the vector width, row 16-byte aligned).
template <class T>
__device__ __forceinline__ double warp_dot_dense_vec(const T* __restrict__ row, const float* __restrict__ vec, int64_t d, int lane)
{
    constexpr int N = RowVec<T>::N;
    const uint4* rv = reinterpret_cast<const uint4*>(row);
    const float4* vv = reinterpret_cast<const float4*>(vec);
    const int nv = (int)(d / N);
    float s[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll 4
    for (int v = lane; v < nv; v += 32) {
        float f[N];
        RowVec<T>::unpack(__ldg(rv + v), f);
#pragma unroll
        for (int q = 0; q < N / 4; ++q) {
            const float4 x4 = __ldg(vv + v * (N / 4) + q);
            s[0] = fmaf(f[q * 4 + 0], x4.x, s[0]); s[1] = fmaf(f[q * 4 + 1], x4.y, s[1]);
            s[2] = fmaf(f[q * 4 + 2], x4.z, s[2]); s[3] = fmaf(f[q * 4 + 3], x4.w, s[3]);
        }
    }
    return warp_sum(((double)s[0] + (double)s[1]) + ((double)s[2] + (double)s[3]));
}

// Vectorised dense worker gradient: same plan as worker_grad_dense_kernel with 16-byte loads and stores
// (d a multiple of the vector width).  The rows read in phase A are read again in phase B while they are
// still in L2.
template <class T>
__global__ void __launch_bounds__(kThreads)
worker_grad_dense_vec_kernel(const T* __restrict__ X, const float* __restrict__ labels, const float* __restrict__ diff,
                             const float* __restrict__ z_snap, const __grid_constant__ PhiloxKeys K, BatchSource bs, int B, int64_t d,
                             float* __restrict__ alpha)
{
    pdl_prologue();
    constexpr int N = RowVec<T>::N;
    __shared__ float s_r[kRowsPerBlock];
    __shared__ const uint4* s_rowp[kRowsPerBlock];
    clear_word(bs);
    const int w = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nv = (int)(d / N);
    float* out = alpha + (int64_t)w * d;
    for (int j0 = 0; j0 < B; j0 += kRowsPerBlock) {
        const int nrows = min(kRowsPerBlock, B - j0);
        for (int j = warp; j < nrows; j += kThreads / 32) {
            const int64_t a = batch_row(bs, K, w, j0 + j, B, lane == 0);
            const float dz = (float)warp_dot_dense_vec(X + a * d, diff_of_worker(bs, diff, w), d, lane);
            if (lane == 0) { s_r[j] = slope_difference(labels[a], z_snap[a], dz) / (float)B; s_rowp[j] = reinterpret_cast<const uint4*>(X + a * d); }
        }
        __syncthreads();
        for (int v = threadIdx.x; v < nv; v += blockDim.x) {
            float acc[N];
            float4* o4 = reinterpret_cast<float4*>(out + (int64_t)v * N);
#pragma unroll
            for (int q = 0; q < N / 4; ++q) {                     // the same thread wrote it one chunk ago
                const float4 prev = j0 == 0 ? make_float4(0.0f, 0.0f, 0.0f, 0.0f) : o4[q];
                acc[q * 4] = prev.x; acc[q * 4 + 1] = prev.y; acc[q * 4 + 2] = prev.z; acc[q * 4 + 3] = prev.w;
            }
#pragma unroll 4
            for (int j = 0; j < nrows; ++j) {
                float f[N];
                RowVec<T>::unpack(__ldg(s_rowp[j] + v), f);
                const float r = s_r[j];
#pragma unroll
                for (int q = 0; q < N; ++q) acc[q] = fmaf(r, f[q], acc[q]);
            }
#pragma unroll
            for (int q = 0; q < N / 4; ++q) o4[q] = make_float4(acc[q * 4], acc[q * 4 + 1], acc[q * 4 + 2], acc[q * 4 + 3]);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------------
// Dense worker gradient for large minibatches, in two kernels and without atomics:
//   worker_margins_kernel   one warp per sampled row: slope difference r_{w,j} / B
//   worker_colsum_kernel    block (column slab, worker): alpha_w[slab] = sum_j r_{w,j} a_j[slab], rows split over
//                           the warps and combined in a fixed order, so alpha is reproducible bit for bit;
//                           also folds ||alpha_w||_inf.  The rows were just read by the first kernel and are
//                           served from L2.
// ---------------------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(kThreads, 8)     // one wave: M B / 8 blocks must all be resident (a second, thin wave doubles the time)
worker_margins_kernel(const T* __restrict__ X, const float* __restrict__ labels, const float* __restrict__ diff,
                      const float* __restrict__ z_snap, const __grid_constant__ PhiloxKeys K, BatchSource bs, int M, int B, int64_t d,
                      float* __restrict__ rbuf)
{
    pdl_prologue();
    clear_word(bs);
    const int lane = threadIdx.x & 31;
    const int64_t slot = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (slot >= (int64_t)M * B) return;
    const int w = (int)(slot / B), j = (int)(slot % B);
    const int64_t a = batch_row(bs, K, w, j, B, lane == 0);
    const float dz = (float)warp_dot_dense_vec(X + a * d, diff_of_worker(bs, diff, w), d, lane);
    if (lane == 0) rbuf[slot] = slope_difference(labels[a], z_snap[a], dz) / (float)B;
}

template <class T>
__global__ void __launch_bounds__(kThreads)
worker_colsum_kernel(const T* __restrict__ X, const int32_t* __restrict__ rows, const float* __restrict__ rbuf, int B, int64_t d,
                     float* __restrict__ alpha, uint32_t* __restrict__ norm_bits)
{
    pdl_prologue();
    constexpr int N = RowVec<T>::N;
    constexpr int kWarps = kThreads / 32;
    __shared__ float s_part[kWarps][32 * N];
    extern __shared__ float s_r[];                 // [B] slope differences, then [B] row indices as int32
    int32_t* s_row = reinterpret_cast<int32_t*>(s_r + B);
    const int w = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int j = threadIdx.x; j < B; j += blockDim.x) { s_r[j] = rbuf[(int64_t)w * B + j]; s_row[j] = rows[(int64_t)w * B + j]; }
    __syncthreads();
    const int nv = (int)(d / N);
    const int v = blockIdx.x * 32 + lane;          // this lane's 16-byte column group
    float acc[N];
#pragma unroll
    for (int q = 0; q < N; ++q) acc[q] = 0.0f;
    if (v < nv) {
        constexpr int U = 8;                       // row slabs in flight per lane; rows are taken in the same order as a plain loop
        for (int j0 = warp; j0 < B; j0 += kWarps * U) {
            uint4 q4[U]; float r[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int j = j0 + u * kWarps;
                const bool in = j < B;
                q4[u] = in ? __ldg(reinterpret_cast<const uint4*>(X + (int64_t)s_row[j] * d) + v) : make_uint4(0u, 0u, 0u, 0u);
                r[u] = in ? s_r[j] : 0.0f;
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (j0 + u * kWarps < B) {
                    float f[N];
                    RowVec<T>::unpack(q4[u], f);
#pragma unroll
                    for (int q = 0; q < N; ++q) acc[q] = fmaf(r[u], f[q], acc[q]);
                }
            }
        }
    }
#pragma unroll
    for (int q = 0; q < N; ++q) s_part[warp][lane * N + q] = acc[q];
    __syncthreads();
    uint32_t nmax = 0;
    for (int c = threadIdx.x; c < 32 * N; c += blockDim.x) {
        const int64_t i = (int64_t)blockIdx.x * 32 * N + c;
        if (i < d) {
            float sum = 0.0f;
#pragma unroll
            for (int k = 0; k < kWarps; ++k) sum += s_part[k][c];
            alpha[(int64_t)w * d + i] = sum;
            nmax = max(nmax, __float_as_uint(sum) & 0x7FFFFFFFu);
        }
    }
    block_atomic_max(nmax, norm_bits + w);
}

// ---------------------------------------------------------------------------------------------------
// Dense worker gradient in ONE pass over the sampled rows (Algorithm 1 step 11 for large minibatches).
// alpha_w = sum_j r_j a_j needs r_j = slope difference of row j, which needs the whole row's margin: a two-kernel
// plan reads every row twice.  Here a row is staged on chip once and used for both.
//
//   tiles      a tile is kFusedRows consecutive minibatch slots of one worker; the M * ceil(B / 8) tiles are split
//              into contiguous runs, one run per block (one block per SM)
//   staging    the load warp draws the tile's row indices and issues one bulk asynchronous copy per row into a ring
//              of kFusedStages shared-memory stages; an mbarrier per stage counts the bytes, a second one counts the
//              compute warps that have taken their groups out of the stage (then it is refilled)
//   margins    compute thread v owns the 16-byte column group v of every row: it keeps the tile's eight groups in
//              registers, forms eight partial dot products with its slice of xhat - xsnap, the warp folds them in a
//              fixed butterfly, and the slope warp adds the warps' partial sums in warp order (double) and turns the
//              eight margins into slope differences
//   columns    one tile later the compute threads add r_j * row_j to their columns from the registers they kept;
//              warps hand over through mbarriers (partials ready / slopes ready), so nobody waits for the slope warp
//              unless it falls a whole tile behind
//   combine    a block's column sums for a worker go to a scratch slot; the block that completes a worker (a
//              counter tells it; nobody waits) adds that worker's slots in block order, writes alpha_w and
//              ||alpha_w||_inf.  The order of every sum is fixed, so alpha is reproducible bit for bit.
// The only waits are on the stage barriers; each is bounded, after which the block records DQ_ERR_TIMEOUT, waits
// (bounded again) for the copies it still has in flight and returns.
// ---------------------------------------------------------------------------------------------------
constexpr int kFusedRows = 8;                      // rows per tile
constexpr int kFusedStages = 3;                    // tiles in flight per block
constexpr int kFusedComputeWarps = 16;             // one 16-byte column group per compute thread
constexpr int kFusedThreads = (kFusedComputeWarps + 2) * 32;   // + the slope warp and the load warp
constexpr int kFusedMaxRowBytes = 8192;            // one 16-byte group per thread
constexpr int kFusedRowPad = 16;                   // bytes between staged rows beyond the row itself (bank spread)
constexpr long long kFusedWaitCycles = 1ll << 31;  // about a second: no copy takes that long

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return done != 0;
}
// Waits for the phase with the given parity, for at most kFusedWaitCycles clock cycles.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kFusedWaitCycles) return false;
    }
    return true;
}
// One row: global -> shared, completion counted in bytes on the stage's barrier (both addresses and the size are
// multiples of 16).  The copy is this block's own: no multicast.
__device__ __forceinline__ void bulk_row_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Eight per-lane values -> per-row sums over the warp in 9 shuffles: each step hands half of the remaining rows
// to the partner lane.  Afterwards lane L holds the sum of row ((L >> 4) & 1) * 4 + ((L >> 3) & 1) * 2 + ((L >> 2) & 1).
__device__ __forceinline__ float fold8(float (&p)[8], int lane)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float send = (lane & 16) ? p[i] : p[i + 4], keep = (lane & 16) ? p[i + 4] : p[i];
        p[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 16);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const float send = (lane & 8) ? p[i] : p[i + 2], keep = (lane & 8) ? p[i + 2] : p[i];
        p[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
    }
    {
        const float send = (lane & 4) ? p[0] : p[1], keep = (lane & 4) ? p[1] : p[0];
        p[0] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
    }
    p[0] += __shfl_xor_sync(0xFFFFFFFFu, p[0], 2);
    p[0] += __shfl_xor_sync(0xFFFFFFFFu, p[0], 1);
    return p[0];
}

// Work split of the fused kernel: worker and first slot of tile t, the run of tiles of block b.
struct FusedPlan {
    int M, B, tiles_per_worker, ntiles, nblocks;              // ntiles * nblocks < 2^32 (checked by the host)
    __host__ __device__ int tile_begin(int b) const { return (int)(((unsigned)b * (unsigned)ntiles) / (unsigned)nblocks); }
    __host__ __device__ int worker_of(int t) const { return t / tiles_per_worker; }
    // blocks whose runs touch worker w: the owners of its first and last tile
    __host__ __device__ int block_of_tile(int t) const
    {
        int b = (int)(((unsigned)t * (unsigned)nblocks) / (unsigned)ntiles);       // tile_begin(b) <= t holds for this b or the next ones
        while (b + 1 < nblocks && tile_begin(b + 1) <= t) ++b;
        while (tile_begin(b) > t) --b;
        return b;
    }
};

// The stages next to the gradient, when its kernel carries them (dense messages, fixed model width 2/4/8, no
// delays).  Prologue: every block quantises the model itself (all blocks draw the same Philox stream, so the
// broadcast of Algorithm 1 step 8 needs no exchange; block 0 writes the packed model).  Epilogue: the block that
// completes a worker quantises and packs that worker's message (step 12) while alpha_w is still in its registers.
// The master step (step 9) needs every message and stays a kernel of its own.  Nobody waits for anybody: counters
// decide who goes on.
struct FusedRound {
    int fold;                                                 // 0: gradient only
    const float* x; const float* xsnap; const uint32_t* normx_in; uint8_t* codes_x; float* delta_x; int bx;   // model quantiser
    int b; uint8_t* codes; int64_t stride; float* scale;                                                      // messages
    uint32_t* normx_out; uint32_t* done;
};

// MODE 0: both products by fp32 FMAs on CUDA cores (any row type).  MODE 1: both products of bfloat16 rows as
// tensor-core MMAs.  MODE 2: the margins X (xhat - xsnap) as MMAs straight from the stage, the column sums X^T r
// by FMAs from the registers that keep the tile (so a stage is free again as soon as the margins are formed).
template <class T, int MODE>
__global__ void __launch_bounds__(kFusedThreads, 1)
worker_grad_fused_kernel(const T* __restrict__ X, const float* __restrict__ labels, const float* __restrict__ diff,
                         const float* __restrict__ z_snap, const __grid_constant__ PhiloxKeys K, BatchSource bs, FusedPlan pl,
                         int64_t d, float* __restrict__ alpha, uint32_t* __restrict__ norm_bits,
                         float* __restrict__ part /* [nblocks + M][d] column sums of (block, worker) */,
                         uint32_t* __restrict__ counters /* [M], zero between launches */, int* __restrict__ status,
                         const __grid_constant__ FusedRound fr)
{
    pdl_prologue();
    clear_word(bs);
    const uint32_t round = bs.rp ? bs.rp->round : bs.round;
    constexpr int N = RowVec<T>::N;                          // features per 16-byte group
    constexpr int S = kFusedStages, R = kFusedRows, CW = kFusedComputeWarps;
    constexpr bool MMA = MODE == 1, MMA_FRONT = MODE != 0;
    extern __shared__ __align__(128) unsigned char s_stage[];    // [S][R][row_bytes + pad]
    __shared__ __align__(8) uint64_t s_full[S], s_empty[S], s_pready[2], s_rready[2];
    __shared__ float s_part[2][CW][R];
    __shared__ float s_r[2][R];
    __shared__ __align__(4) uint16_t s_rsplit[2][3][R];          // MMA: the slopes as three bfloat16 terms (hi + mid + lo = r to 24 bits)
    __shared__ float s_lab[S + 2][R], s_zs[S + 2][R];           // ring of S + 2: tiles it + S and it + S + 1 can be issued while tile it's entries are still read
    __shared__ uint32_t s_max[CW];
    __shared__ int s_abort, s_last, s_issued, s_bfirst, s_blast;
    __shared__ uint32_t s_norm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool slope_warp = warp == CW, load_warp = warp == CW + 1, compute = warp < CW;
    const int row_bytes = (int)(d * (int64_t)sizeof(T)), stride = row_bytes + kFusedRowPad;
    const int nvec = row_bytes >> 4;
    const int v = tid;                                       // a compute thread's column group
    const bool active = compute && v < nvec;
    const int blk = blockIdx.x;
    const int t0 = pl.tile_begin(blk), ntl = pl.tile_begin(blk + 1) - t0;
    // MMA: xhat - xsnap of the current worker as three bfloat16 terms, [3][d], behind the stages
    uint16_t* s_dsplit = reinterpret_cast<uint16_t*>(s_stage + (size_t)S * R * stride);
    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], CW); }
        for (int s = 0; s < 2; ++s) { mbar_init(&s_pready[s], CW); mbar_init(&s_rready[s], 1); }
        s_abort = 0; s_last = 0; s_issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // A wait that gives up: after kFusedWaitCycles the block is marked aborted, DQ_ERR_TIMEOUT is recorded, and from
    // then on no wait of this block blocks any more.  Every thread still walks through the same barriers to the end
    // (the results are void, the status says so), so nothing is left hanging.
    auto wait = [&](uint64_t* bar, uint32_t parity) {
        if (*reinterpret_cast<volatile int*>(&s_abort)) return;
        if (mbar_try_wait(bar, parity)) return;
        const long long c0 = clock64();
        while (!mbar_try_wait(bar, parity)) {
            if (*reinterpret_cast<volatile int*>(&s_abort)) return;
            if (clock64() - c0 > kFusedWaitCycles) { s_abort = 1; set_status(status, DQ_ERR_TIMEOUT); return; }
            if (!compute) __nanosleep(200);                  // the load and slope warps have a tile's time of slack: their polling must not take issue slots from the compute warps
        }
    };
    const auto worker_at = [&](int it) { return it < ntl ? pl.worker_of(t0 + it) : -1; };
    // a worker's last tile in this block has been added when the next tile belongs to another worker (or the run ends)
    const auto flush_at = [&](int it) { return it > 0 && worker_at(it) != worker_at(it - 1); };

    // load warp, in three steps per tile so that no load of one tile holds up the copies of another: draw_row (this
    // lane's row of tile `it`, or -1), copy_rows (start the row copies into stage it % S), publish (labels and snapshot
    // margins beside the rows, then the announcement of the tile).  The labels are fetched into registers one tile
    // ahead, between draw_row and publish.
    int part_w = -1; int64_t part_lo = 0; uint64_t part_cnt = 0;
    auto draw_row = [&](int it) -> int64_t {
        const int t = t0 + it;
        const int w = pl.worker_of(t), j0 = (t - w * pl.tiles_per_worker) * R;
        const int nvalid = min(R, pl.B - j0);
        if (w != part_w) {               // the worker's partition of the rows (two 64-bit divisions: once per worker, not per row)
            part_w = w;
            part_lo = ((int64_t)w * bs.n) / bs.M; part_cnt = (uint64_t)(((int64_t)(w + 1) * bs.n) / bs.M - part_lo);
        }
        int64_t a = -1;
        if (lane < nvalid) {
            const int j = j0 + lane;
            const int64_t slot_j = (int64_t)w * pl.B + j;
            if (bs.rows_in) {
                a = bs.rows_in[slot_j];
            } else {                     // the same draw as sample_row
                uint32_t r4[4];
                philox4x32_10((uint32_t)(j >> 2), round, (uint32_t)w, kStreamBatch, K, r4);
                const uint32_t word = (j & 3) == 0 ? r4[0] : (j & 3) == 1 ? r4[1] : (j & 3) == 2 ? r4[2] : r4[3];
                a = part_lo + (int64_t)(((uint64_t)word * part_cnt) >> 32);
                if (bs.rows_out) bs.rows_out[slot_j] = (int32_t)a;
            }
        }
        return a;
    };
    auto copy_rows = [&](int it, int64_t a) {
        const int t = t0 + it, stage = it % S;
        const int w = pl.worker_of(t), j0 = (t - w * pl.tiles_per_worker) * R;
        const int nvalid = min(R, pl.B - j0);
        if (a >= 0) bulk_row_load(s_stage + ((size_t)stage * R + lane) * stride, X + a * d, (uint32_t)row_bytes, &s_full[stage]);
        if (MMA_FRONT && nvalid < R) {   // the tensor-core paths multiply whole tiles: rows past the minibatch's end must read as zeros
            uint4* z = reinterpret_cast<uint4*>(s_stage + ((size_t)stage * R + nvalid) * stride);
            for (int q = lane; q < (R - nvalid) * (stride >> 4); q += 32) z[q] = make_uint4(0u, 0u, 0u, 0u);
        }
    };
    auto publish = [&](int it, int64_t a, float lab, float zs) {
        const int t = t0 + it, stage = it % S, slot = it % (S + 2);
        const int w = pl.worker_of(t), j0 = (t - w * pl.tiles_per_worker) * R;
        const int nvalid = min(R, pl.B - j0);
        // the row's label and snapshot margin go beside it.  They are stored before this warp's arrival on the stage's
        // barrier below, so whoever has seen the stage full (and whoever hears from them) sees them too.
        if (a >= 0) { s_lab[slot][lane] = lab; s_zs[slot][lane] = zs; }
        __syncwarp();
        // the byte count is announced after the copies were started: the phase cannot complete before this arrival
        if (lane == 0) { mbar_arrive_expect_tx(&s_full[stage], (uint32_t)(nvalid * row_bytes)); s_issued = it + 1; }
    };

    // the flush of worker w: every thread of the block takes part in its barriers
    float acc[N];
#pragma unroll
    for (int n = 0; n < N; ++n) acc[n] = 0.0f;
    auto flush = [&](int w) {
        if (!MMA && active) {
            float4* dst = reinterpret_cast<float4*>(part + (size_t)(blk + w) * d) + (size_t)v * (N / 4);
#pragma unroll
            for (int q = 0; q < N / 4; ++q) dst[q] = make_float4(acc[q * 4], acc[q * 4 + 1], acc[q * 4 + 2], acc[q * 4 + 3]);
        }
#pragma unroll
        for (int n = 0; n < N; ++n) acc[n] = 0.0f;
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int bf = pl.block_of_tile(w * pl.tiles_per_worker), bl = pl.block_of_tile((w + 1) * pl.tiles_per_worker - 1);
            s_bfirst = bf; s_blast = bl;
            const uint32_t old = atomicAdd(counters + w, 1u);
            s_last = old == (uint32_t)(bl - bf);
            if (s_last) counters[w] = 0u;                    // every block of this worker has added: ready for the next launch
        }
        __syncthreads();
        if (s_last) {                                        // this block completes worker w: slots in block order
            const int b_first = s_bfirst, b_last = s_blast;
            __threadfence();
            uint32_t nmax = 0;
            float sum[N];
#pragma unroll
            for (int n = 0; n < N; ++n) sum[n] = 0.0f;
            if (active) {
                constexpr int U = 4;                             // slots fetched together: their loads overlap, the adds keep block order
                for (int bb0 = b_first; bb0 <= b_last; bb0 += U) {
                    float4 x4[U][N / 4];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const float4* src = reinterpret_cast<const float4*>(part + (size_t)(min(bb0 + u, b_last) + w) * d) + (size_t)v * (N / 4);
#pragma unroll
                        for (int q = 0; q < N / 4; ++q) x4[u][q] = __ldcg(src + q);
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (bb0 + u <= b_last) {
#pragma unroll
                            for (int q = 0; q < N / 4; ++q) {
                                sum[q * 4] += x4[u][q].x; sum[q * 4 + 1] += x4[u][q].y; sum[q * 4 + 2] += x4[u][q].z; sum[q * 4 + 3] += x4[u][q].w;
                            }
                        }
                    }
                }
                float4* out = reinterpret_cast<float4*>(alpha + (size_t)w * d) + (size_t)v * (N / 4);
#pragma unroll
                for (int q = 0; q < N / 4; ++q) out[q] = make_float4(sum[q * 4], sum[q * 4 + 1], sum[q * 4 + 2], sum[q * 4 + 3]);
#pragma unroll
                for (int n = 0; n < N; ++n) nmax = max(nmax, __float_as_uint(sum[n]) & 0x7FFFFFFFu);
            }
            nmax = warp_max_u32(nmax);
            if (compute && lane == 0) s_max[warp] = nmax;
            __syncthreads();
            if (tid == 0) {
                uint32_t m = 0;
                for (int k = 0; k < CW; ++k) m = max(m, s_max[k]);
                norm_bits[w] = m; s_norm = m;
            }
            __syncthreads();
            if (fr.fold) {
                // ---- message w: Q_(delta,b) of alpha_w with delta from ||alpha_w||_inf, packed (Algorithm 1 step 12) -------
                const uint32_t nb = s_norm;
                const bool ok = nb < 0x7F800000u && nb != 0u;
                const int L = levels(fr.b);
                const float inv = ok ? __fdiv_rd((float)L, __uint_as_float(nb)) : 0.0f;
                if (tid == 0) {
                    fr.scale[w] = ok ? __fdiv_rn(__uint_as_float(nb), (float)L) : 0.0f;
                    if (nb >= 0x7F800000u) set_status(status, DQ_ERR_NONFINITE);
                }
                const int ngroups = (int)(fr.stride / fr.b);                    // covers the zero padding of the packed message
                if (compute) {
                    // a thread holds N consecutive coordinates; a Philox call serves a group of eight
                    for (int base = 0; base < ngroups; base += (CW * 32 * N) >> 3) {     // the same trip count in every thread (shuffles inside)
                        const int g = base + ((v * N) >> 3);
                        uint32_t r4[4], q[8];
                        philox4x32_10((uint32_t)g, round, (uint32_t)w, kStreamGrad, K, r4);
                        float a8[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) a8[j] = 0.0f;
                        if (N == 8) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) a8[j] = (active && base == 0) ? sum[j % N] : 0.0f;
                        } else {                                                    // N == 4: the group's other half sits in the neighbour lane
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float mine = (active && base == 0) ? sum[j % N] : 0.0f;
                                const float other = __shfl_xor_sync(0xFFFFFFFFu, mine, 1);
                                a8[j] = (v & 1) ? other : mine; a8[4 + j] = (v & 1) ? mine : other;
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j) q[j] = nb < 0x7F800000u ? round_fixed<8>(a8[j], inv, half16(r4, j)) : (128u << 16);
                        if (g < ngroups && (N == 8 || !(v & 1))) {
                            uint8_t* dst = fr.codes + (size_t)w * fr.stride + (size_t)g * fr.b;
                            if (fr.b == 8) store_group<8>(dst, pack8<8>(q)); else if (fr.b == 4) store_group<4>(dst, pack8<4>(q)); else store_group<2>(dst, pack8<2>(q));
                        }
                    }
                }
                // ---- the block that completes the last message clears ||x||_inf for the master kernel's maximum (every block has
                // long read it: the model was quantised in the prologue) -------------------------------------------------------
                __threadfence();
                __syncthreads();
                if (tid == 0) {
                    const uint32_t old = atomicAdd(fr.done, 1u);
                    if (old == (uint32_t)(pl.M - 1)) { *fr.done = 0u; *fr.normx_out = 0u; }
                }
            }
        }
    };

    // Prologue of a whole round: Q_(delta_x, b_x) of the model for this thread's N coordinates (every block draws the same
    // codes; block 0 writes the packed model and delta_x), returned as xhat - xsnap.
    auto model_diff = [&](float (&out)[N]) {
        const uint32_t nb = *fr.normx_in;
        const bool ok = nb < 0x7F800000u && nb != 0u;
        const int L = levels(fr.bx);
        const float inv = ok ? __fdiv_rd((float)L, __uint_as_float(nb)) : 0.0f;
        const float delta = ok ? __fdiv_rn(__uint_as_float(nb), (float)L) : 0.0f;
        if (blk == 0 && tid == 0) { *fr.delta_x = delta; if (nb >= 0x7F800000u) set_status(status, DQ_ERR_NONFINITE); }
        const int ngroups_x = (int)((((d * fr.bx + 7) / 8 + 15) / 16 * 16) / fr.bx);      // block 0 also writes the padding of the packed model
        for (int base = 0; base < (blk == 0 ? ngroups_x : 1); base += (CW * 32 * N) >> 3) {
            const int g = base + ((v * N) >> 3);
            const int64_t i0 = (int64_t)g << 3;
            float a8[8], xs8[N];
#pragma unroll
            for (int j = 0; j < 8; ++j) a8[j] = (i0 + j < d) ? __ldcg(fr.x + i0 + j) : 0.0f;
#pragma unroll
            for (int n = 0; n < N; ++n) {                    // the snapshot's coordinates travel together with the model's
                const int64_t i = i0 + (N == 8 ? n : (v & 1) * 4 + n);
                xs8[n] = (base == 0 && active && i < d) ? __ldg(fr.xsnap + i) : 0.0f;
            }
            uint32_t r4[4], q[8];
            philox4x32_10((uint32_t)g, round, kMaster, kStreamModel, K, r4);
#pragma unroll
            for (int j = 0; j < 8; ++j) q[j] = nb < 0x7F800000u ? round_fixed<8>(a8[j], inv, half16(r4, j)) : (128u << 16);
            if (blk == 0 && g < ngroups_x && (N == 8 || !(v & 1))) {
                uint8_t* dst = fr.codes_x + (size_t)g * fr.bx;
                if (fr.bx == 8) store_group<8>(dst, pack8<8>(q)); else if (fr.bx == 4) store_group<4>(dst, pack8<4>(q)); else store_group<2>(dst, pack8<2>(q));
            }
            if (base == 0) {
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const int j = N == 8 ? n : (v & 1) * 4 + n;
                    const int64_t i = i0 + j;
                    const float k = (float)((int)((q[j] >> 16) & 0xFFu) - 128);
                    out[n] = (active && i < d) ? __fsub_rn(__fmul_rn(k, delta), xs8[n]) : 0.0f;
                }
            }
        }
    };

    if (load_warp) {
        // ---- copies: S tiles ahead; a stage is refilled once every compute warp has taken its groups out of it -------
        int64_t a0[S]; float lab0[S], zs0[S];
#pragma unroll
        for (int k = 0; k < S; ++k) {                        // rows of the first tiles, their small loads in flight,
            a0[k] = k < ntl ? draw_row(k) : -1; lab0[k] = zs0[k] = 0.0f;
            if (a0[k] >= 0) { lab0[k] = __ldg(labels + a0[k]); zs0[k] = __ldg(z_snap + a0[k]); }
        }
#pragma unroll
        for (int k = 0; k < S; ++k) if (k < ntl) copy_rows(k, a0[k]);              // all row copies,
#pragma unroll
        for (int k = 0; k < S; ++k) if (k < ntl) publish(k, a0[k], lab0[k], zs0[k]);   // then the announcements
        int64_t a_n = S < ntl ? draw_row(S) : -1;            // one tile ahead: its labels arrive while the stage is still in use
        float lab_n = 0.0f, zs_n = 0.0f;
        if (a_n >= 0) { lab_n = __ldg(labels + a_n); zs_n = __ldg(z_snap + a_n); }
        for (int it = 0; it <= ntl; ++it) {
            if (flush_at(it)) flush(worker_at(it - 1));
            if (it + S < ntl) {
                wait(&s_empty[it % S], (uint32_t)((it / S) & 1));
                copy_rows(it + S, a_n);
                publish(it + S, a_n, lab_n, zs_n);
                a_n = it + S + 1 < ntl ? draw_row(it + S + 1) : -1;
                if (a_n >= 0) { lab_n = __ldg(labels + a_n); zs_n = __ldg(z_snap + a_n); }
            }
        }
    } else if (slope_warp) {
        // ---- slopes: margins of tile it from the warps' partial sums (warp order, double), slope differences --------
        for (int it = 0; it <= ntl; ++it) {
            if (flush_at(it)) flush(worker_at(it - 1));
            if (it == ntl) break;
            const int par = it & 1;
            const int w_cur = worker_at(it), j0 = (t0 + it - w_cur * pl.tiles_per_worker) * R;
            const int nvalid = min(R, pl.B - j0);
            wait(&s_pready[par], (uint32_t)((it >> 1) & 1));
            // lane = 4 * row + quarter: a quarter of the warps' partial sums each, then the quarters in order
            const int row = lane >> 2, qtr = lane & 3;
            double dz = 0.0;
#pragma unroll
            for (int k = 0; k < CW / 4; ++k) dz += (double)s_part[par][qtr * (CW / 4) + k][row];
            const double d1 = __shfl_xor_sync(0xFFFFFFFFu, dz, 1);
            dz = (qtr & 1) ? d1 + dz : dz + d1;                  // (q0 + q1), (q2 + q3): the same order in both lanes
            const double d2 = __shfl_xor_sync(0xFFFFFFFFu, dz, 2);
            dz = (qtr & 2) ? d2 + dz : dz + d2;
            if (qtr == 0) {
                float rj = 0.0f;
                if (row < nvalid) {
                    const int slot = it % (S + 2);
                    rj = slope_difference(*reinterpret_cast<volatile float*>(&s_lab[slot][row]), *reinterpret_cast<volatile float*>(&s_zs[slot][row]), (float)dz) / (float)pl.B;
                }
                s_r[par][row] = rj;
                if (MMA) {
                    const __nv_bfloat16 hi = __float2bfloat16_rn(rj);
                    const float r1 = rj - __bfloat162float(hi);
                    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                    s_rsplit[par][0][row] = __bfloat16_as_ushort(hi); s_rsplit[par][1][row] = __bfloat16_as_ushort(mid);
                    s_rsplit[par][2][row] = __bfloat16_as_ushort(lo);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_rready[par]);
        }
    } else if (MMA) {
        // ---- compute warps, tensor cores -----------------------------------------------------------------------------
        // Both products of a tile run as warp-level bf16 MMAs with fp32 accumulation; an fp32 factor enters as three
        // bfloat16 terms in three columns of the narrow operand.  Warp wp owns the columns [wp cpw, (wp + 1) cpw).
        //   margins  D[variant][row] += sum_k diff_variant[k] X[row][k]: m16n8k16, A = the three terms of xhat - xsnap
        //            (rows 0..2 of 16), B = the tile's eight rows straight from the stage (ldmatrix)
        //   columns  D[col][variant] += sum_row X[row][col] r_variant[row]: m16n8k8, A = the tile transposed
        //            (ldmatrix.trans), B = the three terms of the slopes; 16 columns x 8 per MMA, 4 accumulators each
        const int g = lane >> 2, c2 = (lane & 3) * 2;
        const int ksteps = (int)(d >> 4), kpw = (ksteps + CW - 1) / CW;               // 16-column steps in all, per warp
        const int k_first = warp * kpw, k_count = max(0, min(kpw, ksteps - k_first));
        float cacc[kFusedMaxRowBytes / 2 / 16 / CW][4];                               // [m-tile][4]: columns of this warp
#pragma unroll
        for (int i = 0; i < kFusedMaxRowBytes / 2 / 16 / CW; ++i) { cacc[i][0] = cacc[i][1] = cacc[i][2] = cacc[i][3] = 0.0f; }
        int w_prev = -1;
        const uint32_t lane_row_off = (uint32_t)((lane & 7) * stride + ((lane >> 3) & 1) * 16);   // ldmatrix: lanes 0-7 first matrix, 8-15 second
        if (fr.fold) {                                       // the model's xhat - xsnap, formed here, as hi + mid + lo
            float df[N];
            model_diff(df);
            if (active) {
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const int64_t i = (int64_t)v * N + n;
                    const __nv_bfloat16 hi = __float2bfloat16_rn(df[n]);
                    const float r1 = df[n] - __bfloat162float(hi);
                    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                    s_dsplit[i] = __bfloat16_as_ushort(hi); s_dsplit[d + i] = __bfloat16_as_ushort(mid); s_dsplit[2 * d + i] = __bfloat16_as_ushort(lo);
                }
            }
            asm volatile("bar.sync 1, %0;" :: "n"(CW * 32) : "memory");
        }
        for (int it = 0; it <= ntl; ++it) {
            const int par = it & 1, stage = it % S;
            const int w_cur = worker_at(it);
            if (it < ntl) {
                if (!fr.fold && w_cur != w_prev) {           // new worker: its xhat - xsnap as hi + mid + lo
                    asm volatile("bar.sync 1, %0;" :: "n"(CW * 32) : "memory");      // every compute warp is done with the old terms
                    const float* dv = diff_of_worker(bs, diff, w_cur);
                    for (int64_t i = tid; i < d; i += CW * 32) {
                        const float x = __ldg(dv + i);
                        const __nv_bfloat16 hi = __float2bfloat16_rn(x);
                        const float r1 = x - __bfloat162float(hi);
                        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                        const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                        s_dsplit[i] = __bfloat16_as_ushort(hi); s_dsplit[d + i] = __bfloat16_as_ushort(mid); s_dsplit[2 * d + i] = __bfloat16_as_ushort(lo);
                    }
                    asm volatile("bar.sync 1, %0;" :: "n"(CW * 32) : "memory");
                }
                wait(&s_full[stage], (uint32_t)((it / S) & 1));
                const uint32_t sbase = smem_u32(s_stage + (size_t)stage * R * stride) + lane_row_off;
                float c0 = 0.0f, c1 = 0.0f, c2r = 0.0f, c3 = 0.0f;
#pragma unroll 4
                for (int ks = 0; ks < k_count; ++ks) {
                    const int col = (k_first + ks) << 4;
                    uint32_t a0 = 0u, a2 = 0u, b0, b1;
                    if (g < 3) {
                        const uint16_t* dp = s_dsplit + (size_t)g * d + col + c2;
                        a0 = *reinterpret_cast<const uint32_t*>(dp); a2 = *reinterpret_cast<const uint32_t*>(dp + 8);
                    }
                    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(sbase + (uint32_t)col * 2u));
                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                 : "+f"(c0), "+f"(c1), "+f"(c2r), "+f"(c3) : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
                }
                // rows 0..2 of D hold the three terms' sums for tile rows c2, c2 + 1: add them up (the other rows are zero)
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) { c0 += __shfl_xor_sync(0xFFFFFFFFu, c0, o); c1 += __shfl_xor_sync(0xFFFFFFFFu, c1, o); }
                if (it >= 2) wait(&s_rready[par], (uint32_t)(((it - 2) >> 1) & 1));      // the slopes of tile it - 2 have been formed: its partial sums are free
                if (lane < 4) { s_part[par][warp][c2] = c0; s_part[par][warp][c2 + 1] = c1; }
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_pready[par]);
            }
            if (it > 0) {
                // back: the rows of tile it - 1 (still in their stage) times their slopes
                wait(&s_rready[par ^ 1], (uint32_t)(((it - 1) >> 1) & 1));
                const int pstage = (it - 1) % S;
                const uint32_t sbase = smem_u32(s_stage + (size_t)pstage * R * stride) + lane_row_off;
                const uint32_t b0 = g < 3 ? *reinterpret_cast<const uint32_t*>(&s_rsplit[par ^ 1][g][c2]) : 0u;
#pragma unroll
                for (int i = 0; i < kFusedMaxRowBytes / 2 / 16 / CW; ++i) {
                    if (i < k_count) {
                        const int col = (k_first + i) << 4;
                        uint32_t a0, a1;
                        asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(a0), "=r"(a1) : "r"(sbase + (uint32_t)col * 2u));
                        asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                                     : "+f"(cacc[i][0]), "+f"(cacc[i][1]), "+f"(cacc[i][2]), "+f"(cacc[i][3]) : "r"(a0), "r"(a1), "r"(b0));
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_empty[pstage]);    // the tile has been used for both products: the stage may be refilled
            }
            if (flush_at(it)) {
                // column sum = hi + mid + lo columns of D: lanes with c2 == 0 hold the first two, their neighbour the third
                float* dst = part + (size_t)(blk + w_prev) * d;
#pragma unroll
                for (int i = 0; i < kFusedMaxRowBytes / 2 / 16 / CW; ++i) {
                    float u0 = cacc[i][0] + cacc[i][1], u1 = cacc[i][2] + cacc[i][3];
                    u0 += __shfl_xor_sync(0xFFFFFFFFu, u0, 1); u1 += __shfl_xor_sync(0xFFFFFFFFu, u1, 1);
                    if (i < k_count && c2 == 0) { const int col = ((k_first + i) << 4) + g; dst[col] = u0; dst[col + 8] = u1; }
                    cacc[i][0] = cacc[i][1] = cacc[i][2] = cacc[i][3] = 0.0f;
                }
                flush(w_prev);
            }
            w_prev = w_cur;
        }
    } else {
        // ---- compute warps, CUDA cores ---------------------------------------------------------------------------------
        float dreg[N];
#pragma unroll
        for (int n = 0; n < N; ++n) dreg[n] = 0.0f;
        if (fr.fold) model_diff(dreg);                       // the model's xhat - xsnap, formed here
        const int g = lane >> 2, c2 = (lane & 3) * 2;        // MMA_FRONT: this lane's row of A / pair of columns of D
        const int ksteps = (int)(d >> 4), kpw = (ksteps + CW - 1) / CW;
        const int k_first = warp * kpw, k_count = max(0, min(kpw, ksteps - k_first));
        const uint32_t lane_row_off = (uint32_t)((lane & 7) * stride + ((lane >> 3) & 1) * 16);
        auto split_to_smem = [&](const float (&df)[N]) {     // this thread's N coordinates of xhat - xsnap as hi + mid + lo
            if (active) {
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const int64_t i = (int64_t)v * N + n;
                    const __nv_bfloat16 hi = __float2bfloat16_rn(df[n]);
                    const float r1 = df[n] - __bfloat162float(hi);
                    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                    s_dsplit[i] = __bfloat16_as_ushort(hi); s_dsplit[d + i] = __bfloat16_as_ushort(mid); s_dsplit[2 * d + i] = __bfloat16_as_ushort(lo);
                }
            }
            asm volatile("bar.sync 1, %0;" :: "n"(CW * 32) : "memory");
        };
        if (MMA_FRONT && fr.fold) split_to_smem(dreg);
        uint4 q_old[R], q_new[R];
#pragma unroll
        for (int r = 0; r < R; ++r) q_old[r] = q_new[r] = make_uint4(0u, 0u, 0u, 0u);
        int w_prev = -1, nvalid_prev = 0;
        for (int it = 0; it <= ntl; ++it) {
            const int par = it & 1, stage = it % S;
            const int w_cur = worker_at(it);
            const int j0 = it < ntl ? (t0 + it - w_cur * pl.tiles_per_worker) * R : 0;
            const int nvalid = it < ntl ? min(R, pl.B - j0) : 0;
            if (it < ntl) {
                // front: margins of tile it
                if (!fr.fold && w_cur != w_prev) {             // this worker's xhat - xsnap (a lagging worker reads an older one)
                    if (MMA_FRONT) asm volatile("bar.sync 1, %0;" :: "n"(CW * 32) : "memory");    // every compute warp is done with the old terms
                    if (active) {
                        const float4* dv = reinterpret_cast<const float4*>(diff_of_worker(bs, diff, w_cur)) + (size_t)v * (N / 4);
#pragma unroll
                        for (int q = 0; q < N / 4; ++q) { const float4 x4 = __ldg(dv + q); dreg[q * 4] = x4.x; dreg[q * 4 + 1] = x4.y; dreg[q * 4 + 2] = x4.z; dreg[q * 4 + 3] = x4.w; }
                    }
                    if (MMA_FRONT) split_to_smem(dreg);
                }
                wait(&s_full[stage], (uint32_t)((it / S) & 1));
                const unsigned char* base = s_stage + (size_t)stage * R * stride + (size_t)v * 16;
                if (nvalid == R && active) {
#pragma unroll
                    for (int r = 0; r < R; ++r) q_new[r] = *reinterpret_cast<const uint4*>(base + (size_t)r * stride);
                } else {
#pragma unroll
                    for (int r = 0; r < R; ++r)
                        q_new[r] = (active && r < nvalid) ? *reinterpret_cast<const uint4*>(base + (size_t)r * stride) : make_uint4(0u, 0u, 0u, 0u);
                }
                if (!MMA_FRONT) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s_empty[stage]);     // this warp's groups are in registers: the stage may be refilled
                    float p[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        float f[N];
                        RowVec<T>::unpack(q_new[r], f);
                        float s = 0.0f;
#pragma unroll
                        for (int n = 0; n < N; ++n) s = fmaf(f[n], dreg[n], s);
                        p[r] = s;
                    }
                    if (it >= 2) wait(&s_rready[par], (uint32_t)(((it - 2) >> 1) & 1));      // the slopes of tile it - 2 have been formed: its partial sums are free
                    const float folded = fold8(p, lane);
                    if ((lane & 3) == 0) s_part[par][warp][((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1)] = folded;
                } else {
                    // margins by MMA from the stage: D[term][row] += sum_k diff_term[k] X[row][k] over this warp's columns
                    const uint32_t sbase = smem_u32(s_stage + (size_t)stage * R * stride) + lane_row_off;
                    float c0 = 0.0f, c1 = 0.0f, c2r = 0.0f, c3 = 0.0f;
#pragma unroll 4
                    for (int ks = 0; ks < k_count; ++ks) {
                        const int col = (k_first + ks) << 4;
                        uint32_t a0 = 0u, a2 = 0u, b0, b1;
                        if (g < 3) {
                            const uint16_t* dp = s_dsplit + (size_t)g * d + col + c2;
                            a0 = *reinterpret_cast<const uint32_t*>(dp); a2 = *reinterpret_cast<const uint32_t*>(dp + 8);
                        }
                        asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(sbase + (uint32_t)col * 2u));
                        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                     : "+f"(c0), "+f"(c1), "+f"(c2r), "+f"(c3) : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s_empty[stage]);     // the margins are formed and the groups are in registers
#pragma unroll
                    for (int o = 4; o < 32; o <<= 1) { c0 += __shfl_xor_sync(0xFFFFFFFFu, c0, o); c1 += __shfl_xor_sync(0xFFFFFFFFu, c1, o); }
                    if (it >= 2) wait(&s_rready[par], (uint32_t)(((it - 2) >> 1) & 1));
                    if (lane < 4) { s_part[par][warp][c2] = c0; s_part[par][warp][c2 + 1] = c1; }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_pready[par]);
            }
            if (it > 0) {
                // back: add the rows of tile it - 1 to the columns
                wait(&s_rready[par ^ 1], (uint32_t)(((it - 1) >> 1) & 1));
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    if (r < nvalid_prev) {                   // (rows past the end were loaded as zeros, but their slot of s_r is stale)
                        const float rr = s_r[par ^ 1][r];
                        float f[N];
                        RowVec<T>::unpack(q_old[r], f);
#pragma unroll
                        for (int n = 0; n < N; ++n) acc[n] = fmaf(rr, f[n], acc[n]);
                    }
                }
            }
            if (flush_at(it)) flush(w_prev);
#pragma unroll
            for (int r = 0; r < R; ++r) q_old[r] = q_new[r];
            w_prev = w_cur; nvalid_prev = nvalid;
        }
    }
    __syncthreads();
    if (s_abort && tid == 0) {
        // a copy did not arrive in time: give the copies still in flight a bounded time to land before the block's
        // shared memory is released
        for (int k = 0; k < s_issued; ++k) (void)mbar_wait_bounded(&s_full[k % S], (uint32_t)((k / S) & 1));
    }
}

// ---------------------------------------------------------------------------------------------------
// Full gradient over all n rows at xsnap, accumulated in double; also stores the margins z_snap.
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
full_grad_csr_kernel(const float* __restrict__ val, const int32_t* __restrict__ col, const int64_t* __restrict__ row_ptr,
                     const float* __restrict__ labels, const float* __restrict__ x, int64_t n, float* __restrict__ z_out,
                     double* __restrict__ g64)
{
    pdl_prologue();
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t a = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; a < n; a += nwarps) {
        const int64_t k0 = row_ptr[a], k1 = row_ptr[a + 1];
        const double z = warp_dot_csr(val, col, k0, k1, x, lane);
        const double y = (double)labels[a];
        const double c = -y / (1.0 + exp(y * z));
        if (lane == 0 && z_out) z_out[a] = (float)z;
        for (int64_t k = k0 + lane; k < k1; k += 32) atomicAdd(g64 + __ldg(col + k), c * (double)__ldg(val + k));
    }
}

template <class T>
__global__ void __launch_bounds__(kThreads)
full_grad_dense_kernel(const T* __restrict__ X, const float* __restrict__ labels, const float* __restrict__ x, int64_t n,
                       int64_t d, float* __restrict__ z_out, double* __restrict__ g64)
{
    pdl_prologue();
    __shared__ float s_c[kRowsPerBlock];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t a0 = (int64_t)blockIdx.x * kRowsPerBlock; a0 < n; a0 += (int64_t)gridDim.x * kRowsPerBlock) {
        const int nrows = (int)min((int64_t)kRowsPerBlock, n - a0);
        for (int j = warp; j < nrows; j += kThreads / 32) {
            const double z = warp_dot_dense(X + (a0 + j) * d, x, d, lane);
            const double y = (double)labels[a0 + j];
            if (lane == 0) { s_c[j] = (float)(-y / (1.0 + exp(y * z))); if (z_out) z_out[a0 + j] = (float)z; }
        }
        __syncthreads();
        for (int64_t i = threadIdx.x; i < d; i += blockDim.x) {
            double s = 0.0;
            for (int j = 0; j < nrows; ++j) s += (double)s_c[j] * (double)to_float(X[(a0 + j) * d + i]);
            atomicAdd(g64 + i, s);
        }
        __syncthreads();
    }
}

// Vectorised variant of full_grad_dense_kernel (d a multiple of the 16-byte vector width).
template <class T>
__global__ void __launch_bounds__(kThreads)
full_grad_dense_vec_kernel(const T* __restrict__ X, const float* __restrict__ labels, const float* __restrict__ x, int64_t n,
                           int64_t d, float* __restrict__ z_out, double* __restrict__ g64)
{
    pdl_prologue();
    constexpr int N = RowVec<T>::N;
    __shared__ float s_c[kRowsPerBlock];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nv = (int)(d / N);
    for (int64_t a0 = (int64_t)blockIdx.x * kRowsPerBlock; a0 < n; a0 += (int64_t)gridDim.x * kRowsPerBlock) {
        const int nrows = (int)min((int64_t)kRowsPerBlock, n - a0);
        for (int j = warp; j < nrows; j += kThreads / 32) {
            const double z = warp_dot_dense_vec(X + (a0 + j) * d, x, d, lane);
            const double y = (double)labels[a0 + j];
            if (lane == 0) { s_c[j] = (float)(-y / (1.0 + exp(y * z))); if (z_out) z_out[a0 + j] = (float)z; }
        }
        __syncthreads();
        for (int v = threadIdx.x; v < nv; v += blockDim.x) {
            double acc[N];
#pragma unroll
            for (int q = 0; q < N; ++q) acc[q] = 0.0;
            for (int j = 0; j < nrows; ++j) {
                float f[N];
                RowVec<T>::unpack(__ldg(reinterpret_cast<const uint4*>(X + (a0 + j) * d) + v), f);
                const double c = (double)s_c[j];
#pragma unroll
                for (int q = 0; q < N; ++q) acc[q] += c * (double)f[q];
            }
#pragma unroll
            for (int q = 0; q < N; ++q) atomicAdd(g64 + (int64_t)v * N + q, acc[q]);
        }
        __syncthreads();
    }
}

__global__ void finish_full_grad_kernel(const double* __restrict__ g64, int64_t d, double inv_n, float* __restrict__ g)
{
    pdl_prologue();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x)
        g[i] = (float)(g64[i] * inv_n);
}

// Epoch boundary on the iterates.  Algorithms 1/2: xsnap <- x.  Algorithm 3: xsnap <- xsum / m (if m > 0),
// xsum <- 0, x <- xsnap + theta (y - xsnap).  Also ||x||_inf.
__global__ void __launch_bounds__(kThreads)
epoch_state_kernel(float* __restrict__ x, float* __restrict__ xsnap, const float* __restrict__ y, float* __restrict__ xsum,
                   int64_t d, int accelerated, int64_t m_prev, float theta, uint32_t* __restrict__ normx_bits)
{
    pdl_prologue();
    uint32_t nmax = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
        float xi;
        if (!accelerated) {
            xi = x[i]; xsnap[i] = xi;
        } else {
            float xs = xsnap[i];
            if (m_prev > 0) { xs = __fdiv_rn(xsum[i], (float)m_prev); xsnap[i] = xs; }
            xsum[i] = 0.0f;
            xi = __fmaf_rn(theta, __fsub_rn(y[i], xs), xs);
            x[i] = xi;
        }
        nmax = max(nmax, __float_as_uint(xi) & 0x7FFFFFFFu);
    }
    block_atomic_max(nmax, normx_bits);
}

// ---------------------------------------------------------------------------------------------------
// Objective P(x) = (1/n) sum log(1+exp(-y z)) + lambda1 |x|_1 + (lambda2/2) |x|^2 into one double.
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ double softplus(double m) { return m > 0.0 ? m + log1p(exp(-m)) : log1p(exp(m)); }

__device__ __forceinline__ void block_add_double(double v, double* dst)
{
    __shared__ double s_part[kThreads / 32];
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) { double t = 0.0; for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += s_part[i]; atomicAdd(dst, t); }
    __syncthreads();
}

template <int FMT>
__global__ void __launch_bounds__(kThreads)
objective_loss_kernel(dq_data D, const float* __restrict__ x, double* __restrict__ P)
{
    pdl_prologue();
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    double acc = 0.0;
    for (int64_t a = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; a < D.n; a += nwarps) {
        double z;
        if (FMT == DQ_CSR_F32) z = warp_dot_csr((const float*)D.values, D.col_idx, D.row_ptr[a], D.row_ptr[a + 1], x, lane);
        else if (FMT == DQ_DENSE_F32) z = warp_dot_dense((const float*)D.values + a * D.d, x, D.d, lane);
        else z = warp_dot_dense((const __nv_bfloat16*)D.values + a * D.d, x, D.d, lane);
        if (lane == 0) acc += softplus(-(double)D.labels[a] * z) / (double)D.n;
    }
    block_add_double(acc, P);
}

__global__ void __launch_bounds__(kThreads)
objective_reg_kernel(const float* __restrict__ x, int64_t d, float l1, float l2, double* __restrict__ P)
{
    pdl_prologue();
    double acc = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
        const double v = (double)x[i];
        acc += (double)l1 * fabs(v) + 0.5 * (double)l2 * v * v;
    }
    block_add_double(acc, P);
}

// ---------------------------------------------------------------------------------------------------
// Second smooth part (Section 5.2): 3-layer fully connected network, in -> hidden (ReLU) -> classes, softmax
// cross-entropy.  Parameters x = [W1 (hidden x in, row-major), b1, W2 (classes x hidden), b2]; labels hold class
// indices.  The worker needs grad f_B(xhat) - grad f_B(xsnap): three small kernels evaluate both parameter
// vectors side by side (either may be absent: NULL), rows listed explicitly or drawn from the batch stream.
//   mlp_hidden_kernel   block per tile of eight sampled rows and eight hidden units: hidden activations of both parameter
//                       vectors as 8x8x4 fp64 tensor-core MMAs (rows x units x inputs)
//   mlp_output_kernel   block per sampled row: logits, softmax, d loss / d logits, d loss / d hidden (ReLU-gated)
//   mlp_param_kernel    block per (tile of eight hidden units or the tail, worker): the first-layer gradient as 8x8x4 fp64
//                       MMAs (units x inputs x rows) over the worker's rows in slot order, no atomics
// The forward pass (hidden pre-activations, activations, logits, softmax) runs in double precision: a class
// probability depends on sums of hundreds of products that cancel, and an fp32 sum's error of 2^-24 of the
// absolute terms passes through the softmax into every coordinate of the gradient, where the attainable accuracy
// is set by much smaller per-sample terms.  The derivatives leave the forward pass rounded to fp32 once.
// ---------------------------------------------------------------------------------------------------
struct MlpShape { int64_t in; int hidden, classes; };

__device__ __forceinline__ int64_t mlp_off_b1(const MlpShape& s) { return (int64_t)s.hidden * s.in; }
__device__ __forceinline__ int64_t mlp_off_w2(const MlpShape& s) { return mlp_off_b1(s) + s.hidden; }
__device__ __forceinline__ int64_t mlp_off_b2(const MlpShape& s) { return mlp_off_w2(s) + (int64_t)s.classes * s.hidden; }

constexpr int kMlpUnits = 8;         // hidden units whose first-layer gradients one block forms from the same rows
constexpr int kMlpTile = 16;         // sampled rows that share one pass over a hidden unit's weights
constexpr int kMlpRowChunk = 128;    // rows whose slope differences a block of mlp_param_kernel stages at a time

// D (8x8, fp64) += A (8x4, row-major) * B (4x8, column-major) on the tensor cores' double-precision path: every
// product and sum is an IEEE fp64 fused multiply-add.  Lane l holds A[l / 4][l % 4], B[l % 4][l / 4] and the pair
// D[l / 4][2 (l % 4)], D[l / 4][2 (l % 4) + 1].
__device__ __forceinline__ void dmma_8x8x4(double& d0, double& d1, double a, double b)
{
    asm("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};" : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
}

// Four consecutive floats of a row starting at feature i (zero beyond the row's end, or when the row is absent).
// VEC: the row length is a multiple of four and the rows are 16-byte aligned, so one 16-byte load serves.
template <bool VEC>
__device__ __forceinline__ float4 mlp_load4(const float* __restrict__ p, int i, int in)
{
    float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    if (!p || i >= in) return v;
    if (VEC) return __ldg(reinterpret_cast<const float4*>(p + i));
    v.x = __ldg(p + i);
    if (i + 1 < in) v.y = __ldg(p + i + 1);
    if (i + 2 < in) v.z = __ldg(p + i + 2);
    if (i + 3 < in) v.w = __ldg(p + i + 3);
    return v;
}

// grid (ceil(nslots / kMlpTile), ceil(hidden / 8)): a block forms the pre-activations of kMlpTile = 16 sampled rows
// (two tiles of eight) and eight hidden units, for both parameter vectors, as 8x8 fp64 tensor-core tiles: A = the
// rows' features, B = the units' weight rows, both read straight from global memory (L2-resident).  A lane loads
// 16 bytes of its row and of its unit's two weight rows per chunk of 16 inputs: input 16 c + 4 (lane % 4) + e is
// the lane's k of the chunk's e-th MMA step (the order of a sum's terms is free, and fixed here), so every 32-byte
// sector that is fetched is used, and four row tiles x models share each weight load.  The chunks are split over
// the block's eight warps, kMlpBatch chunks in flight per warp; the warps' partial tiles are added in warp order,
// then bias and ReLU.
constexpr int kMlpBatch = 3;
template <bool VEC>
__global__ void __launch_bounds__(kThreads)
mlp_hidden_kernel(const float* __restrict__ X, MlpShape sh, const float* xa, const float* __restrict__ xb,
                  const __grid_constant__ PhiloxKeys K, BatchSource bs, int B, int32_t* __restrict__ row_of_slot,
                  double* __restrict__ act_a, double* __restrict__ act_b, int64_t nslots)
{
    pdl_prologue();
    __shared__ int64_t s_row[kMlpTile], s_slot[kMlpTile];
    __shared__ double s_red[kThreads / 32][2][kMlpTile * 8];      // [warp][model][row * 8 + unit]
    clear_word(bs);
    // Workers that lag read their own copy of the model (a slot of the ring): then a tile holds rows of one worker only.
    const bool per_worker = B > 0 && bs.diff_slot != nullptr;
    const int tpw = per_worker ? (B + kMlpTile - 1) / kMlpTile : 1;             // tiles per worker
    const int tile_w = per_worker ? (int)blockIdx.x / tpw : 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < kMlpTile) {
        int64_t slot;
        if (per_worker) {
            const int j = ((int)blockIdx.x % tpw) * kMlpTile + (int)threadIdx.x;
            slot = j < B ? (int64_t)tile_w * B + j : -1;
        } else {
            slot = (int64_t)blockIdx.x * kMlpTile + threadIdx.x;
        }
        int64_t a = -1;
        if (slot >= 0 && slot < nslots) {
            a = B > 0 ? batch_row(bs, K, (int)(slot / B), (int)(slot % B), B, blockIdx.y == 0) : slot;   // B = 0: row = slot
            if (row_of_slot && blockIdx.y == 0) row_of_slot[slot] = (int32_t)a;
        } else {
            slot = -1;
        }
        s_row[threadIdx.x] = a; s_slot[threadIdx.x] = slot;
    }
    __syncthreads();
    if (per_worker && xa) xa = diff_of_worker(bs, xa, tile_w);
    const int j0 = blockIdx.y * 8;
    const int kk = lane & 3, rn = lane >> 2;             // this lane's k of A and B; its row of A / unit of B
    const int ju = j0 + rn;
    const bool unit_ok = ju < sh.hidden;
    const int in = (int)sh.in;
    const float* wa = (xa && unit_ok) ? xa + (int64_t)ju * in : nullptr;
    const float* wb = (xb && unit_ok) ? xb + (int64_t)ju * in : nullptr;
    const float* arow0 = s_row[rn] >= 0 ? X + s_row[rn] * in : nullptr;
    const float* arow1 = s_row[8 + rn] >= 0 ? X + s_row[8 + rn] * in : nullptr;
    double d[2][2][2];                                   // [row tile][model][pair]
#pragma unroll
    for (int q = 0; q < 8; ++q) (&d[0][0][0])[q] = 0.0;
    const int nchunk = (in + 15) >> 4;
    constexpr int W = kThreads / 32;
    for (int c0 = warp; c0 < nchunk; c0 += W * kMlpBatch) {
        float4 fa0[kMlpBatch], fa1[kMlpBatch], fwa[kMlpBatch], fwb[kMlpBatch];
#pragma unroll
        for (int u = 0; u < kMlpBatch; ++u) {
            const int i = ((c0 + u * W) << 4) + (kk << 2);   // beyond the last chunk i >= in: zeros
            fa0[u] = mlp_load4<VEC>(arow0, i, in);
            fa1[u] = mlp_load4<VEC>(arow1, i, in);
            fwa[u] = mlp_load4<VEC>(wa, i, in);
            fwb[u] = mlp_load4<VEC>(wb, i, in);
        }
#pragma unroll
        for (int u = 0; u < kMlpBatch; ++u) {
            if (c0 + u * W >= nchunk) break;             // (the same for the whole warp)
            const float a0[4] = {fa0[u].x, fa0[u].y, fa0[u].z, fa0[u].w}, a1[4] = {fa1[u].x, fa1[u].y, fa1[u].z, fa1[u].w};
            const float ba[4] = {fwa[u].x, fwa[u].y, fwa[u].z, fwa[u].w}, bb[4] = {fwb[u].x, fwb[u].y, fwb[u].z, fwb[u].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                dmma_8x8x4(d[0][0][0], d[0][0][1], (double)a0[e], (double)ba[e]);
                dmma_8x8x4(d[0][1][0], d[0][1][1], (double)a0[e], (double)bb[e]);
                dmma_8x8x4(d[1][0][0], d[1][0][1], (double)a1[e], (double)ba[e]);
                dmma_8x8x4(d[1][1][0], d[1][1][1], (double)a1[e], (double)bb[e]);
            }
        }
    }
#pragma unroll
    for (int rt = 0; rt < 2; ++rt)
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            s_red[warp][m][(rt * 8 + rn) * 8 + kk * 2] = d[rt][m][0];
            s_red[warp][m][(rt * 8 + rn) * 8 + kk * 2 + 1] = d[rt][m][1];
        }
    __syncthreads();
    for (int q = threadIdx.x; q < 2 * kMlpTile * 8; q += blockDim.x) {
        const int model = q / (kMlpTile * 8), e = q % (kMlpTile * 8), t = e >> 3, u = e & 7;
        const float* xm = model == 0 ? xa : xb;
        double* act = model == 0 ? act_a : act_b;
        if (xm && j0 + u < sh.hidden && s_slot[t] >= 0) {
            double v = 0.0;
#pragma unroll
            for (int k = 0; k < kThreads / 32; ++k) v += s_red[k][model][e];
            act[s_slot[t] * sh.hidden + j0 + u] = fmax(v + (double)xm[mlp_off_b1(sh) + j0 + u], 0.0);
        }
    }
}

// Block per sampled row, both parameter vectors side by side: logits (a warp per (model, class)), softmax,
// dz = (p - onehot) * wgt, dh_j = relu'(h_j) sum_c dz_c W2[c][j], and the loss of model b.  One thread per
// (model, class) takes the exponential; every sum runs in class order.  p_label - 1 is formed as -others / sum
// (the sum without the label's term), which has no cancellation.
__global__ void __launch_bounds__(kThreads)
mlp_output_kernel(MlpShape sh, const float* __restrict__ labels, const int32_t* __restrict__ row_of_slot,
                  const float* xa, const float* __restrict__ xb, const double* __restrict__ act_a,
                  const double* __restrict__ act_b, double wgt, float* __restrict__ dz_a, float* __restrict__ dz_b,
                  float* __restrict__ dh_a, float* __restrict__ dh_b, double* __restrict__ loss_b, int staged,
                  int B, const int32_t* __restrict__ a_slot, int64_t a_stride /* lagging workers: model a of worker slot / B sits in ring slot a_slot[.] */)
{
    pdl_prologue();
    if (a_slot && xa) xa += (int64_t)a_slot[blockIdx.x / B] * a_stride;
    extern __shared__ double s_zd[];     // [2 models][logits, exponentials, dz][classes], [2][hidden] activations, staged: [2][W2, b2]
    const int C = sh.classes, H = sh.hidden;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t slot = blockIdx.x;
    const int label = (int)labels[row_of_slot[slot]];
    double* s_act = s_zd + 6 * C;
    float* s_w2 = reinterpret_cast<float*>(s_act + 2 * H);
    const int nw2 = C * H + C;                           // W2 and b2 are adjacent in the parameter vector
    if (staged) {
        for (int q0 = threadIdx.x; q0 < 2 * nw2; q0 += 8 * kThreads) {      // eight loads in flight per thread
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int q = q0 + u * kThreads, m = q >= nw2;
                const float* x = m ? xb : xa;
                v[u] = (x && q < 2 * nw2) ? __ldg(x + mlp_off_w2(sh) + (q - m * nw2)) : 0.0f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) if (q0 + u * kThreads < 2 * nw2) s_w2[q0 + u * kThreads] = v[u];
        }
    }
    for (int q = threadIdx.x; q < 2 * H; q += blockDim.x) {
        const int m = q >= H, j = q - m * H;
        const double* act = m ? act_b : act_a;
        s_act[q] = ((m ? xb : xa) && act) ? act[slot * H + j] : 0.0;
    }
    __syncthreads();
    for (int q = warp; q < 2 * C; q += kThreads / 32) {
        const int m = q >= C, c = q - m * C;
        const float* x = m ? xb : xa;
        if (!x) continue;
        const float* w2 = staged ? s_w2 + m * nw2 : x + mlp_off_w2(sh);
        const float* wrow = w2 + (int64_t)c * H;
        const double* act = s_act + m * H;
        double s = 0.0;
#pragma unroll 4
        for (int j = lane; j < H; j += 32) s = fma((double)wrow[j], act[j], s);
        s = warp_sum(s);
        if (lane == 0) s_zd[m * 3 * C + c] = s + (double)w2[(int64_t)C * H + c];
    }
    __syncthreads();
    for (int q = threadIdx.x; q < 2 * C; q += blockDim.x) {
        const int m = q >= C, c = q - m * C;
        if (!(m ? xb : xa)) continue;
        const double* z = s_zd + m * 3 * C;
        double zmax = -INFINITY;
        for (int cc = 0; cc < C; ++cc) zmax = fmax(zmax, z[cc]);
        s_zd[m * 3 * C + C + c] = exp(z[c] - zmax);
    }
    __syncthreads();
    for (int q = threadIdx.x; q < 2 * C; q += blockDim.x) {
        const int m = q >= C, c = q - m * C;
        if (!(m ? xb : xa)) continue;
        const double* z = s_zd + m * 3 * C;
        const double* e = z + C;
        double sum = 0.0, others = 0.0;
        for (int cc = 0; cc < C; ++cc) { sum += e[cc]; if (cc != label) others += e[cc]; }
        const double v = (c == label ? -others / sum : e[c] / sum) * wgt;
        s_zd[m * 3 * C + 2 * C + c] = v;
        float* dz = m ? dz_b : dz_a;
        if (dz) dz[slot * C + c] = (float)v;
        if (m && c == 0 && loss_b) {
            double zmax = -INFINITY;
            for (int cc = 0; cc < C; ++cc) zmax = fmax(zmax, z[cc]);
            atomicAdd(loss_b, ((zmax + log(sum)) - z[label]) * wgt);
        }
    }
    __syncthreads();
    for (int q = threadIdx.x; q < 2 * H; q += blockDim.x) {
        const int m = q >= H, j = q - m * H;
        const float* x = m ? xb : xa;
        float* dh = m ? dh_b : dh_a;
        if (!x || !dh) continue;
        const double* dzs = s_zd + m * 3 * C + 2 * C;
        const float* wcol = (staged ? s_w2 + m * nw2 : x + mlp_off_w2(sh)) + j;
        double s = 0.0;
#pragma unroll 10
        for (int c = 0; c < C; ++c) s = fma(dzs[c], (double)wcol[(int64_t)c * H], s);
        dh[slot * H + j] = s_act[q] > 0.0 ? (float)s : 0.0f;
    }
}

// grid (ceil(hidden / kMlpUnits) + ceil(classes (hidden + 1) / threads), groups): block (j, w) sums over the rows
// [w*B, (w+1)*B) of its group, in slot order and in double.  The first ceil(hidden / kMlpUnits) blocks: rows
// j0 .. j0 + kMlpUnits - 1 of W1 and their b1; the blocks after them: W2 and b2, an entry per thread.
// Output = model a minus model b (either may be absent).  FULL: sums added to g64 with atomics (epoch gradient over
// many groups); otherwise rounded once and stored to out [groups][P] with the norm folded in.
template <bool FULL, bool VEC>
__global__ void __launch_bounds__(kThreads)
mlp_param_kernel(const float* __restrict__ X, MlpShape sh, const int32_t* __restrict__ row_of_slot, int B, int64_t total_rows,
                 const double* __restrict__ act_a, const double* __restrict__ act_b, const float* __restrict__ dz_a,
                 const float* __restrict__ dz_b, const float* __restrict__ dh_a, const float* __restrict__ dh_b,
                 float* __restrict__ out, int64_t P, uint32_t* __restrict__ norm_bits, double* __restrict__ g64)
{
    pdl_prologue();
    constexpr int kTiles = 13, W = kThreads / 32, kPassIn = W * kTiles * 8, kR = 8;
    constexpr int kStage = (kR * (kPassIn / 4) + kThreads - 1) / kThreads;     // 16-byte groups a thread stages per eight rows
    __shared__ __align__(16) float s_x[kR][kPassIn + 8]; // features of eight rows, the inputs of the current pass (+8: bank spread)
    __shared__ double s_w[kMlpUnits][kR];                // slope differences of those rows
    __shared__ int s_rowid[kMlpRowChunk];
    const int j0 = blockIdx.x * kMlpUnits, w = blockIdx.y;     // the blocks after the last tile of hidden units do W2, b2
    const int64_t r0 = (int64_t)w * B;
    const int nrows = (int)min((int64_t)B, total_rows - r0);
    uint32_t nmax = 0;
    float* o = FULL ? nullptr : out + (int64_t)w * P;
    if (j0 < sh.hidden) {
        // First-layer gradient of eight hidden units as 8x8 fp64 tensor-core tiles: D[unit][input] += sum_r A[unit][r] B[r][input]
        // with A[u][r] = dh_a[r][j0 + u] - dh_b[r][j0 + u] and B[r][i] = feature i of row r, both staged in shared memory
        // eight rows at a time (the rows with 16-byte loads by the whole block).  Tiles of eight inputs are dealt to the
        // warps round robin, kTiles per warp and pass (8 * 13 tiles cover the 784 inputs of the image workloads in one
        // pass); a warp keeps its tiles' sums across the rows.  Rows enter in slot order.
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const int kk = lane & 3, un = lane >> 2;             // this lane's k (row of the chunk) of A and B; its unit of A / input of B
        const int in = (int)sh.in, ntile = (in + 7) >> 3;
        double bias = 0.0;                                   // thread u < 8: d loss / d b1[j0 + u]
        for (int in0 = 0; in0 < in; in0 += kPassIn) {
            const int tile0 = in0 >> 3;
            const int nv = ((min(kPassIn, in - in0) + 7) >> 3) << 1;     // 16-byte groups per staged row
            double acc[kTiles][2];
#pragma unroll
            for (int t = 0; t < kTiles; ++t) { acc[t][0] = 0.0; acc[t][1] = 0.0; }
            for (int c0 = 0; c0 < nrows; c0 += kMlpRowChunk) {
                const int cn = min(kMlpRowChunk, nrows - c0);
                __syncthreads();
                for (int r = threadIdx.x; r < cn; r += blockDim.x) s_rowid[r] = row_of_slot[r0 + c0 + r];
                __syncthreads();
                // eight rows at a time; the loads of the next eight are in flight while these are multiplied
                float4 buf[kStage]; float wa = 0.0f, wb = 0.0f;
                auto fetch = [&](int c1) {
                    const int rn = min(kR, cn - c1);
#pragma unroll
                    for (int it = 0; it < kStage; ++it) {
                        const int q = threadIdx.x + it * kThreads, r = q / nv, v = q - r * nv;
                        const float* xr = r < rn ? X + (int64_t)s_rowid[c1 + min(r, rn - 1)] * in : nullptr;
                        buf[it] = mlp_load4<VEC>(xr, in0 + 4 * v, in);     // (rows beyond the chunk: zeros)
                    }
                    if (threadIdx.x < kMlpUnits * kR) {
                        const int u = threadIdx.x / kR, r = threadIdx.x % kR, j = j0 + u;
                        const bool ok = r < rn && j < sh.hidden;
                        wa = (dh_a && ok) ? dh_a[(r0 + c0 + c1 + r) * sh.hidden + j] : 0.0f;
                        wb = (dh_b && ok) ? dh_b[(r0 + c0 + c1 + r) * sh.hidden + j] : 0.0f;
                    }
                };
                fetch(0);
                for (int c1 = 0; c1 < cn; c1 += kR) {
                    const int rn = min(kR, cn - c1);
                    if (c1) __syncthreads();                 // the previous eight rows have been used
#pragma unroll
                    for (int it = 0; it < kStage; ++it) {
                        const int q = threadIdx.x + it * kThreads, r = q / nv, v = q - r * nv;
                        if (r < kR) *reinterpret_cast<float4*>(&s_x[r][4 * v]) = buf[it];
                    }
                    if (threadIdx.x < kMlpUnits * kR) s_w[threadIdx.x / kR][threadIdx.x % kR] = (double)wa - (double)wb;   // zero beyond the last row
                    __syncthreads();
                    if (c1 + kR < cn) fetch(c1 + kR);
                    if (in0 == 0 && threadIdx.x < kMlpUnits) for (int r = 0; r < rn; ++r) bias += s_w[threadIdx.x][r];
#pragma unroll
                    for (int ks = 0; ks < kR / 4; ++ks) {
                        if (ks * 4 < rn) {
                            const int r = (ks << 2) + kk;
                            const double a = s_w[un][r];
#pragma unroll
                            for (int t = 0; t < kTiles; ++t)
                                if (tile0 + t * W + warp < ntile)                                  // (the same for the whole warp)
                                    dmma_8x8x4(acc[t][0], acc[t][1], a, (double)s_x[r][((t * W + warp) << 3) + un]);
                        }
                    }
                }
            }
#pragma unroll
            for (int t = 0; t < kTiles; ++t) {
                const int i0 = ((tile0 + t * W + warp) << 3) + kk * 2;                        // D[un][2 kk], D[un][2 kk + 1]
                const int j = j0 + un;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    if (j < sh.hidden && i0 + e < in) {
                        const int64_t pidx = (int64_t)j * in + i0 + e;
                        if (FULL) atomicAdd(g64 + pidx, acc[t][e]);
                        else { o[pidx] = (float)acc[t][e]; nmax = max(nmax, __float_as_uint((float)acc[t][e]) & 0x7FFFFFFFu); }
                    }
                }
            }
        }
        if (threadIdx.x < kMlpUnits && j0 + (int)threadIdx.x < sh.hidden) {
            const int64_t pidx = mlp_off_b1(sh) + j0 + threadIdx.x;
            if (FULL) atomicAdd(g64 + pidx, bias);
            else { o[pidx] = (float)bias; nmax = max(nmax, __float_as_uint((float)bias) & 0x7FFFFFFFu); }
        }
    } else {
        const int nout = sh.classes * (sh.hidden + 1);                       // W2 entries then b2, one per thread
        const int t = (int)(blockIdx.x - (sh.hidden + kMlpUnits - 1) / kMlpUnits) * (int)blockDim.x + (int)threadIdx.x;
        if (t < nout) {
            const bool bias = t >= sh.classes * sh.hidden;
            const int c = bias ? t - sh.classes * sh.hidden : t / sh.hidden, jj = bias ? 0 : t % sh.hidden;
            double s = 0.0;
#pragma unroll 4
            for (int r = 0; r < nrows; ++r) {
                const int64_t q = r0 + r;
                // both products rounded on their own (no fused multiply-subtract): equal models cancel exactly
                const double ta = dz_a ? __dmul_rn((double)dz_a[q * sh.classes + c], bias ? 1.0 : act_a[q * sh.hidden + jj]) : 0.0;
                const double tb = dz_b ? __dmul_rn((double)dz_b[q * sh.classes + c], bias ? 1.0 : act_b[q * sh.hidden + jj]) : 0.0;
                s += ta - tb;
            }
            const int64_t pidx = bias ? mlp_off_b2(sh) + c : mlp_off_w2(sh) + (int64_t)c * sh.hidden + jj;
            if (FULL) atomicAdd(g64 + pidx, s);
            else { o[pidx] = (float)s; nmax = max(nmax, __float_as_uint((float)s) & 0x7FFFFFFFu); }
        }
    }
    if (!FULL) block_atomic_max(nmax, norm_bits + w);
}

// ---------------------------------------------------------------------------------------------------
// Whole rounds in one kernel for small problems.  A round of Algorithm 1 / 3 is a chain of dependent stages; as
// separate kernels each costs a launch gap of a few microseconds, which is all the time a problem of a few
// thousand coordinates needs.  Here one thread-block cluster of M blocks runs `nrounds` consecutive rounds.
// Block w IS worker w: it dequantises the broadcast model into its own shared memory (every block draws the same
// codes, so nothing has to be exchanged), computes its minibatch gradient alpha_w there, takes the norm,
// quantises and packs its message -- all behind block-level barriers only.  The blocks meet at the hardware
// cluster barrier (release/acquire at cluster scope) twice per round: before the master step, which all blocks
// share by coordinate range, and after it.  The arithmetic of every stage is that of the stand-alone kernels:
// same quantiser, same draws, same master update; the global buffers and their layouts are the same too.
// ---------------------------------------------------------------------------------------------------
struct SmallRound {
    // data
    const float* values; const int32_t* col; const int64_t* row_ptr; const float* labels; int64_t n;
    // problem
    int64_t d; int M, B, bx, b; ProxParams pp;
    // state
    float* x; float* y; float* xsum; const float* xsnap; const float* gfull; const float* zsnap; uint32_t* normx;
    // buffers of the round
    float* alpha; uint32_t* ninf; int32_t* rows; uint8_t* codes_x; float* delta_x; uint32_t* xnorm2 /* [2] scratch */;
    uint8_t* codes; int64_t stride; float* scale; uint64_t* bits_down; uint64_t* bits_up; int* status;
    // what to run
    uint32_t round0; int nrounds; float eta, theta;
    double acc_scale, acc_inv;      // CSR data: the integer grid of the gradient accumulator (see worker_grad_csr_kernel)
};

constexpr int kSmallThreads = 1024;
// A packed message is padded to 16 bytes, i.e. up to 64 coordinates at two bits: shared vectors carry that many zeros.
__host__ __device__ inline int64_t small_round_pad(int64_t d) { return ((d + 63) / 64 + 1) * 64; }

__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Block-wide maximum through shared memory; every thread gets the result.
__device__ __forceinline__ uint32_t small_block_max(uint32_t v, uint32_t* s_red)
{
    v = warp_max_u32(v);
    __syncthreads();                                          // s_red may still be in use by the previous reduction
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t t = (threadIdx.x & 31) < (blockDim.x >> 5) ? s_red[threadIdx.x & 31] : 0u;
    return warp_max_u32(t);
}

// Eight consecutive floats (16-byte aligned): from L2, through the read-only path, and the store.
__device__ __forceinline__ void small_load8_cg(const float* p, float (&v)[8])
{
    const float4 lo = __ldcg(reinterpret_cast<const float4*>(p)), hi = __ldcg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = lo.x; v[1] = lo.y; v[2] = lo.z; v[3] = lo.w; v[4] = hi.x; v[5] = hi.y; v[6] = hi.z; v[7] = hi.w;
}
__device__ __forceinline__ void small_load8_ro(const float* p, float (&v)[8])
{
    const float4 lo = __ldg(reinterpret_cast<const float4*>(p)), hi = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = lo.x; v[1] = lo.y; v[2] = lo.z; v[3] = lo.w; v[4] = hi.x; v[5] = hi.y; v[6] = hi.z; v[7] = hi.w;
}
__device__ __forceinline__ void small_store8(float* p, const float (&v)[8])
{
    reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}

// Q_(delta,b) of one vector held by this block (v in shared or global memory, read with plain loads when `shared`,
// else from L2), packed codes to `out` if not NULL; with `diff`, code * delta - ref goes to shared memory.
// Data that another block wrote earlier in the same launch is read with ld.global.cg: L2 is where the writes of
// all blocks meet, and the read-only path may serve stale lines for such data.
template <int BITS, bool SHARED_IN>
__device__ __forceinline__ void small_quantize(const float* v, int64_t d, uint32_t nb, uint8_t* out, float* scale_out,
                                               const PhiloxKeys& K, uint32_t round, uint32_t worker, uint32_t stream,
                                               int* status, const float* __restrict__ ref, float* diff)
{
    const int64_t ngroups = ((((d * BITS + 7) / 8) + 15) / 16 * 16) / BITS;       // covers the zero padding
    const float nrm = __uint_as_float(nb);
    const bool ok = nb < 0x7F800000u && nb != 0u;
    const float inv = ok ? __fdiv_rd((float)levels(BITS), nrm) : 0.0f;
    const float delta = ok ? __fdiv_rn(nrm, (float)levels(BITS)) : 0.0f;
    if (threadIdx.x == 0 && scale_out) { *scale_out = delta; if (nb >= 0x7F800000u) set_status(status, DQ_ERR_NONFINITE); }
    const bool al16 = (reinterpret_cast<uintptr_t>(v) & 15) == 0 && (!ref || (reinterpret_cast<uintptr_t>(ref) & 15) == 0);
    for (int64_t g = threadIdx.x; g < ngroups; g += blockDim.x) {
        float a[8];
        const int64_t i0 = g << 3;
        const bool whole = SHARED_IN || (al16 && i0 + 8 <= d);     // shared vectors are padded with zeros past d
        if (whole) {
            const float4 lo = SHARED_IN ? reinterpret_cast<const float4*>(v + i0)[0] : __ldcg(reinterpret_cast<const float4*>(v + i0));
            const float4 hi = SHARED_IN ? reinterpret_cast<const float4*>(v + i0)[1] : __ldcg(reinterpret_cast<const float4*>(v + i0) + 1);
            a[0] = lo.x; a[1] = lo.y; a[2] = lo.z; a[3] = lo.w; a[4] = hi.x; a[5] = hi.y; a[6] = hi.z; a[7] = hi.w;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) a[j] = (i0 + j < d) ? __ldcg(v + i0 + j) : 0.0f;
        }
        uint32_t r[4], s[8];
        philox4x32_10((uint32_t)g, round, worker, stream, K, r);
#pragma unroll
        for (int j = 0; j < 8; ++j) s[j] = round_fixed<BITS>(a[j], inv, half16(r, j));
        if (nb >= 0x7F800000u) {                               // NaN or Inf in the vector: every code is 0
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = 128u << 16;
        }
        if (out) store_group<BITS>(out + g * BITS, pack8<BITS>(s));
        if (diff) {                                            // diff is a padded shared vector
            float rf[8], o[8];
            if (whole) {
                const float4 lo = __ldg(reinterpret_cast<const float4*>(ref + i0)), hi = __ldg(reinterpret_cast<const float4*>(ref + i0) + 1);
                rf[0] = lo.x; rf[1] = lo.y; rf[2] = lo.z; rf[3] = lo.w; rf[4] = hi.x; rf[5] = hi.y; rf[6] = hi.z; rf[7] = hi.w;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) rf[j] = (i0 + j < d) ? ref[i0 + j] : 0.0f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) o[j] = (i0 + j < d) ? __fsub_rn(__fmul_rn((float)((int)((s[j] >> 16) & 0xFFu) - 128), delta), rf[j]) : 0.0f;
            reinterpret_cast<float4*>(diff + i0)[0] = make_float4(o[0], o[1], o[2], o[3]);
            reinterpret_cast<float4*>(diff + i0)[1] = make_float4(o[4], o[5], o[6], o[7]);
        }
    }
}

template <int FMT, bool ACC>
__global__ void __launch_bounds__(kSmallThreads, 1)
round_cluster_kernel(const __grid_constant__ SmallRound P, const __grid_constant__ PhiloxKeys K)
{
    pdl_prologue();
    extern __shared__ float s_mem[];
    __shared__ uint32_t s_red[32];
    __shared__ float s_scale[16];
    __shared__ float s_r[FMT == DQ_DENSE_F32 ? 1024 : 1];
    __shared__ int64_t s_rowi[FMT == DQ_DENSE_F32 ? 1024 : 1];
    const int64_t d = P.d; const int M = P.M, B = P.B;
    const int64_t dpad = small_round_pad(d);                  // room for the zero padding of a packed message
    float* s_diff = s_mem;                                    // [dpad] xhat - xsnap
    float* s_alpha = s_mem + dpad;                            // [dpad] this worker's gradient difference, zeros past d
    long long* s_acc = reinterpret_cast<long long*>(s_mem + 2 * dpad);   // [d] CSR data: exact integer accumulator (dpad is even: 8-byte aligned)
    const int w = blockIdx.x, lane = threadIdx.x & 31;
    const int64_t gtid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, gnth = (int64_t)gridDim.x * blockDim.x;
    for (int it = 0; it < P.nrounds; ++it) {
        const uint32_t round = P.round0 + (uint32_t)it;
        // ---- model: every block draws the same codes; block 0 also writes them out ---------------------------------
        const uint32_t* nsrc = it == 0 ? P.normx : P.xnorm2 + ((it - 1) & 1);
        const uint32_t nbx = __ldcg(nsrc);
        if (gtid == 0) P.xnorm2[it & 1] = 0u;                 // read last in the previous round, two barriers ago
        DQ_DISPATCH_BITS(P.bx, (small_quantize<BITS_, false>(P.x, d, nbx, w == 0 ? P.codes_x : nullptr, w == 0 ? P.delta_x : nullptr, K,
                                                              round, kMaster, kStreamModel, P.status, P.xsnap, s_diff)));
        for (int64_t i = d + threadIdx.x; i < dpad; i += blockDim.x) s_alpha[i] = 0.0f;
        if (FMT == DQ_CSR_F32) for (int64_t i = threadIdx.x; i < d; i += blockDim.x) s_acc[i] = 0;
        __syncthreads();
        // ---- worker w: slope differences of its sampled rows ------------------------------------------------------
        if (FMT == DQ_CSR_F32) {
            // sixteen lanes per row: a row of a text-like matrix has a few dozen nonzeros
            const int sub = threadIdx.x >> 4, nsub = blockDim.x >> 4, l16 = threadIdx.x & 15;
            const uint32_t submask = 0xFFFFu << (lane & 16);
            for (int j = sub; j < B; j += nsub) {
                const int64_t a = sample_row(K, round, w, j, M, P.n);
                if (l16 == 0) P.rows[(int64_t)w * B + j] = (int32_t)a;
                const int64_t k0 = P.row_ptr[a], k1 = P.row_ptr[a + 1];
                const float ya = P.labels[a], za = P.zsnap[a];
                double sdot = 0.0;
#pragma unroll 4
                for (int64_t k = k0 + l16; k < k1; k += 16) sdot += (double)__ldg(P.values + k) * (double)s_diff[__ldg(P.col + k)];
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) sdot += __shfl_xor_sync(submask, sdot, o);
                const float r = slope_difference(ya, za, (float)sdot) / (float)B;
                for (int64_t k = k0 + l16; k < k1; k += 16) fixed_add(s_acc + __ldg(P.col + k), r, __ldg(P.values + k), P.acc_scale);
            }
            __syncthreads();
            for (int64_t i = threadIdx.x; i < d; i += blockDim.x) s_alpha[i] = (float)((double)s_acc[i] * P.acc_inv);
            __syncthreads();
        } else {
            const bool vec = (d & 3) == 0;
            for (int j = threadIdx.x >> 5; j < B; j += (int)(blockDim.x >> 5)) {
                const int64_t a = sample_row(K, round, w, j, M, P.n);
                const float* row = P.values + a * d;
                const float ya = P.labels[a], za = P.zsnap[a];     // in flight together with the row
                float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
                if (vec) {
#pragma unroll 8
                    for (int64_t v = lane; v < (d >> 2); v += 32) {
                        const float4 f = __ldg(reinterpret_cast<const float4*>(row) + v), x4 = reinterpret_cast<const float4*>(s_diff)[v];
                        s0 = fmaf(f.x, x4.x, s0); s1 = fmaf(f.y, x4.y, s1); s2 = fmaf(f.z, x4.z, s2); s3 = fmaf(f.w, x4.w, s3);
                    }
                } else {
#pragma unroll 8
                    for (int64_t i = lane; i < d; i += 32) s0 = fmaf(__ldg(row + i), s_diff[i], s0);
                }
                const double dz = warp_sum(((double)s0 + (double)s1) + ((double)s2 + (double)s3));
                if (lane == 0) {
                    P.rows[(int64_t)w * B + j] = (int32_t)a;
                    s_r[j] = slope_difference(ya, za, (float)dz) / (float)B; s_rowi[j] = a;
                }
            }
            __syncthreads();
            // alpha_w[i] = sum_j r_j a_j[i], rows in slot order (no atomics: reproducible bit for bit)
            for (int64_t i = threadIdx.x; i < d; i += blockDim.x) {
                float acc = 0.0f;
#pragma unroll 16
                for (int j = 0; j < B; ++j) acc = fmaf(s_r[j], __ldg(P.values + s_rowi[j] * d + i), acc);
                s_alpha[i] = acc;
            }
            __syncthreads();
        }
        // ---- ||alpha_w||_inf, message w --------------------------------------------------------------------------------
        uint32_t m = 0;
        for (int64_t i = threadIdx.x; i < d; i += blockDim.x) {
            const float av = s_alpha[i];
            P.alpha[(int64_t)w * d + i] = av;
            m = max(m, __float_as_uint(av) & 0x7FFFFFFFu);
        }
        m = small_block_max(m, s_red);
        if (threadIdx.x == 0) P.ninf[w] = m;
        DQ_DISPATCH_BITS(P.b, (small_quantize<BITS_, true>(s_alpha, d, m, P.codes + (int64_t)w * P.stride, P.scale + w, K, round, (uint32_t)w,
                                                            kStreamGrad, P.status, nullptr, nullptr)));
        cluster_barrier();
        // ---- master step, groups of eight coordinates shared by all blocks -----------------------------------------------
        {
            if (threadIdx.x < M) s_scale[threadIdx.x] = __ldcg(P.scale + threadIdx.x);
            __syncthreads();
            const float inv_m = __fdiv_rn(1.0f, (float)M);
            const float thr = __fmul_rn(P.eta, P.pp.lambda1), den = __fadd_rn(1.0f, __fmul_rn(P.eta, P.pp.lambda2));
            const int b = P.b;
            const bool al16 = ((reinterpret_cast<uintptr_t>(P.x) | reinterpret_cast<uintptr_t>(P.gfull) | reinterpret_cast<uintptr_t>(P.y) |
                                reinterpret_cast<uintptr_t>(P.xsnap) | reinterpret_cast<uintptr_t>(P.xsum)) & 15) == 0;
            uint32_t nmax = 0;
            for (int64_t g = gtid; (g << 3) < d; g += gnth) {
                const int64_t i0 = g << 3;
                const bool whole = al16 && i0 + 8 <= d;
                float cur[8], gf[8], xs[8], sm[8], acc[8];
                float* tgt = ACC ? P.y : P.x;
                if (whole) {
                    small_load8_cg(tgt + i0, cur); small_load8_ro(P.gfull + i0, gf);
                    if (ACC) { small_load8_ro(P.xsnap + i0, xs); small_load8_cg(P.xsum + i0, sm); }
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const bool in = i0 + j < d;
                        cur[j] = in ? __ldcg(tgt + i0 + j) : 0.0f; gf[j] = in ? P.gfull[i0 + j] : 0.0f;
                        if (ACC) { xs[j] = in ? P.xsnap[i0 + j] : 0.0f; sm[j] = in ? __ldcg(P.xsum + i0 + j) : 0.0f; }
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) { acc[j] = 0.0f; if (!ACC) { xs[j] = 0.0f; sm[j] = 0.0f; } }
                // the group's codes are b bytes of every message
                for (int w0 = 0; w0 < M; w0 += 4) {
                    uint64_t cw[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint8_t* src = P.codes + (int64_t)min(w0 + k, M - 1) * P.stride + g * b;
                        cw[k] = b == 8 ? (uint64_t)__ldcg(reinterpret_cast<const unsigned long long*>(src))
                              : b == 4 ? (uint64_t)__ldcg(reinterpret_cast<const uint32_t*>(src))
                                       : (uint64_t)__ldcg(reinterpret_cast<const unsigned short*>(src));
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (w0 + k < M) {
                            const float sc = s_scale[w0 + k];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int code = (int)((int64_t)(cw[k] << (64 - b * (j + 1))) >> (64 - b));
                                acc[j] = __fmaf_rn((float)code, sc, acc[j]);
                            }
                        }
                    }
                }
                float xo[8], yo[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    xo[j] = master_update<ACC>(acc[j], inv_m, P.eta, P.theta, thr, den, P.pp, gf[j], cur[j], xs[j], yo[j], sm[j]);
                    if (i0 + j < d) nmax = max(nmax, __float_as_uint(xo[j]) & 0x7FFFFFFFu);
                }
                if (whole) {
                    small_store8(P.x + i0, xo);
                    if (ACC) { small_store8(P.y + i0, yo); small_store8(P.xsum + i0, sm); }
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (i0 + j < d) { P.x[i0 + j] = xo[j]; if (ACC) { P.y[i0 + j] = yo[j]; P.xsum[i0 + j] = sm[j]; } }
                    }
                }
            }
            nmax = small_block_max(nmax, s_red);
            if (threadIdx.x == 0 && nmax != 0u) atomicMax(P.xnorm2 + (it & 1), nmax);
            if (gtid == 0 && P.bits_down) {
                const BitsArgs ba = {P.bits_down, P.bits_up, nullptr, 0, 0, P.bx, P.b, nullptr};
                write_round_bits(ba, M, d);
            }
        }
        cluster_barrier();
    }
    if (gtid == 0 && P.nrounds > 0) *P.normx = __ldcg(P.xnorm2 + ((P.nrounds - 1) & 1));
}

// ---------------------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------------------
static inline int blocks_for(int64_t threads_needed, int sm_count, int per_sm = 8)
{
    int64_t need = (threads_needed + kThreads - 1) / kThreads, cap = (int64_t)sm_count * per_sm;
    if (need < 1) need = 1;
    return (int)(need < cap ? need : cap);
}

// ---- network launchers ------------------------------------------------------------------------------------
static MlpShape mlp_shape(const dq_ctx* ctx) { return MlpShape{ctx->data.d, ctx->cfg.hidden, ctx->cfg.classes}; }
static dim3 mlp_hidden_grid(int64_t nslots, const MlpShape& sh, int M = 0, int B = 0 /* both set: tiles of one worker each */)
{
    if (M > 0) return dim3((unsigned)(M * ((B + kMlpTile - 1) / kMlpTile)), (unsigned)((sh.hidden + 7) / 8));
    return dim3((unsigned)((nslots + kMlpTile - 1) / kMlpTile), (unsigned)((sh.hidden + kThreads / 32 - 1) / (kThreads / 32)));
}
constexpr int kMlpGroup = 256;      // rows per block of the epoch-gradient sums
static unsigned mlp_param_grid_x(const MlpShape& sh)
{
    return (unsigned)((sh.hidden + kMlpUnits - 1) / kMlpUnits + (sh.classes * (sh.hidden + 1) + kThreads - 1) / kThreads);
}
// Shared memory of mlp_output_kernel; *staged: both models' output layers fit beside the per-row scratch.
static size_t mlp_output_smem(const MlpShape& sh, int* staged)
{
    const size_t base = sizeof(double) * (6 * (size_t)sh.classes + 2 * (size_t)sh.hidden);
    const size_t w2 = sizeof(float) * 2 * ((size_t)sh.classes * sh.hidden + sh.classes);
    *staged = base + w2 <= 48u * 1024u;
    return base + (*staged ? w2 : 0);
}
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static void launch_mlp_hidden(dq_ctx* ctx, int64_t nslots, const MlpShape& sh, const float* xa, const float* xb, const BatchSource& bs,
                              int B, double* act_a, double* act_b, cudaStream_t st)
{
    const float* X = (const float*)ctx->data.values;
    // rows and weight rows on 16-byte boundaries; a lagging worker's parameters start slot * d floats into the ring
    const bool vec = sh.in % 4 == 0 && aligned16(X) && aligned16(xa) && aligned16(xb) && (!(B > 0 && bs.diff_slot) || bs.diff_stride % 4 == 0);
    const dim3 grid = (B > 0 && bs.diff_slot) ? mlp_hidden_grid(nslots, sh, (int)(nslots / B), B) : mlp_hidden_grid(nslots, sh);
    if (vec) launch_k(mlp_hidden_kernel<true>, grid, kThreads, 0, st, X, sh, xa, xb, ctx->keys, bs, B, ctx->mlp_rows, act_a, act_b, nslots);
    else launch_k(mlp_hidden_kernel<false>, grid, kThreads, 0, st, X, sh, xa, xb, ctx->keys, bs, B, ctx->mlp_rows, act_a, act_b, nslots);
}

// g <- (1/n) sum_i grad loss_i(x) over all rows (double sums), via the "a" slots of the activation buffers.
static void launch_mlp_full_grad(dq_ctx* ctx, const float* x, float* g, cudaStream_t st)
{
    const dq_data& D = ctx->data; const MlpShape sh = mlp_shape(ctx);
    const BatchSource none = {nullptr, nullptr, 0u, nullptr, 1, D.n, nullptr};
    const int64_t P = ctx->cfg.d;
    launch_mlp_hidden(ctx, D.n, sh, x, nullptr, none, 0, ctx->mlp_act[0], nullptr, st);
    int staged; const size_t osm = mlp_output_smem(sh, &staged);
    launch_k(mlp_output_kernel, (unsigned)D.n, kThreads, osm, st, sh, D.labels, ctx->mlp_rows, x, nullptr, ctx->mlp_act[0],
        nullptr, 1.0 / (double)D.n, ctx->mlp_dz[0], nullptr, ctx->mlp_dh[0], nullptr, nullptr, staged, 1, nullptr, 0);
    cudaMemsetAsync(ctx->g64, 0, sizeof(double) * P, st);
    dim3 grid(mlp_param_grid_x(sh), (unsigned)((D.n + kMlpGroup - 1) / kMlpGroup));
    if (sh.in % 4 == 0 && aligned16(D.values))
        launch_k(mlp_param_kernel<true, true>, grid, kThreads, 0, st, (const float*)D.values, sh, ctx->mlp_rows, kMlpGroup, D.n,
            ctx->mlp_act[0], nullptr, ctx->mlp_dz[0], nullptr, ctx->mlp_dh[0], nullptr, nullptr, P, nullptr, ctx->g64);
    else
        launch_k(mlp_param_kernel<true, false>, grid, kThreads, 0, st, (const float*)D.values, sh, ctx->mlp_rows, kMlpGroup, D.n,
            ctx->mlp_act[0], nullptr, ctx->mlp_dz[0], nullptr, ctx->mlp_dh[0], nullptr, nullptr, P, nullptr, ctx->g64);
    launch_k(finish_full_grad_kernel, blocks_for(P, ctx->sm_count), kThreads, 0, st, ctx->g64, P, 1.0, g);
    ctx->launches += 4;
}

// alpha_w = minibatch grad at xhat minus minibatch grad at xsnap, and ||alpha_w||_inf.
static void launch_mlp_worker_grad(dq_ctx* ctx, const float* xhat, const dq_state* s, const BatchSource& bs, float* alpha,
                                   float* norm_inf, cudaStream_t st)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data; const MlpShape sh = mlp_shape(ctx);
    const unsigned R = (unsigned)(c.M * c.B);
    uint32_t* nb = reinterpret_cast<uint32_t*>(norm_inf);
    launch_mlp_hidden(ctx, R, sh, xhat, s->x_snap, bs, c.B, ctx->mlp_act[0], ctx->mlp_act[1], st);
    int staged; const size_t osm = mlp_output_smem(sh, &staged);
    launch_k(mlp_output_kernel, R, kThreads, osm, st, sh, D.labels, ctx->mlp_rows, xhat, s->x_snap, ctx->mlp_act[0],
        ctx->mlp_act[1], 1.0 / (double)c.B, ctx->mlp_dz[0], ctx->mlp_dz[1], ctx->mlp_dh[0], ctx->mlp_dh[1], nullptr, staged, c.B, bs.diff_slot, bs.diff_stride);
    if (!ctx->ninf_zeroed) cudaMemsetAsync(nb, 0, sizeof(uint32_t) * c.M, st);
    dim3 grid(mlp_param_grid_x(sh), c.M);
    if (sh.in % 4 == 0 && aligned16(D.values))
        launch_k(mlp_param_kernel<false, true>, grid, kThreads, 0, st, (const float*)D.values, sh, ctx->mlp_rows, c.B, (int64_t)R,
            ctx->mlp_act[0], ctx->mlp_act[1], ctx->mlp_dz[0], ctx->mlp_dz[1], ctx->mlp_dh[0], ctx->mlp_dh[1], alpha, c.d, nb, nullptr);
    else
        launch_k(mlp_param_kernel<false, false>, grid, kThreads, 0, st, (const float*)D.values, sh, ctx->mlp_rows, c.B, (int64_t)R,
            ctx->mlp_act[0], ctx->mlp_act[1], ctx->mlp_dz[0], ctx->mlp_dz[1], ctx->mlp_dh[0], ctx->mlp_dh[1], alpha, c.d, nb, nullptr);
    ctx->launches += 3;
}

void launch_epoch_begin(dq_ctx* ctx, dq_state* s, float theta, cudaStream_t st)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    uint32_t* nx = reinterpret_cast<uint32_t*>(s->norm_x);
    cudaMemsetAsync(nx, 0, sizeof(uint32_t), st);
    launch_k(epoch_state_kernel, blocks_for(c.d, ctx->sm_count), kThreads, 0, st, s->x, s->x_snap, s->y, s->x_sum, c.d, c.accelerated,
                                                                            ctx->ticks_in_epoch, theta, nx);
    if (c.model == DQ_MODEL_MLP) { launch_mlp_full_grad(ctx, s->x_snap, s->g_full, st); ctx->launches += 1; return; }
    cudaMemsetAsync(ctx->g64, 0, sizeof(double) * c.d, st);
    if (D.format == DQ_CSR_F32) {
        launch_k(full_grad_csr_kernel, blocks_for(D.n * 32, ctx->sm_count), kThreads, 0, st, (const float*)D.values, D.col_idx, D.row_ptr, D.labels, s->x_snap, D.n, s->z_snap, ctx->g64);
    } else {
        const int64_t nblk = (D.n + kRowsPerBlock - 1) / kRowsPerBlock;
        const int grid = (int)(nblk < (int64_t)ctx->sm_count * 8 ? nblk : (int64_t)ctx->sm_count * 8);
        const bool f32 = D.format == DQ_DENSE_F32;
        const bool vec = (D.d % (f32 ? 4 : 8)) == 0;
        if (f32 && vec)
            launch_k(full_grad_dense_vec_kernel<float>, grid, kThreads, 0, st, (const float*)D.values, D.labels, s->x_snap, D.n, D.d, s->z_snap, ctx->g64);
        else if (f32)
            launch_k(full_grad_dense_kernel<float>, grid, kThreads, 0, st, (const float*)D.values, D.labels, s->x_snap, D.n, D.d, s->z_snap, ctx->g64);
        else if (vec)
            launch_k(full_grad_dense_vec_kernel<__nv_bfloat16>, grid, kThreads, 0, st, (const __nv_bfloat16*)D.values, D.labels, s->x_snap, D.n, D.d, s->z_snap, ctx->g64);
        else
            launch_k(full_grad_dense_kernel<__nv_bfloat16>, grid, kThreads, 0, st, (const __nv_bfloat16*)D.values, D.labels, s->x_snap, D.n, D.d, s->z_snap, ctx->g64);
    }
    launch_k(finish_full_grad_kernel, blocks_for(c.d, ctx->sm_count), kThreads, 0, st, ctx->g64, c.d, 1.0 / (double)D.n, s->g_full);
    ctx->launches += 3;
}

// The one-pass kernel takes dense rows of at most kFusedMaxRowBytes on the 16-byte grid; the context then owns its
// scratch (column sums per (block, worker), per-worker counters).
// bfloat16 rows whose length is a multiple of 16 can take a tensor-core variant (cfg.tensor_cores: 1 both products, 2 the margins)
static int fused_grad_mode(const dq_ctx* ctx)
{
    if (ctx->data.format != DQ_DENSE_BF16 || (ctx->cfg.d & 15) != 0) return 0;
    return ctx->cfg.tensor_cores == 1 ? 1 : ctx->cfg.tensor_cores == 2 ? 2 : 0;
}
static bool fused_grad_mma(const dq_ctx* ctx) { return fused_grad_mode(ctx) != 0; }
static size_t fused_grad_smem(const dq_ctx* ctx)
{
    const size_t row_bytes = (size_t)ctx->cfg.d * (ctx->data.format == DQ_DENSE_F32 ? 4 : 2);
    return (size_t)kFusedStages * kFusedRows * (row_bytes + kFusedRowPad) + (fused_grad_mma(ctx) ? 3 * row_bytes : 0);
}
bool fused_grad_applies(const dq_ctx* ctx) { return ctx->fused_part != nullptr && ctx->cfg.no_fused != 1; }
typedef void (*FusedKernelF32)(const float*, const float*, const float*, const float*, const PhiloxKeys, BatchSource, FusedPlan, int64_t,
                               float*, uint32_t*, float*, uint32_t*, int*, const FusedRound);
typedef void (*FusedKernelBf16)(const __nv_bfloat16*, const float*, const float*, const float*, const PhiloxKeys, BatchSource, FusedPlan,
                                int64_t, float*, uint32_t*, float*, uint32_t*, int*, const FusedRound);
static FusedKernelBf16 fused_kernel_bf16(const dq_ctx* ctx)
{
    const int mode = fused_grad_mode(ctx);
    return mode == 1 ? worker_grad_fused_kernel<__nv_bfloat16, 1> : mode == 2 ? worker_grad_fused_kernel<__nv_bfloat16, 2> : worker_grad_fused_kernel<__nv_bfloat16, 0>;
}

static FusedPlan fused_plan(const dq_ctx* ctx)
{
    const dq_config& c = ctx->cfg;
    FusedPlan pl;
    pl.M = c.M; pl.B = c.B; pl.tiles_per_worker = (c.B + kFusedRows - 1) / kFusedRows;
    pl.ntiles = c.M * pl.tiles_per_worker; pl.nblocks = pl.ntiles < ctx->sm_count ? pl.ntiles : ctx->sm_count;
    return pl;
}

static void launch_fused(dq_ctx* ctx, const BatchSource& bs, const dq_state* s, float* alpha, uint32_t* nb, const FusedRound& fr, cudaStream_t st)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    const FusedPlan pl = fused_plan(ctx);
    const size_t smem = fused_grad_smem(ctx);
    if (D.format == DQ_DENSE_F32)
        launch_k(worker_grad_fused_kernel<float, 0>, pl.nblocks, kFusedThreads, smem, st, (const float*)D.values, D.labels, ctx->xhat_diff,
                 s->z_snap, ctx->keys, bs, pl, c.d, alpha, nb, ctx->fused_part, ctx->fused_cnt, ctx->status, fr);
    else
        launch_k(fused_kernel_bf16(ctx), pl.nblocks, kFusedThreads, smem, st, (const __nv_bfloat16*)D.values, D.labels,
                 ctx->xhat_diff, s->z_snap, ctx->keys, bs, pl, c.d, alpha, nb, ctx->fused_part, ctx->fused_cnt, ctx->status, fr);
    ctx->launches += 1;
}

// Model quantiser and message quantiser inside the gradient kernel: dense rows that take the one-pass kernel, dense
// messages, a fixed model width of 2, 4 or 8 bits, no lagging workers.  (The master step follows as its own kernel.)
bool fused_round_applies(const dq_ctx* ctx)
{
    const dq_config& c = ctx->cfg;
    if (!ctx->fused_part || c.no_fused || c.sparsify || c.mu > 0.0f || c.max_delay > 0 || c.B < 64) return false;
    if (c.bx != 2 && c.bx != 4 && c.bx != 8) return false;
    const int64_t elt = ctx->data.format == DQ_DENSE_F32 ? 4 : 8;
    return (c.d % elt) == 0;
}

void launch_fused_round(dq_ctx* ctx, dq_state* s, uint32_t round, cudaStream_t st)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    const BatchSource bs = {nullptr, ctx->rows, round, ctx->rp_active, c.M, D.n, nullptr, nullptr, c.d};
    FusedRound fr = {};
    fr.fold = 1;
    fr.normx_in = reinterpret_cast<const uint32_t*>(s->norm_x); fr.codes_x = ctx->codes_x; fr.delta_x = ctx->delta_x; fr.bx = c.bx;
    fr.b = c.b; fr.codes = ctx->msgs.codes; fr.stride = ctx->msgs.stride; fr.scale = ctx->msgs.scale;
    fr.x = s->x; fr.xsnap = s->x_snap;
    fr.normx_out = reinterpret_cast<uint32_t*>(s->norm_x); fr.done = ctx->fused_done;
    launch_fused(ctx, bs, s, ctx->alpha, reinterpret_cast<uint32_t*>(ctx->ninf), fr, st);
}

// Called once per context: scratch and the shared-memory opt-in of the one-pass dense gradient kernel.
int fused_grad_setup(dq_ctx* ctx)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    if (!ctx->has_data || c.model != DQ_MODEL_LOGISTIC || (D.format != DQ_DENSE_F32 && D.format != DQ_DENSE_BF16)) return DQ_OK;
    const size_t row_bytes = (size_t)c.d * (D.format == DQ_DENSE_F32 ? 4 : 2);
    if (row_bytes > kFusedMaxRowBytes || (row_bytes & 15) || c.B < 64) return DQ_OK;
    if ((int64_t)c.M * ((c.B + kFusedRows - 1) / kFusedRows) > ((int64_t)1 << 24)) return DQ_OK;    // the tile arithmetic is 32-bit
    const int smem = (int)fused_grad_smem(ctx);
    const FusedKernelF32 kf = worker_grad_fused_kernel<float, 0>;
    const FusedKernelBf16 kb = fused_kernel_bf16(ctx);
    const cudaError_t e = D.format == DQ_DENSE_F32 ? cudaFuncSetAttribute(kf, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                                                   : cudaFuncSetAttribute(kb, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) { cudaGetLastError(); return DQ_OK; }          // the two-kernel path remains
    int resident = 0;                                                    // a block must fit an SM (registers, shared memory)
    const cudaError_t o = D.format == DQ_DENSE_F32 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kf, kFusedThreads, (size_t)smem)
                                                   : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kb, kFusedThreads, (size_t)smem);
    if (o != cudaSuccess || resident < 1) { cudaGetLastError(); return DQ_OK; }
    if (cudaMalloc(reinterpret_cast<void**>(&ctx->fused_part), sizeof(float) * (size_t)(ctx->sm_count + c.M) * c.d) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&ctx->fused_cnt), sizeof(uint32_t) * (c.M + 1)) != cudaSuccess ||
        cudaMemset(ctx->fused_cnt, 0, sizeof(uint32_t) * (c.M + 1)) != cudaSuccess) return DQ_ERR_CUDA;
    ctx->fused_done = ctx->fused_cnt + c.M;
    return DQ_OK;
}

// Whether the worker stage accumulates into alpha with atomics (and so needs it cleared first).
bool worker_accumulates(const dq_ctx* ctx)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    (void)c; (void)D;
    return false;      // every gradient kernel stores alpha: CSR rows meet in an integer accumulator that is kept all-zero between rounds
}

void launch_worker_grad(dq_ctx* ctx, const uint8_t* codes_x, const float* delta_x, int is_snapshot, const dq_state* s,
                        uint32_t round, const int32_t* batch_idx, float* alpha, float* norm_inf, cudaStream_t st)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    const bool list = ctx->list_mode && alpha == ctx->alpha;   // sparse gradients tracked as a list of touched groups
    if (is_snapshot) {                     // xhat = xsnap: every slope difference is exactly zero
        cudaMemsetAsync(alpha, 0, sizeof(float) * c.M * c.d, st);
        cudaMemsetAsync(norm_inf, 0, sizeof(float) * c.M, st);
        if (list) cudaMemsetAsync(ctx->gcount, 0, sizeof(uint32_t) * c.M, st);
        if (list && ctx->ptouched) cudaMemsetAsync(ctx->ptouched, 0, sizeof(uint32_t) * c.M * ctx->bm_words, st);
        return;
    }
    if (list && !ctx->defer_list) launch_clear_listed(ctx, st);  // alpha is all-zero again before this round adds to it
    const BatchSource bs = {batch_idx, batch_idx ? nullptr : ctx->rows, round, ctx->rp_active, c.M, D.n,
                            ctx->normx_zeroed ? reinterpret_cast<uint32_t*>(s->norm_x) : nullptr,
                            ctx->use_slots ? ctx->slots_dev : nullptr, c.d};
    if (!ctx->diff_ready && c.bx != 2 && c.bx != 4 && c.bx != 8) {
        launch_dequant_diff_any(ctx, codes_x, delta_x, c.model == DQ_MODEL_MLP ? nullptr : s->x_snap, ctx->xhat_diff, c.bx, st);
    } else if (!ctx->diff_ready) {
        DQ_DISPATCH_BITS(c.bx, (launch_k(dequant_diff_kernel<BITS_>, blocks_for(c.d, ctx->sm_count), kThreads, 0, st, codes_x, delta_x, c.model == DQ_MODEL_MLP ? nullptr : s->x_snap, c.d, ctx->xhat_diff)));
        ctx->launches += 1;
    }
    if (c.model == DQ_MODEL_MLP) {        // xhat_diff holds xhat itself for the network (no reference subtracted)
        launch_mlp_worker_grad(ctx, ctx->xhat_diff, s, bs, alpha, norm_inf, st);
        return;
    }
    if (D.format == DQ_CSR_F32) {
        const FixedAcc fa = {ctx->acc64, ctx->acc_scale, ctx->acc_inv};
        launch_k(worker_grad_csr_kernel, (int)(((int64_t)c.M * c.B * 32 + kThreads - 1) / kThreads), kThreads, 0, st, (const float*)D.values, D.col_idx, D.row_ptr, D.labels, ctx->xhat_diff, s->z_snap, ctx->keys, bs, c.M, c.B, c.d, fa,
            list ? ctx->touched : nullptr, ctx->bm_words);
        ctx->launches += 1;
        if (list && ctx->defer_list) return;                 // the message kernel turns bitmap and accumulator into list, alpha and norm
        if (list) { launch_build_group_list(ctx, reinterpret_cast<uint32_t*>(norm_inf), st); ctx->list_ready = true; return; }
        uint32_t* nb = reinterpret_cast<uint32_t*>(norm_inf);
        if (!ctx->ninf_zeroed) cudaMemsetAsync(nb, 0, sizeof(uint32_t) * c.M, st);
        dim3 gc((unsigned)blocks_for(c.d, ctx->sm_count, 2), c.M);
        launch_k(acc_to_alpha_kernel, gc, kThreads, 0, st, fa, c.d, alpha, nb);
        ctx->launches += 1;
        return;
    } else {
        dim3 grid(1, c.M);
        const bool f32 = D.format == DQ_DENSE_F32;
        const bool vec = (c.d % (f32 ? 4 : 8)) == 0 && (reinterpret_cast<uintptr_t>(alpha) & 15) == 0;   // data is 16-byte aligned by contract
        if (vec && c.B >= 64 && fused_grad_applies(ctx)) {      // large minibatch, rows that fit a stage: one pass over the rows
            FusedRound fr = {};                                   // the gradient stage alone
            launch_fused(ctx, bs, s, alpha, reinterpret_cast<uint32_t*>(norm_inf), fr, st);
            return;
        }
        if (vec && c.B >= 64) {        // large minibatch, long rows: margins, then atomics-free column sums with the norm folded in
            const int32_t* rows_eff = batch_idx ? batch_idx : ctx->rows;
            uint32_t* nb = reinterpret_cast<uint32_t*>(norm_inf);
            if (!ctx->ninf_zeroed) cudaMemsetAsync(nb, 0, sizeof(uint32_t) * c.M, st);
            const int gm = (int)(((int64_t)c.M * c.B * 32 + kThreads - 1) / kThreads);
            const size_t smem = sizeof(float) * 2 * c.B;
            if (f32) {
                launch_k(worker_margins_kernel<float>, gm, kThreads, 0, st, (const float*)D.values, D.labels, ctx->xhat_diff, s->z_snap,
                                                                       ctx->keys, bs, c.M, c.B, c.d, ctx->rbuf);
                dim3 gc((unsigned)((c.d / 4 + 31) / 32), c.M);
                launch_k(worker_colsum_kernel<float>, gc, kThreads, smem, st, (const float*)D.values, rows_eff, ctx->rbuf, c.B, c.d, alpha, nb);
            } else {
                launch_k(worker_margins_kernel<__nv_bfloat16>, gm, kThreads, 0, st, (const __nv_bfloat16*)D.values, D.labels, ctx->xhat_diff,
                                                                               s->z_snap, ctx->keys, bs, c.M, c.B, c.d, ctx->rbuf);
                dim3 gc((unsigned)((c.d / 8 + 31) / 32), c.M);
                launch_k(worker_colsum_kernel<__nv_bfloat16>, gc, kThreads, smem, st, (const __nv_bfloat16*)D.values, rows_eff, ctx->rbuf, c.B,
                                                                                 c.d, alpha, nb);
            }
            ctx->launches += 2;
            return;
        } else if (f32 && vec)
            launch_k(worker_grad_dense_vec_kernel<float>, grid, kThreads, 0, st, (const float*)D.values, D.labels, ctx->xhat_diff, s->z_snap, ctx->keys, bs, c.B, c.d, alpha);
        else if (f32)
            launch_k(worker_grad_dense_kernel<float>, grid, kThreads, 0, st, (const float*)D.values, D.labels, ctx->xhat_diff, s->z_snap, ctx->keys, bs, c.B, c.d, alpha);
        else if (vec)
            launch_k(worker_grad_dense_vec_kernel<__nv_bfloat16>, grid, kThreads, 0, st, (const __nv_bfloat16*)D.values, D.labels, ctx->xhat_diff, s->z_snap, ctx->keys, bs, c.B, c.d, alpha);
        else
            launch_k(worker_grad_dense_kernel<__nv_bfloat16>, grid, kThreads, 0, st, (const __nv_bfloat16*)D.values, D.labels, ctx->xhat_diff, s->z_snap, ctx->keys, bs, c.B, c.d, alpha);
    }
    ctx->launches += 1;
    launch_norm_inf(ctx, alpha, c.d, c.M, reinterpret_cast<uint32_t*>(norm_inf), st);
}

// ---- whole rounds in one cluster kernel ---------------------------------------------------------------------
typedef void (*SmallRoundKernel)(const SmallRound, const PhiloxKeys);

static SmallRoundKernel small_round_kernel_for(const dq_ctx* ctx)
{
    const bool csr = ctx->data.format == DQ_CSR_F32, acc = ctx->cfg.accelerated != 0;
    if (csr) return acc ? round_cluster_kernel<DQ_CSR_F32, true> : round_cluster_kernel<DQ_CSR_F32, false>;
    return acc ? round_cluster_kernel<DQ_DENSE_F32, true> : round_cluster_kernel<DQ_DENSE_F32, false>;
}

static void small_round_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int blocks, size_t smem, cudaStream_t st)
{
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)blocks; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3((unsigned)blocks); cfg->blockDim = dim3(kSmallThreads); cfg->dynamicSmemBytes = smem; cfg->stream = st;
    cfg->attrs = attr; cfg->numAttrs = 2;
}

static size_t small_round_smem(const dq_ctx* ctx)
{
    const size_t acc = ctx->data.format == DQ_CSR_F32 ? sizeof(long long) * (size_t)ctx->cfg.d : 0;
    return sizeof(float) * 2 * (size_t)small_round_pad(ctx->cfg.d) + acc;
}

// Decides once per context whether its rounds can run in the cluster kernel: logistic model on dense fp32 or CSR
// data, dense messages, synchronous master, fixed model width, one block per worker (M <= 16, the largest
// cluster), and a model of at most 8192 coordinates.
void small_round_setup(dq_ctx* ctx)
{
    ctx->cluster_blocks = 0;
    const dq_config& c = ctx->cfg;
    if (!ctx->has_data || c.no_fused || c.model != DQ_MODEL_LOGISTIC || c.sparsify || c.sequential || c.mu > 0.0f || c.max_delay > 0) return;
    if (c.bx != 2 && c.bx != 4 && c.bx != 8) return;          // the kernel is specialised for the widths that divide eight
    if (ctx->data.format != DQ_DENSE_F32 && ctx->data.format != DQ_CSR_F32) return;
    // beyond about one group of eight coordinates per thread the stages stop being latency-bound and one
    // block per worker is slower than the whole GPU working through separate kernels
    if (c.M > 16 || c.B > 1024 || c.d > 8 * kSmallThreads || small_round_smem(ctx) > 200 * 1024) return;
    SmallRoundKernel kern = small_round_kernel_for(ctx);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)small_round_smem(ctx)) != cudaSuccess ||
        (c.M > 8 && cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)) { cudaGetLastError(); return; }
    cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[2];
    small_round_config(&cfg, attr, c.M, small_round_smem(ctx), nullptr);
    int nclusters = 0;
    if (cudaOccupancyMaxActiveClusters(&nclusters, kern, &cfg) == cudaSuccess && nclusters >= 1) ctx->cluster_blocks = c.M;
    else cudaGetLastError();
}

void launch_round_cluster(dq_ctx* ctx, dq_state* s, uint32_t round0, int nrounds, float eta, float theta, uint64_t* bits_down,
                          uint64_t* bits_up, cudaStream_t st)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    SmallRound P;
    P.values = (const float*)D.values; P.col = D.col_idx; P.row_ptr = D.row_ptr; P.labels = D.labels; P.n = D.n;
    P.d = c.d; P.M = c.M; P.B = c.B; P.bx = c.bx; P.b = c.b; P.pp = ProxParams{c.lambda1, c.lambda2, c.box_lo, c.box_hi};
    P.x = s->x; P.y = s->y; P.xsum = s->x_sum; P.xsnap = s->x_snap; P.gfull = s->g_full; P.zsnap = s->z_snap;
    P.normx = reinterpret_cast<uint32_t*>(s->norm_x);
    P.alpha = ctx->alpha; P.ninf = reinterpret_cast<uint32_t*>(ctx->ninf); P.rows = ctx->rows;
    P.codes_x = ctx->codes_x; P.delta_x = ctx->delta_x; P.xnorm2 = ctx->xnorm_bits;
    P.codes = ctx->msgs.codes; P.stride = ctx->msgs.stride; P.scale = ctx->msgs.scale;
    P.bits_down = (bits_down || bits_up) ? (bits_down ? bits_down : ctx->bits) : nullptr;
    P.bits_up = bits_up ? bits_up : ctx->bits + 1;
    P.status = ctx->status;
    P.round0 = round0; P.nrounds = nrounds; P.eta = eta; P.theta = theta;
    P.acc_scale = ctx->acc_scale; P.acc_inv = ctx->acc_inv;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[2];
    small_round_config(&cfg, attr, ctx->cluster_blocks, small_round_smem(ctx), st);
    cudaLaunchKernelEx(&cfg, small_round_kernel_for(ctx), P, ctx->keys);
    ctx->launches += 1;
}

void launch_objective(dq_ctx* ctx, const float* x, double* P, cudaStream_t st)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    cudaMemsetAsync(P, 0, sizeof(double), st);
    if (c.model == DQ_MODEL_MLP) {
        const MlpShape sh = mlp_shape(ctx);
        const BatchSource none = {nullptr, nullptr, 0u, nullptr, 1, D.n, nullptr};
        launch_mlp_hidden(ctx, D.n, sh, nullptr, x, none, 0, nullptr, ctx->mlp_act[1], st);
        int staged; const size_t osm = mlp_output_smem(sh, &staged);
        launch_k(mlp_output_kernel, (unsigned)D.n, kThreads, osm, st, sh, D.labels, ctx->mlp_rows, nullptr, x, nullptr,
            ctx->mlp_act[1], 1.0 / (double)D.n, nullptr, nullptr, nullptr, nullptr, P, staged, 1, nullptr, 0);
        launch_k(objective_reg_kernel, blocks_for(c.d, ctx->sm_count), kThreads, 0, st, x, c.d, c.lambda1, c.lambda2, P);
        ctx->launches += 3;
        return;
    }
    const int grid = blocks_for(D.n * 32, ctx->sm_count);
    if (D.format == DQ_CSR_F32) launch_k(objective_loss_kernel<DQ_CSR_F32>, grid, kThreads, 0, st, D, x, P);
    else if (D.format == DQ_DENSE_F32) launch_k(objective_loss_kernel<DQ_DENSE_F32>, grid, kThreads, 0, st, D, x, P);
    else launch_k(objective_loss_kernel<DQ_DENSE_BF16>, grid, kThreads, 0, st, D, x, P);
    launch_k(objective_reg_kernel, blocks_for(c.d, ctx->sm_count), kThreads, 0, st, x, c.d, c.lambda1, c.lambda2, P);
    ctx->launches += 2;
}

// Ring slot that each worker reads in round t of the epoch: the broadcast of round t - min(delay, t), ring of tau + 1.
__global__ void set_slots_kernel(const int32_t* __restrict__ delays, int M, int t, int tau, int32_t* __restrict__ slots,
                                 const RoundParams* __restrict__ rp)
{
    pdl_prologue();
    if (rp) t = (int)rp->t_epoch;
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w < M) { const int D = min(min(max(delays[w], 0), tau), t); slots[w] = (t - D) % (tau + 1); }
}

void launch_set_slots(dq_ctx* ctx, int t, cudaStream_t st)
{
    launch_k(set_slots_kernel, (ctx->cfg.M + kThreads - 1) / kThreads, kThreads, 0, st, ctx->delays_dev, ctx->cfg.M, t, ctx->cfg.max_delay, ctx->slots_dev, ctx->rp_active);
    ctx->launches += 1;
}

// Delays across epochs: the ring of xhat - xsnap formed again from the kept broadcasts when the snapshot has changed
// (the same single subtraction as in the model quantiser, so a slot equals what that round would have written against
// the new snapshot).
__global__ void __launch_bounds__(kThreads)
rediff_ring_kernel(const float* __restrict__ xhat_ring, const float* __restrict__ xsnap, int64_t d, int nslots, float* __restrict__ diff_ring)
{
    pdl_prologue();
    const int64_t n = d * nslots, nth = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += nth) diff_ring[i] = __fsub_rn(xhat_ring[i], xsnap[i % d]);
}

void launch_rediff_ring(dq_ctx* ctx, const float* x_snap, cudaStream_t st)
{
    const int nslots = ctx->cfg.max_delay + 1;
    launch_k(rediff_ring_kernel, blocks_for(ctx->cfg.d * nslots, ctx->sm_count), kThreads, 0, st, (const float*)ctx->xhat_ring, x_snap, ctx->cfg.d, nslots, ctx->xhat_diff);
    ctx->launches += 1;
}

// xhat = codes * delta_x of the packed model (no reference subtracted).
void launch_dequant_xhat(dq_ctx* ctx, const uint8_t* codes_x, const float* delta_x, float* xhat, cudaStream_t st)
{
    const dq_config& c = ctx->cfg;
    if (c.bx != 2 && c.bx != 4 && c.bx != 8) { launch_dequant_diff_any(ctx, codes_x, delta_x, nullptr, xhat, c.bx, st); return; }
    DQ_DISPATCH_BITS(c.bx, (launch_k(dequant_diff_kernel<BITS_>, blocks_for(c.d, ctx->sm_count), kThreads, 0, st, codes_x, delta_x, (const float*)nullptr, c.d, xhat)));
    ctx->launches += 1;
}

__global__ void set_round_params_kernel(RoundParams* rp, uint32_t round, float eta, float theta, uint32_t t_epoch)
{
    pdl_prologue();
    rp->round = round; rp->eta = eta; rp->theta = theta; rp->pad = 0u; rp->t_epoch = t_epoch;
}

void launch_set_round_params(dq_ctx* ctx, uint32_t round, float eta, float theta, uint32_t t_epoch, cudaStream_t st)
{
    launch_k(set_round_params_kernel, 1, 1, 0, st, ctx->rp_dev, round, eta, theta, t_epoch);
    ctx->launches += 1;
}

}  // namespace dq
