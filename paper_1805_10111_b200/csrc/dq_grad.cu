// Gradient kernels: the worker's variance-reduced minibatch gradient (Algorithm 1 step 11), the epoch's
// full gradient (step 5), the epoch-boundary state update (steps 3/14, Algorithm 3 steps 3/15), the
// objective of eq. (1) and the transmitted-bit counters.  f_a(x) = log(1 + exp(-y_a <a_a, x>)).
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
// row is scattered into alpha_w with fp32 atomics (alpha must be zero on entry).
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
worker_grad_csr_kernel(const float* __restrict__ val, const int32_t* __restrict__ col, const int64_t* __restrict__ row_ptr,
                       const float* __restrict__ labels, const float* __restrict__ diff, const float* __restrict__ z_snap,
                       const __grid_constant__ PhiloxKeys K, BatchSource bs, int M, int B, int64_t d, float* __restrict__ alpha,
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
    float* out = alpha + (int64_t)w * d;
    uint32_t* bm = touched ? touched + (int64_t)w * bm_words : nullptr;
    for (int64_t k = k0 + lane; k < k1; k += 32) {
        const int32_t c = __ldg(col + k);
        atomicAdd(out + c, r * __ldg(val + k));
        if (bm) {
            const uint32_t bit = 1u << ((c >> 3) & 31);
            uint32_t* word = bm + (c >> 8);
            if (!(*reinterpret_cast<volatile uint32_t*>(word) & bit)) atomicOr(word, bit);
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// Dense worker gradient (fp32 or bf16 features).  grid (ceil(B / kRowsPerBlock), M).  Phase A: one warp
// per row computes the slope difference; phase B: threads own columns and add the block's rows.
// alpha must be zero on entry when more than one block serves a worker.
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
    const int j0 = blockIdx.x * kRowsPerBlock;
    const int nrows = min(kRowsPerBlock, B - j0);
    for (int j = warp; j < nrows; j += kThreads / 32) {
        const int64_t a = batch_row(bs, K, w, j0 + j, B, lane == 0);
        const float dz = (float)warp_dot_dense(X + a * d, diff_of_worker(bs, diff, w), d, lane);
        if (lane == 0) { s_r[j] = slope_difference(labels[a], z_snap[a], dz) / (float)B; s_row[j] = a; }
    }
    __syncthreads();
    float* out = alpha + (int64_t)w * d;
    for (int64_t i = threadIdx.x; i < d; i += blockDim.x) {
        float s = 0.0f;
        for (int j = 0; j < nrows; ++j) s = fmaf(s_r[j], to_float(X[s_row[j] * d + i]), s);
        if (gridDim.x == 1) out[i] = s; else atomicAdd(out + i, s);
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

// Vectorised dense worker gradient: same plan as worker_grad_dense_kernel with 16-byte loads and
// 16-byte atomics (d a multiple of the vector width).  The rows read in phase A are read again in phase
// B while they are still in L2.
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
    const int j0 = blockIdx.x * kRowsPerBlock;
    const int nrows = min(kRowsPerBlock, B - j0);
    for (int j = warp; j < nrows; j += kThreads / 32) {
        const int64_t a = batch_row(bs, K, w, j0 + j, B, lane == 0);
        const float dz = (float)warp_dot_dense_vec(X + a * d, diff_of_worker(bs, diff, w), d, lane);
        if (lane == 0) { s_r[j] = slope_difference(labels[a], z_snap[a], dz) / (float)B; s_rowp[j] = reinterpret_cast<const uint4*>(X + a * d); }
    }
    __syncthreads();
    const int nv = (int)(d / N);
    float* out = alpha + (int64_t)w * d;
    for (int v = threadIdx.x; v < nv; v += blockDim.x) {
        float acc[N];
#pragma unroll
        for (int q = 0; q < N; ++q) acc[q] = 0.0f;
#pragma unroll 4
        for (int j = 0; j < nrows; ++j) {
            float f[N];
            RowVec<T>::unpack(__ldg(s_rowp[j] + v), f);
            const float r = s_r[j];
#pragma unroll
            for (int q = 0; q < N; ++q) acc[q] = fmaf(r, f[q], acc[q]);
        }
        float4* o4 = reinterpret_cast<float4*>(out + (int64_t)v * N);
#pragma unroll
        for (int q = 0; q < N / 4; ++q) {
            const float4 val = make_float4(acc[q * 4], acc[q * 4 + 1], acc[q * 4 + 2], acc[q * 4 + 3]);
            if (gridDim.x == 1) o4[q] = val; else atomicAdd(o4 + q, val);
        }
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

// Transmitted bits of one round by the paper's message sizes (Section 3.1; remark after Theorem 3).
__global__ void bits_kernel(int M, int64_t d, int bx, int b, int flag_round, int sparse_msgs, const uint32_t* __restrict__ nnz,
                            uint64_t* __restrict__ bits_down, uint64_t* __restrict__ bits_up)
{
    pdl_prologue();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    *bits_down = flag_round ? (uint64_t)M : (uint64_t)M * (32ull + (uint64_t)bx * (uint64_t)d);
    uint64_t up = 0;
    int logd = 0; while (((int64_t)1 << logd) < d) ++logd;
    for (int w = 0; w < M; ++w) up += sparse_msgs ? 32ull + (uint64_t)nnz[w] * (uint64_t)(logd + b) : 32ull + (uint64_t)b * (uint64_t)d;
    *bits_up = up;
}

// ---------------------------------------------------------------------------------------------------
// Second smooth part (Section 5.2): 3-layer fully connected network, in -> hidden (ReLU) -> classes, softmax
// cross-entropy.  Parameters x = [W1 (hidden x in, row-major), b1, W2 (classes x hidden), b2]; labels hold class
// indices.  The worker needs grad f_B(xhat) - grad f_B(xsnap): three small kernels evaluate both parameter
// vectors side by side (either may be absent: NULL), rows listed explicitly or drawn from the batch stream.
//   mlp_hidden_kernel   block per tile of sampled rows and eight hidden units: hidden activations (one warp per unit, coalesced along in)
//   mlp_output_kernel   block per sampled row: logits, softmax, d loss / d logits, d loss / d hidden (ReLU-gated)
//   mlp_param_kernel    block per (hidden unit or the tail, worker): sums over the worker's rows, no atomics
// ---------------------------------------------------------------------------------------------------
struct MlpShape { int64_t in; int hidden, classes; };

__device__ __forceinline__ int64_t mlp_off_b1(const MlpShape& s) { return (int64_t)s.hidden * s.in; }
__device__ __forceinline__ int64_t mlp_off_w2(const MlpShape& s) { return mlp_off_b1(s) + s.hidden; }
__device__ __forceinline__ int64_t mlp_off_b2(const MlpShape& s) { return mlp_off_w2(s) + (int64_t)s.classes * s.hidden; }

constexpr int kMlpUnits = 8;         // hidden units whose first-layer gradients one block forms from the same rows
constexpr int kMlpTile = 8;          // sampled rows that share one pass over a hidden unit's weights

// grid (ceil(nslots / kMlpTile), ceil(hidden / 8)): a block holds kMlpTile rows in shared memory and each of its
// eight warps owns one hidden unit, so a weight row is read once for the whole tile (a block per row would read the
// first layer once per sample).  Per row the sum runs in the same order as before: lanes stride over the inputs,
// then a butterfly across lanes.
__global__ void __launch_bounds__(kThreads)
mlp_hidden_kernel(const float* __restrict__ X, MlpShape sh, const float* __restrict__ xa, const float* __restrict__ xb,
                  const __grid_constant__ PhiloxKeys K, BatchSource bs, int B, int32_t* __restrict__ row_of_slot,
                  float* __restrict__ act_a, float* __restrict__ act_b, int64_t nslots)
{
    pdl_prologue();
    extern __shared__ float s_in[];                      // [kMlpTile][in] features of the tile's rows
    __shared__ int64_t s_row[kMlpTile];
    clear_word(bs);
    const int64_t slot0 = (int64_t)blockIdx.x * kMlpTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < kMlpTile) {
        const int64_t slot = slot0 + threadIdx.x;
        int64_t a = -1;
        if (slot < nslots) {
            a = B > 0 ? batch_row(bs, K, (int)(slot / B), (int)(slot % B), B, blockIdx.y == 0) : slot;   // B = 0: row = slot
            if (row_of_slot && blockIdx.y == 0) row_of_slot[slot] = (int32_t)a;
        }
        s_row[threadIdx.x] = a;
    }
    __syncthreads();
    for (int64_t q = threadIdx.x; q < (int64_t)kMlpTile * sh.in; q += blockDim.x) {
        const int t = (int)(q / sh.in); const int64_t i = q - (int64_t)t * sh.in;
        s_in[q] = s_row[t] >= 0 ? X[s_row[t] * sh.in + i] : 0.0f;
    }
    __syncthreads();
    const int j = blockIdx.y * (kThreads / 32) + warp;
    if (j >= sh.hidden) return;
    float sa[kMlpTile], sb[kMlpTile];
#pragma unroll
    for (int t = 0; t < kMlpTile; ++t) { sa[t] = 0.0f; sb[t] = 0.0f; }
#pragma unroll 2
    for (int64_t i = lane; i < sh.in; i += 32) {
        const float wa = xa ? xa[(int64_t)j * sh.in + i] : 0.0f, wb = xb ? xb[(int64_t)j * sh.in + i] : 0.0f;
#pragma unroll
        for (int t = 0; t < kMlpTile; ++t) {
            const float f = s_in[(int64_t)t * sh.in + i];
            sa[t] = fmaf(wa, f, sa[t]); sb[t] = fmaf(wb, f, sb[t]);
        }
    }
    const float ba = xa ? xa[mlp_off_b1(sh) + j] : 0.0f, bb = xb ? xb[mlp_off_b1(sh) + j] : 0.0f;
#pragma unroll
    for (int t = 0; t < kMlpTile; ++t) {
        const float va = warp_sum(sa[t]), vb = warp_sum(sb[t]);
        if (lane == 0 && slot0 + t < nslots) {
            if (xa) act_a[(slot0 + t) * sh.hidden + j] = fmaxf(va + ba, 0.0f);
            if (xb) act_b[(slot0 + t) * sh.hidden + j] = fmaxf(vb + bb, 0.0f);
        }
    }
}

// One model of one row: logits -> softmax -> dz = (p - onehot) * wgt, dh_j = relu'(h_j) sum_c dz_c W2[c][j]; returns loss.
__device__ __forceinline__ void mlp_output_one(const MlpShape& sh, const float* __restrict__ x, const float* __restrict__ act,
                                               int label, float wgt, float* __restrict__ dz, float* __restrict__ dh,
                                               float* s_z, double* loss_out)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int c = warp; c < sh.classes; c += kThreads / 32) {
        float s = 0.0f;
        for (int j = lane; j < sh.hidden; j += 32) s = fmaf(x[mlp_off_w2(sh) + (int64_t)c * sh.hidden + j], act[j], s);
        s = warp_sum(s);
        if (lane == 0) s_z[c] = s + x[mlp_off_b2(sh) + c];
    }
    __syncthreads();
    float zmax = -INFINITY, sum = 0.0f, others = 0.0f;      // others: the sum without the label's term, so that
    for (int c = 0; c < sh.classes; ++c) zmax = fmaxf(zmax, s_z[c]);     // p_label - 1 = -others/sum has no cancellation
    for (int c = 0; c < sh.classes; ++c) { const float e = expf(s_z[c] - zmax); sum += e; if (c != label) others += e; }
    if (threadIdx.x == 0 && loss_out) *loss_out = (double)(zmax + logf(sum)) - (double)s_z[label];
    __syncthreads();
    for (int c = threadIdx.x; c < sh.classes; c += blockDim.x) {
        const float v = (c == label ? -others / sum : expf(s_z[c] - zmax) / sum) * wgt;
        s_z[sh.classes + c] = v;
        if (dz) dz[c] = v;
    }
    __syncthreads();
    if (dh) {
        for (int j = threadIdx.x; j < sh.hidden; j += blockDim.x) {
            float s = 0.0f;
            for (int c = 0; c < sh.classes; ++c) s = fmaf(s_z[sh.classes + c], x[mlp_off_w2(sh) + (int64_t)c * sh.hidden + j], s);
            dh[j] = act[j] > 0.0f ? s : 0.0f;
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads)
mlp_output_kernel(MlpShape sh, const float* __restrict__ labels, const int32_t* __restrict__ row_of_slot,
                  const float* __restrict__ xa, const float* __restrict__ xb, const float* __restrict__ act_a,
                  const float* __restrict__ act_b, float wgt, float* __restrict__ dz_a, float* __restrict__ dz_b,
                  float* __restrict__ dh_a, float* __restrict__ dh_b, double* __restrict__ loss_b)
{
    pdl_prologue();
    extern __shared__ float s_z[];                       // [2 * classes]
    const int64_t slot = blockIdx.x;
    const int label = (int)labels[row_of_slot[slot]];
    if (xa) mlp_output_one(sh, xa, act_a + slot * sh.hidden, label, wgt, dz_a + slot * sh.classes, dh_a + slot * sh.hidden, s_z, nullptr);
    if (xb) {
        double loss = 0.0;
        mlp_output_one(sh, xb, act_b + slot * sh.hidden, label, wgt, dz_b ? dz_b + slot * sh.classes : nullptr,
                       dh_b ? dh_b + slot * sh.hidden : nullptr, s_z, loss_b ? &loss : nullptr);
        if (loss_b && threadIdx.x == 0) atomicAdd(loss_b, loss * (double)wgt);
    }
}

// grid (hidden + 1, groups): block (j, w) sums over the rows [w*B, (w+1)*B) of its group.  j < hidden: row j of W1 and
// b1[j]; j == hidden: W2 and b2.  Output = model a minus model b (either may be absent).  FULL: double sums added to
// g64 with atomics (epoch gradient over many groups); otherwise stored to out [groups][P] with the norm folded in.
template <bool FULL>
__global__ void __launch_bounds__(kThreads)
mlp_param_kernel(const float* __restrict__ X, MlpShape sh, const int32_t* __restrict__ row_of_slot, int B, int64_t total_rows,
                 const float* __restrict__ act_a, const float* __restrict__ act_b, const float* __restrict__ dz_a,
                 const float* __restrict__ dz_b, const float* __restrict__ dh_a, const float* __restrict__ dh_b,
                 float* __restrict__ out, int64_t P, uint32_t* __restrict__ norm_bits, double* __restrict__ g64)
{
    pdl_prologue();
    typedef typename std::conditional<FULL, double, float>::type acc_t;
    extern __shared__ float s_w[];                       // [kMlpUnits][B] slope differences, then [B] row indices
    const int j0 = blockIdx.x * kMlpUnits, w = blockIdx.y;     // the block after the last tile of hidden units does W2, b2
    const int64_t r0 = (int64_t)w * B;
    const int nrows = (int)min((int64_t)B, total_rows - r0);
    uint32_t nmax = 0;
    float* o = FULL ? nullptr : out + (int64_t)w * P;
    if (j0 < sh.hidden) {
        // s_w[u][r] = dh_a[r][j0 + u] - dh_b[r][j0 + u]; the rows' indices sit behind them: no dependent load in the loop.
        // The block's hidden units share every feature value that a thread loads.
        int* s_rowid = reinterpret_cast<int*>(s_w + kMlpUnits * B);
        for (int q = threadIdx.x; q < kMlpUnits * nrows; q += blockDim.x) {
            const int u = q / nrows, r = q - u * nrows, j = j0 + u;
            const float da = (dh_a && j < sh.hidden) ? dh_a[(r0 + r) * sh.hidden + j] : 0.0f;
            const float db = (dh_b && j < sh.hidden) ? dh_b[(r0 + r) * sh.hidden + j] : 0.0f;
            s_w[u * B + r] = da - db;
        }
        for (int r = threadIdx.x; r < nrows; r += blockDim.x) s_rowid[r] = row_of_slot[r0 + r];
        __syncthreads();
        for (int64_t i = threadIdx.x; i <= sh.in; i += blockDim.x) {       // i == in: the bias b1[j]
            acc_t s[kMlpUnits];
#pragma unroll
            for (int u = 0; u < kMlpUnits; ++u) s[u] = 0;
#pragma unroll 4
            for (int r = 0; r < nrows; ++r) {
                const float f = (i < sh.in) ? X[(int64_t)s_rowid[r] * sh.in + i] : 1.0f;
#pragma unroll
                for (int u = 0; u < kMlpUnits; ++u) s[u] += (acc_t)(s_w[u * B + r] * f);
            }
#pragma unroll
            for (int u = 0; u < kMlpUnits; ++u) {
                const int j = j0 + u;
                if (j >= sh.hidden) break;
                const int64_t pidx = (i < sh.in) ? (int64_t)j * sh.in + i : mlp_off_b1(sh) + j;
                if (FULL) atomicAdd(g64 + pidx, (double)s[u]);
                else { o[pidx] = (float)s[u]; nmax = max(nmax, __float_as_uint((float)s[u]) & 0x7FFFFFFFu); }
            }
        }
    } else {
        const int nout = sh.classes * (sh.hidden + 1);                       // W2 entries then b2
        for (int t = threadIdx.x; t < nout; t += blockDim.x) {
            const bool bias = t >= sh.classes * sh.hidden;
            const int c = bias ? t - sh.classes * sh.hidden : t / sh.hidden, jj = bias ? 0 : t % sh.hidden;
            acc_t s = 0;
            for (int r = 0; r < nrows; ++r) {
                const int64_t q = r0 + r;
                const float ta = dz_a ? dz_a[q * sh.classes + c] * (bias ? 1.0f : act_a[q * sh.hidden + jj]) : 0.0f;
                const float tb = dz_b ? dz_b[q * sh.classes + c] * (bias ? 1.0f : act_b[q * sh.hidden + jj]) : 0.0f;
                s += (acc_t)(ta - tb);
            }
            const int64_t pidx = bias ? mlp_off_b2(sh) + c : mlp_off_w2(sh) + (int64_t)c * sh.hidden + jj;
            if (FULL) atomicAdd(g64 + pidx, (double)s);
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
        for (int64_t i = (FMT == DQ_CSR_F32 ? 0 : d) + threadIdx.x; i < dpad; i += blockDim.x) s_alpha[i] = 0.0f;
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
                for (int64_t k = k0 + l16; k < k1; k += 16) atomicAdd(s_alpha + __ldg(P.col + k), r * __ldg(P.values + k));
            }
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
static dim3 mlp_hidden_grid(int64_t nslots, const MlpShape& sh)
{
    return dim3((unsigned)((nslots + kMlpTile - 1) / kMlpTile), (unsigned)((sh.hidden + kThreads / 32 - 1) / (kThreads / 32)));
}
constexpr int kMlpGroup = 256;      // rows per block of the epoch-gradient sums

// g <- (1/n) sum_i grad loss_i(x) over all rows (double sums), via the "a" slots of the activation buffers.
static void launch_mlp_full_grad(dq_ctx* ctx, const float* x, float* g, cudaStream_t st)
{
    const dq_data& D = ctx->data; const MlpShape sh = mlp_shape(ctx);
    const BatchSource none = {nullptr, nullptr, 0u, nullptr, 1, D.n, nullptr};
    const int64_t P = ctx->cfg.d;
    launch_k(mlp_hidden_kernel, mlp_hidden_grid(D.n, sh), kThreads, sizeof(float) * kMlpTile * sh.in, st, (const float*)D.values, sh, x, nullptr, ctx->keys, none, 0,
                                                                             ctx->mlp_rows, ctx->mlp_act[0], nullptr, (int64_t)D.n);
    launch_k(mlp_output_kernel, (unsigned)D.n, kThreads, sizeof(float) * 2 * sh.classes, st, sh, D.labels, ctx->mlp_rows, x, nullptr, ctx->mlp_act[0],
        nullptr, (float)(1.0 / (double)D.n), ctx->mlp_dz[0], nullptr, ctx->mlp_dh[0], nullptr, nullptr);
    cudaMemsetAsync(ctx->g64, 0, sizeof(double) * P, st);
    dim3 grid((sh.hidden + kMlpUnits - 1) / kMlpUnits + 1, (unsigned)((D.n + kMlpGroup - 1) / kMlpGroup));
    launch_k(mlp_param_kernel<true>, grid, kThreads, sizeof(float) * (kMlpUnits + 1) * kMlpGroup, st, (const float*)D.values, sh, ctx->mlp_rows, kMlpGroup, D.n,
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
    launch_k(mlp_hidden_kernel, mlp_hidden_grid(R, sh), kThreads, sizeof(float) * kMlpTile * sh.in, st, (const float*)D.values, sh, xhat, s->x_snap, ctx->keys, bs, c.B, ctx->mlp_rows,
                                                                   ctx->mlp_act[0], ctx->mlp_act[1], (int64_t)R);
    launch_k(mlp_output_kernel, R, kThreads, sizeof(float) * 2 * sh.classes, st, sh, D.labels, ctx->mlp_rows, xhat, s->x_snap, ctx->mlp_act[0],
        ctx->mlp_act[1], 1.0f / (float)c.B, ctx->mlp_dz[0], ctx->mlp_dz[1], ctx->mlp_dh[0], ctx->mlp_dh[1], nullptr);
    if (!ctx->ninf_zeroed) cudaMemsetAsync(nb, 0, sizeof(uint32_t) * c.M, st);
    dim3 grid((sh.hidden + kMlpUnits - 1) / kMlpUnits + 1, c.M);
    launch_k(mlp_param_kernel<false>, grid, kThreads, sizeof(float) * (kMlpUnits + 1) * c.B, st, (const float*)D.values, sh, ctx->mlp_rows, c.B, (int64_t)R,
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

// Whether the worker stage accumulates into alpha with atomics (and so needs it cleared first).
bool worker_accumulates(const dq_ctx* ctx)
{
    const dq_config& c = ctx->cfg; const dq_data& D = ctx->data;
    if (c.model == DQ_MODEL_MLP) return false;
    if (D.format == DQ_CSR_F32) return !ctx->list_mode;
    const bool vec = (c.d % (D.format == DQ_DENSE_F32 ? 4 : 8)) == 0;
    if (vec && c.B >= 64) return false;                        // column sums are stored, not added
    return (c.B + kRowsPerBlock - 1) / kRowsPerBlock > 1;
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
        return;
    }
    if (list) launch_clear_listed(ctx, st);                      // alpha is all-zero again before this round adds to it
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
        if (!ctx->alpha_zeroed && !list) cudaMemsetAsync(alpha, 0, sizeof(float) * c.M * c.d, st);
        launch_k(worker_grad_csr_kernel, (int)(((int64_t)c.M * c.B * 32 + kThreads - 1) / kThreads), kThreads, 0, st, (const float*)D.values, D.col_idx, D.row_ptr, D.labels, ctx->xhat_diff, s->z_snap, ctx->keys, bs, c.M, c.B, c.d, alpha,
            list ? ctx->touched : nullptr, ctx->bm_words);
    } else {
        dim3 grid((c.B + kRowsPerBlock - 1) / kRowsPerBlock, c.M);
        const bool f32 = D.format == DQ_DENSE_F32;
        const bool vec = (c.d % (f32 ? 4 : 8)) == 0 && (reinterpret_cast<uintptr_t>(alpha) & 15) == 0;   // data is 16-byte aligned by contract
        if (grid.x > 1 && !ctx->alpha_zeroed && !(vec && c.B >= 64)) cudaMemsetAsync(alpha, 0, sizeof(float) * c.M * c.d, st);
        if (vec && c.B >= 64) {        // large minibatch: margins, then atomics-free column sums with the norm folded in
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
    if (list) { launch_build_group_list(ctx, reinterpret_cast<uint32_t*>(norm_inf), st); ctx->list_ready = true; }
    else launch_norm_inf(ctx, alpha, c.d, c.M, reinterpret_cast<uint32_t*>(norm_inf), st);
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

static size_t small_round_smem(const dq_ctx* ctx) { return sizeof(float) * 2 * (size_t)small_round_pad(ctx->cfg.d); }

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
        launch_k(mlp_hidden_kernel, mlp_hidden_grid(D.n, sh), kThreads, sizeof(float) * kMlpTile * sh.in, st, (const float*)D.values, sh, nullptr, x, ctx->keys, none, 0,
                                                                                 ctx->mlp_rows, nullptr, ctx->mlp_act[1], (int64_t)D.n);
        launch_k(mlp_output_kernel, (unsigned)D.n, kThreads, sizeof(float) * 2 * sh.classes, st, sh, D.labels, ctx->mlp_rows, nullptr, x, nullptr,
            ctx->mlp_act[1], (float)(1.0 / (double)D.n), nullptr, nullptr, nullptr, nullptr, P);
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
__global__ void set_slots_kernel(const int32_t* __restrict__ delays, int M, int t, int tau, int32_t* __restrict__ slots)
{
    pdl_prologue();
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w < M) { const int D = min(min(max(delays[w], 0), tau), t); slots[w] = (t - D) % (tau + 1); }
}

void launch_set_slots(dq_ctx* ctx, int t, cudaStream_t st)
{
    launch_k(set_slots_kernel, (ctx->cfg.M + kThreads - 1) / kThreads, kThreads, 0, st, ctx->delays_dev, ctx->cfg.M, t, ctx->cfg.max_delay, ctx->slots_dev);
    ctx->launches += 1;
}

__global__ void set_round_params_kernel(RoundParams* rp, uint32_t round, float eta, float theta)
{
    pdl_prologue();
    rp->round = round; rp->eta = eta; rp->theta = theta; rp->pad = 0u;
}

void launch_set_round_params(dq_ctx* ctx, uint32_t round, float eta, float theta, cudaStream_t st)
{
    launch_k(set_round_params_kernel, 1, 1, 0, st, ctx->rp_dev, round, eta, theta);
    ctx->launches += 1;
}

void launch_bits(dq_ctx* ctx, int flag_round, bool sparse_msgs, const uint32_t* nnz, uint64_t* bits_down, uint64_t* bits_up,
                 cudaStream_t st)
{
    const dq_config& c = ctx->cfg;
    launch_k(bits_kernel, 1, 32, 0, st, c.M, c.d, c.bx, c.b, flag_round, sparse_msgs ? 1 : 0, nnz, bits_down, bits_up);
    ctx->launches += 1;
}

}  // namespace dq
