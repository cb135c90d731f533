// Streaming codec kernels: infinity norm, Q_(delta,b) + bit packing (Section 3.1; Algorithm 1 steps 8
// and 12), sparsification (eq. (4), Lemma 2; Algorithm 2 steps 12-13), and the master's unpack +
// aggregate + prox step (Algorithm 1 step 9, Algorithm 3 step 9).  All are bandwidth kernels: 256-bit
// coalesced loads, one Philox call per eight coordinates, codes packed in registers.
#include <atomic>

#include "dq_common.cuh"
#include "dq_kernels.cuh"

namespace dq {

// ---------------------------------------------------------------------------------------------------
// ||v_w||_inf as the maximum of the absolute-value bit patterns (exact, order-free).  NaN/Inf patterns
// compare above every finite value, so a non-finite input surfaces as a non-finite norm.
// grid (blocks, M); norm_bits must be zero on entry.
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) norm_inf_kernel(const float* __restrict__ v, int64_t d, int vec_ok,
                                                            uint32_t* __restrict__ norm_bits)
{
    pdl_prologue();
    const float* row = v + (int64_t)blockIdx.y * d;
    uint32_t m = 0;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, nth = (int64_t)gridDim.x * blockDim.x;
    if (vec_ok) {
        const int64_t ng = d >> 3;
        for (int64_t g = tid; g < ng; g += nth) {
            float a[8]; load8(row + (g << 3), a);
#pragma unroll
            for (int j = 0; j < 8; ++j) m = max(m, __float_as_uint(a[j]) & 0x7FFFFFFFu);
        }
        for (int64_t i = (ng << 3) + tid; i < d; i += nth) m = max(m, __float_as_uint(__ldg(row + i)) & 0x7FFFFFFFu);
    } else {
        for (int64_t i = tid; i < d; i += nth) m = max(m, __float_as_uint(__ldg(row + i)) & 0x7FFFFFFFu);
    }
    block_atomic_max(m, norm_bits + blockIdx.y);
}

// ---------------------------------------------------------------------------------------------------
// Dense Q_(delta,b) + pack.  grid (blocks, M).  Each thread turns groups of eight coordinates into BITS
// bytes.  ngroups covers the zero padding of the packed message (coordinates >= d quantise to code 0).
// ---------------------------------------------------------------------------------------------------
// With DIFF the kernel also writes code*delta - ref (the dequantised vector minus a reference), which is what the
// worker-gradient stage needs from the broadcast model.
template <int BITS, bool DIFF = false>
__global__ void __launch_bounds__(kThreads)
quantize_pack_kernel(const float* __restrict__ v, int64_t d, int vec_ok, const uint32_t* __restrict__ norm_bits,
                     uint8_t* __restrict__ codes, int64_t stride, float* __restrict__ scale,
                     const __grid_constant__ PhiloxKeys K, uint32_t round, uint32_t worker_base, uint32_t stream,
                     int64_t ngroups, int* __restrict__ status, const RoundParams* __restrict__ rp,
                     const float* __restrict__ ref = nullptr, float* __restrict__ diff = nullptr,
                     float* __restrict__ zero_f = nullptr, int64_t zero_n = 0, uint32_t* __restrict__ zero_u = nullptr, int zero_un = 0,
                     const int32_t* __restrict__ bits_gate = nullptr /* run only if *bits_gate == BITS */,
                     int ring = 0 /* diff is a ring of this many vectors: write the slot of the device's round counter */)
{
    pdl_prologue();
    if (bits_gate && *bits_gate != BITS) return;
    if (rp) round = rp->round;
    if (DIFF && rp && ring > 1) diff += (int64_t)(rp->t_epoch % (uint32_t)ring) * d;
    if (DIFF) {   // also clears the buffers that the next stages of the round accumulate into
        const int64_t nth0 = (int64_t)gridDim.x * gridDim.y * blockDim.x;
        const int64_t tid0 = ((int64_t)blockIdx.y * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x;
        for (int64_t i = tid0; i < zero_n; i += nth0) zero_f[i] = 0.0f;
        for (int64_t i = tid0; i < zero_un; i += nth0) zero_u[i] = 0u;
    }
    const int w = blockIdx.y;
    const uint32_t nb = norm_bits[w];
    const float nrm = __uint_as_float(nb);
    const bool finite = nb < 0x7F800000u;
    // delta = nrm / L; inv = 1/delta rounded toward zero so that |v| <= nrm stays inside the hull.
    const float inv = (finite && nb != 0u) ? __fdiv_rd((float)levels(BITS), nrm) : 0.0f;
    const float delta = (finite && nb != 0u) ? __fdiv_rn(nrm, (float)levels(BITS)) : 0.0f;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        scale[w] = delta;
        if (!finite) set_status(status, DQ_ERR_NONFINITE);
    }
    const float* row = v + (int64_t)w * d;
    uint8_t* out = codes + (int64_t)w * stride;
    const uint32_t worker = worker_base + (uint32_t)w;
    const int64_t nth = (int64_t)gridDim.x * blockDim.x;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < ngroups; g += nth) {
        const int64_t i0 = g << 3;
        uint32_t s[8];
        if (finite) {
            float a[8];
            if (vec_ok && i0 + 8 <= d) load8(row + i0, a); else load8_guarded(row, i0, d, a);
            uint32_t r[4];
            philox4x32_10((uint32_t)g, round, worker, stream, K, r);
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = round_fixed<BITS>(a[j], inv, half16(r, j));
        } else {                                   // NaN or Inf in the message: every code is 0 (a NaN would pick its own bits)
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = 128u << 16;
        }
        store_group<BITS>(out + g * BITS, pack8<BITS>(s));
        if (DIFF) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (i0 + j < d) {
                    const float k = (float)((int)((s[j] >> 16) & 0xFFu) - 128);
                    diff[i0 + j] = __fsub_rn(__fmul_rn(k, delta), ref ? ref[i0 + j] : 0.0f);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// ||alpha_w||_1 on an integer grid (order-free): with ||alpha||_inf in [2^(e-1), 2^e) each |alpha_i| is
// scaled by 2^(35-e), truncated, and the integers are added.  l1_sum must be zero on entry.
// ---------------------------------------------------------------------------------------------------
// trunc(|a| * 2^(35-e)) in integer arithmetic: the 24-bit significand shifted by the exponent distance.
// (|a| < 2^e, so the result is below 2^35; bits that fall off the right end are the truncation.)
__device__ __forceinline__ unsigned long long l1_term(float a, int e)
{
    const uint32_t bits = __float_as_uint(a) & 0x7FFFFFFFu;
    uint32_t ex = bits >> 23, mant = bits & 0x007FFFFFu;
    if (ex != 0u) mant |= 0x00800000u; else ex = 1u;                 // subnormals have no hidden bit
    const int sh = (int)ex - 115 - e;                                // value = mant * 2^(ex-150); times 2^(35-e)
    if (sh >= 0) return (unsigned long long)mant << sh;              // sh <= 11
    return (sh > -24) ? (unsigned long long)(mant >> (-sh)) : 0ull;
}

// The same term without integer shifts, for e >= -100 (so that 2^(23-e) is a normal fp32 number): with
// t = |a| 2^(23-e) < 2^23, adding 2^23 toward zero leaves floor(t) in the significand, t - floor(t) is exact, and
// the next 12 bits come out of a second add of the same kind; trunc(|a| 2^(35-e)) = 4096 floor(t) + floor(4096 frac t).
// Every step is exact, so the two integers equal the ones l1_term produces.
__device__ __forceinline__ void l1_term_split(float a, float scale23, uint32_t& hi, uint32_t& lo)
{
    const float t = __fmul_rn(fabsf(a), scale23);
    const float m1 = __fadd_rz(t, 8388608.0f);
    const float fr = __fsub_rn(t, __fsub_rn(m1, 8388608.0f));
    const float m2 = __fmaf_rz(fr, 4096.0f, 8388608.0f);
    hi += __float_as_uint(m1) & 0x007FFFFFu;
    lo += __float_as_uint(m2) & 0x007FFFFFu;
}

__global__ void __launch_bounds__(kThreads) norm_l1_kernel(const float* __restrict__ v, int64_t d, int vec_ok,
                                                           const uint32_t* __restrict__ norm_bits,
                                                           unsigned long long* __restrict__ l1_sum)
{
    pdl_prologue();
    const int w = blockIdx.y;
    const uint32_t nb = norm_bits[w];
    if (nb == 0u || nb >= 0x7F800000u) return;
    int e; (void)frexpf(__uint_as_float(nb), &e);
    const float* row = v + (int64_t)w * d;
    unsigned long long acc = 0;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, nth = (int64_t)gridDim.x * blockDim.x;
    const int64_t ng = vec_ok ? (d >> 3) : 0;
    if (e >= -100) {
        const float scale23 = __uint_as_float((uint32_t)(127 + 23 - e) << 23);     // 2^(23-e)
        unsigned long long acc_hi = 0, acc_lo = 0;
        for (int64_t g = tid; g < ng; g += nth) {
            float a[8]; load8(row + (g << 3), a);
            uint32_t hi = 0, lo = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) l1_term_split(a[j], scale23, hi, lo);
            acc_hi += hi; acc_lo += lo;
        }
        acc = (acc_hi << 12) + acc_lo;
    } else {
        for (int64_t g = tid; g < ng; g += nth) {
            float a[8]; load8(row + (g << 3), a);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc += l1_term(a[j], e);
        }
    }
    for (int64_t i = (ng << 3) + tid; i < d; i += nth) acc += l1_term(__ldg(row + i), e);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    __shared__ unsigned long long s_acc[kThreads / 32];
    if ((threadIdx.x & 31) == 0) s_acc[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += s_acc[i];
        if (t) atomicAdd(l1_sum + w, t);
    }
}

// The same sum over an ascending list of groups (all other coordinates are zero).
__global__ void __launch_bounds__(kThreads) norm_l1_list_kernel(const float* __restrict__ v, int64_t d, int vec_ok, GroupList gl,
                                                                const uint32_t* __restrict__ norm_bits,
                                                                unsigned long long* __restrict__ l1_sum)
{
    pdl_prologue();
    const int w = blockIdx.y;
    const uint32_t nb = norm_bits[w];
    if (nb == 0u || nb >= 0x7F800000u) return;
    int e; (void)frexpf(__uint_as_float(nb), &e);
    const float* row = v + (int64_t)w * d;
    unsigned long long acc = 0;
    const int64_t n = gl.count[w];
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < n; p += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i0 = (int64_t)gl.groups[(int64_t)w * gl.cap + p] << 3;
        float a[8];
        if (vec_ok && i0 + 8 <= d) load8(row + i0, a); else load8_guarded(row, i0, d, a);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc += l1_term(a[j], e);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    __shared__ unsigned long long s_acc[kThreads / 32];
    if ((threadIdx.x & 31) == 0) s_acc[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += s_acc[i];
        if (t) atomicAdd(l1_sum + w, t);
    }
}

// Per-worker constants of eq. (4) with Lemma 2's probabilities, from the two norms.
struct SparsifyScale { float s; bool empty; bool s_inf; };   // s_inf: |alpha|_1 so small that s overflowed

__device__ __forceinline__ SparsifyScale sparsify_scale(uint32_t nb, unsigned long long l1, float phi)
{
    SparsifyScale r; r.s = 0.0f; r.empty = true; r.s_inf = false;
    if (nb == 0u || nb >= 0x7F800000u) return r;
    const float ninf = __uint_as_float(nb);
    int e; (void)frexpf(ninf, &e);
    const float n1 = (float)ldexp((double)l1, e - 35);
    if (n1 == 0.0f) return r;
    const float cap = __fdiv_rn(n1, ninf);                       // Lemma 2: phi <= |alpha|_1 / |alpha|_inf
    const float phi_eff = (phi > 0.0f) ? fminf(phi, cap) : cap;
    r.s = __fdiv_rn(phi_eff, n1); r.empty = false; r.s_inf = r.s > 3.4028234e38f;
    return r;
}

// Survivor mask of one group of eight coordinates and the survivors' beta_i = alpha_i / p_i, with
// p_i = m_i / 2^16, m_i = min(2^16, ceil(|alpha_i| s 2^16)).  For an integer draw u, u < ceil(y) is the same
// as u < y, so the test needs neither the rounding nor an integer conversion; the draw becomes a float by
// placing it in the significand of 2^23.  m_i is only formed for the rare survivors.
__device__ __forceinline__ uint32_t sparsify8(const float (&a)[8], float s, const uint32_t (&r)[4], float (&beta)[8])
{
    uint32_t mask = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float y = __fmul_rn(__fmul_rn(fabsf(a[j]), s), 65536.0f);
        const float uf = __fsub_rn(__uint_as_float(0x4B000000u | half16(r, j)), 8388608.0f);
        mask |= (uint32_t)(uf < y) << j;
        beta[j] = 0.0f;
    }
    if (mask) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if ((mask >> j) & 1u) {
                const float y = __fmul_rn(__fmul_rn(fabsf(a[j]), s), 65536.0f);
                const float m = fminf(ceilf(y), 65536.0f);
                beta[j] = __fdiv_rn(__fmul_rn(a[j], 65536.0f), m);
            }
        }
    }
    return mask;
}

// The survivor mask without float compares or selects.  u < y for an integer draw u is u < ceil(y); adding 2^23 to
// y with rounding toward +inf leaves ceil(y) in the significand (y <= 2^16 (1 + ulp) because phi is clamped to
// |alpha|_1 / |alpha|_inf), the draw is placed under the same exponent with one logic operation, and the sign of
// the difference of the two words is shifted into the mask.  Same mask as sparsify8 for every y that is a number
// (a zero coordinate under an infinite s gives a NaN: the stage kernel clears those bits before it counts).
__device__ __forceinline__ uint32_t mask8(const float (&a)[8], float s, const uint32_t (&r)[4])
{
    uint32_t mask = 0;
#pragma unroll
    for (int j = 7; j >= 0; --j) {
        const float y = __fmul_rn(__fmul_rn(fabsf(a[j]), s), 65536.0f);
        const uint32_t thr = __float_as_uint(__fadd_ru(y, 8388608.0f));
        const uint32_t draw = (j & 1) ? __byte_perm(r[j >> 1], 0x4B000000u, 0x7632) : ((r[j >> 1] & 0xFFFFu) | 0x4B000000u);
        mask = __funnelshift_l(draw - thr, mask, 1);          // (mask << 1) | (draw < thr)
    }
    return mask;
}

// a[j] for a run-time j without moving the array to local memory.
__device__ __forceinline__ float pick8(const float (&a)[8], int j)
{
    const float lo = (j & 2) ? ((j & 1) ? a[3] : a[2]) : ((j & 1) ? a[1] : a[0]);
    const float hi = (j & 2) ? ((j & 1) ? a[7] : a[6]) : ((j & 1) ? a[5] : a[4]);
    return (j & 4) ? hi : lo;
}

// beta_i = alpha_i / p_i of a survivor, p_i = m_i / 2^16 (see sparsify8).
__device__ __forceinline__ float survivor_beta(float a, float s)
{
    const float y = __fmul_rn(__fmul_rn(fabsf(a), s), 65536.0f);
    const float m = fminf(ceilf(y), 65536.0f);
    return __fdiv_rn(__fmul_rn(a, 65536.0f), m);
}

// ---------------------------------------------------------------------------------------------------
// Sparsifier mask pass over a whole vector, with staging: draw the mask, record ||beta_w||_inf, the number
// of survivors of every chunk, and the survivors themselves.  A warp owns a chunk of kChunk coordinates
// and writes the chunk's (coordinate, beta) pairs, in ascending order, into the chunk's own slot of kStash
// entries of the staging area, so that the quantise/emit step reads the few survivors instead of the whole
// vector again.  A chunk with more than kStash survivors keeps only its count: it sets the worker's fallback
// flag and is redone from the vector by sparsify_emit_kernel.  Only lanes that hold a survivor do
// per-survivor work.  grid (blocks, M), blockDim = kThreads.  sb.flags must be zero on entry.
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 3)
sparsify_stage_kernel(const float* __restrict__ v, int64_t d, int vec_ok, const uint32_t* __restrict__ norm_bits,
                      const unsigned long long* __restrict__ l1_sum, float phi,
                      const __grid_constant__ PhiloxKeys K, uint32_t round,
                      uint32_t* __restrict__ beta_norm_bits, uint32_t* __restrict__ chunk_cnt,
                      int64_t nchunks, const RoundParams* __restrict__ rp, StageBufs sb, int M)
{
    pdl_prologue();
    if (rp) round = rp->round;
    const int w = blockIdx.y, lane = threadIdx.x & 31;
    const SparsifyScale sc = sparsify_scale(norm_bits[w], l1_sum[w], phi);
    const float* row = v + (int64_t)w * d;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    uint32_t bmax = 0;
    uint32_t pos = 0;                                         // survivors of the current chunk so far (same in every lane)
    uint32_t* di = nullptr; float* dv = nullptr;
    // survivors of one step (32 groups of eight coordinates, one per lane): positions in index order, then beta
    auto collect = [&](const float (&a)[8], uint32_t mask, uint32_t any, uint32_t g) {
        if (sc.s_inf) {                       // 0 * inf is a NaN, which mask8's integer test takes for a survivor
#pragma unroll
            for (int j = 0; j < 8; ++j) if (a[j] == 0.0f) mask &= ~(1u << j);
            any = __ballot_sync(0xFFFFFFFFu, mask != 0u);
        }
        const uint32_t cnt = __popc(mask);
        uint32_t before, total;
        if (__ballot_sync(0xFFFFFFFFu, cnt > 1u) == 0u) {                         // at most one survivor per lane
            before = __popc(any & lt); total = __popc(any);
        } else {
            uint32_t incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t; }
            before = incl - cnt; total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
        if (mask) {
            uint32_t p = pos + before, mm = mask;
            do {
                const int j = __ffs(mm) - 1; mm &= mm - 1u;
                const float beta = survivor_beta(pick8(a, j), sc.s);
                bmax = max(bmax, __float_as_uint(beta) & 0x7FFFFFFFu);
                if (p < (uint32_t)kStash) { di[p] = (g << 3) + (uint32_t)j; dv[p] = beta; }
                ++p;
            } while (mm);
        }
        pos += total;
    };
    // Two steps are drawn together so that their generator chains interleave.  The kernel is bound by the number
    // of instructions it issues, so a chunk that lies wholly inside an aligned row takes a loop without bounds
    // checks or 64-bit index arithmetic.
    auto two_steps = [&](const float (&a)[8], const float (&b)[8], uint32_t g) {
        uint32_t ra[4], rb[4];
        philox4x32_10(g, round, (uint32_t)w, kStreamMask, K, ra);
        philox4x32_10(g + 32u, round, (uint32_t)w, kStreamMask, K, rb);
        const uint32_t ma = mask8(a, sc.s, ra), mb = mask8(b, sc.s, rb);
        const uint32_t anya = __ballot_sync(0xFFFFFFFFu, ma != 0u), anyb = __ballot_sync(0xFFFFFFFFu, mb != 0u);
        if (anya) collect(a, ma, anya, g);
        if (anyb) collect(b, mb, anyb, g + 32u);
    };
    for (int64_t c = warp; c < nchunks; c += nwarps) {
        pos = 0;
        di = sb.idx + ((int64_t)w * nchunks + c) * kStash;
        dv = sb.val + ((int64_t)w * nchunks + c) * kStash;
        if (!sc.empty) {
            const uint32_t g0 = (uint32_t)(c * (kChunk / 8)) + (uint32_t)lane;     // d <= 2^32: group numbers fit 32 bits
            float bufa[8], bufb[8];
            if (vec_ok && (c + 1) * kChunk <= d) {
                const float* p = row + c * kChunk + lane * 8;
#pragma unroll 1
                for (int it = 0; it < kChunk / 256; it += 2) {
                    load8(p, bufa); load8(p + 256, bufb);
                    two_steps(bufa, bufb, g0 + (uint32_t)it * 32u);
                    p += 512;
                }
            } else {
#pragma unroll 1
                for (int it = 0; it < kChunk / 256; it += 2) {
                    const uint32_t g = g0 + (uint32_t)it * 32u;
                    load8_guarded(row, (int64_t)g << 3, d, bufa);
                    load8_guarded(row, ((int64_t)g + 32) << 3, d, bufb);
                    two_steps(bufa, bufb, g);
                }
            }
        }
        if (lane == 0) {
            chunk_cnt[(int64_t)w * (nchunks + 1) + c] = pos;
            if (pos > (uint32_t)kStash) { sb.flags[w] = 1u; sb.flags[M] = 1u; }
        }
    }
    block_atomic_max(bmax, beta_norm_bits + w);
}

// 16-bit rounding draw of coordinate i (lane i & 7 of the Philox call of its group).
__device__ __forceinline__ uint32_t grad_draw16(uint32_t i, uint32_t round, uint32_t worker, const PhiloxKeys& K)
{
    uint32_t r[4];
    philox4x32_10(i >> 3, round, worker, kStreamGrad, K, r);
    const uint32_t j = i & 7u;
    const uint32_t wlo = (j & 2u) ? r[1] : r[0], whi = (j & 2u) ? r[3] : r[2];
    const uint32_t word = (j & 4u) ? whi : wlo;
    return (j & 1u) ? (word >> 16) : (word & 0xFFFFu);
}

// Scale of the survivors' quantiser and its reciprocal (rounded toward zero), written once per worker.
template <int BITS>
__device__ __forceinline__ float survivor_scale(const uint32_t* norm_bits, const uint32_t* beta_norm_bits, int w,
                                                float* scale, int* status, bool writer)
{
    const uint32_t bb = beta_norm_bits[w];
    const bool finite = bb < 0x7F800000u && norm_bits[w] < 0x7F800000u;
    const float bnrm = __uint_as_float(bb);
    if (writer) {
        scale[w] = (finite && bb != 0u) ? __fdiv_rn(bnrm, (float)levels(BITS)) : 0.0f;
        if (!finite) set_status(status, DQ_ERR_NONFINITE);
    }
    return (finite && bb != 0u) ? __fdiv_rd((float)levels(BITS), bnrm) : 0.0f;
}

// ---------------------------------------------------------------------------------------------------
// Quantise the staged survivors (delta = ||beta||_inf / L, rounding draw keyed by the coordinate) and move
// each chunk's segment to its place in the ascending (position, code) list.  Eight lanes per chunk.
// grid (blocks, M).  The code buffer must be zero on entry.
// ---------------------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kThreads)
sparsify_finish_sparse_kernel(const uint32_t* __restrict__ norm_bits, const uint32_t* __restrict__ beta_norm_bits,
                              const __grid_constant__ PhiloxKeys K, uint32_t round, const uint32_t* __restrict__ chunk_off,
                              int64_t nchunks, StageBufs sb, uint8_t* __restrict__ codes, int64_t stride,
                              float* __restrict__ scale, uint32_t* __restrict__ idx, int64_t cap, int* __restrict__ status,
                              const RoundParams* __restrict__ rp)
{
    pdl_prologue();
    if (rp) round = rp->round;
    const int w = blockIdx.y;
    const float inv = survivor_scale<BITS>(norm_bits, beta_norm_bits, w, scale, status, blockIdx.x == 0 && threadIdx.x == 0);
    uint32_t* out = reinterpret_cast<uint32_t*>(codes + (int64_t)w * stride);
    uint32_t* oidx = idx + (int64_t)w * cap;
    const uint32_t* off = chunk_off + (int64_t)w * (nchunks + 1);
    const int l8 = threadIdx.x & 7;
    const int64_t sub = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 3, nsub = ((int64_t)gridDim.x * blockDim.x) >> 3;
    for (int64_t c = sub; c < nchunks; c += nsub) {
        const uint32_t first = off[c], cnt = off[c + 1] - first;
        if (cnt > (uint32_t)kStash) continue;                                      // left to the re-reading pass
        const uint32_t* si = sb.idx + ((int64_t)w * nchunks + c) * kStash;
        const float* sv = sb.val + ((int64_t)w * nchunks + c) * kStash;
        for (uint32_t e = l8; e < cnt; e += 8u) {
            const int64_t p = (int64_t)first + e;
            if (p >= cap) break;
            const uint32_t i = si[e];
            const uint32_t s = round_fixed<BITS>(sv[e], inv, grad_draw16(i, round, (uint32_t)w, K));
            oidx[p] = i;
            const uint32_t field = ((s >> 16) ^ (BITS == 8 ? 0x80u : 0u)) & ((1u << BITS) - 1u);
            const int64_t bit = p * BITS;
            atomicOr(out + (bit >> 5), field << (bit & 31));
        }
    }
}

// The same for the dense container: every staged survivor's code is OR-ed into its coordinate's field of the
// zeroed packed message.  Workers with a chunk beyond the staging limit are skipped; the re-reading pass writes
// their whole message.  chunk_cnt holds the chunks' counts (no prefix).  grid (blocks, M).
template <int BITS>
__global__ void __launch_bounds__(kThreads)
sparsify_scatter_dense_kernel(const uint32_t* __restrict__ norm_bits, const uint32_t* __restrict__ beta_norm_bits,
                              const __grid_constant__ PhiloxKeys K, uint32_t round, const uint32_t* __restrict__ chunk_cnt,
                              int64_t nchunks, StageBufs sb, uint8_t* __restrict__ codes, int64_t stride,
                              float* __restrict__ scale, int* __restrict__ status, const RoundParams* __restrict__ rp)
{
    pdl_prologue();
    if (rp) round = rp->round;
    const int w = blockIdx.y;
    const float inv = survivor_scale<BITS>(norm_bits, beta_norm_bits, w, scale, status, blockIdx.x == 0 && threadIdx.x == 0);
    if (sb.flags[w]) return;
    uint32_t* out = reinterpret_cast<uint32_t*>(codes + (int64_t)w * stride);
    const uint32_t* cnts = chunk_cnt + (int64_t)w * (nchunks + 1);
    const int l8 = threadIdx.x & 7;
    const int64_t sub = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 3, nsub = ((int64_t)gridDim.x * blockDim.x) >> 3;
    for (int64_t c = sub; c < nchunks; c += nsub) {
        const uint32_t cnt = cnts[c];
        const uint32_t* si = sb.idx + ((int64_t)w * nchunks + c) * kStash;
        const float* sv = sb.val + ((int64_t)w * nchunks + c) * kStash;
        for (uint32_t e = l8; e < cnt; e += 8u) {
            const uint32_t i = si[e];
            const uint32_t s = round_fixed<BITS>(sv[e], inv, grad_draw16(i, round, (uint32_t)w, K));
            const uint32_t field = ((s >> 16) ^ (BITS == 8 ? 0x80u : 0u)) & ((1u << BITS) - 1u);
            const int64_t bit = (int64_t)i * BITS;
            atomicOr(out + (bit >> 5), field << (bit & 31));
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// Sparsifier pass 1: draw the mask, record ||beta_w||_inf over survivors and, for sparse messages, the
// number of survivors of every chunk of kChunk coordinates (one warp per chunk, no block-level sync).
// grid (blocks, M), blockDim = kThreads.
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
sparsify_count_kernel(const float* __restrict__ v, int64_t d, int vec_ok, const uint32_t* __restrict__ norm_bits,
                      const unsigned long long* __restrict__ l1_sum, float phi,
                      const __grid_constant__ PhiloxKeys K, uint32_t round,
                      uint32_t* __restrict__ beta_norm_bits, uint32_t* __restrict__ chunk_cnt /* may be NULL */,
                      int64_t nchunks, const RoundParams* __restrict__ rp, GroupList gl, int iters /* warp steps per chunk */)
{
    pdl_prologue();
    if (rp) round = rp->round;
    const int w = blockIdx.y, lane = threadIdx.x & 31;
    const SparsifyScale sc = sparsify_scale(norm_bits[w], l1_sum[w], phi);
    const float* row = v + (int64_t)w * d;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    uint32_t bmax = 0;
    const int64_t gpc = 32 * (int64_t)iters;                                       // groups per chunk
    const int64_t nch_eff = gl.groups ? ((int64_t)gl.count[w] + gpc - 1) / gpc : nchunks;   // chunks that hold groups
    for (int64_t c = warp; c < nchunks; c += nwarps) {
        uint32_t cnt = 0;
        if (!sc.empty && c < nch_eff) {
#pragma unroll 2
            for (int it = 0; it < iters; ++it) {
                const int64_t g = group_at(gl, w, c * gpc + it * 32 + lane, d), i0 = g << 3;
                if (g < 0) break;
                float a[8], beta[8];
                if (vec_ok && i0 + 8 <= d) load8(row + i0, a); else load8_guarded(row, i0, d, a);
                uint32_t r[4];
                philox4x32_10((uint32_t)g, round, (uint32_t)w, kStreamMask, K, r);
                const uint32_t mask = sparsify8(a, sc.s, r, beta);
                if (mask) {
                    cnt += __popc(mask);
#pragma unroll
                    for (int j = 0; j < 8; ++j) bmax = max(bmax, __float_as_uint(beta[j]) & 0x7FFFFFFFu);
                }
            }
        }
        if (chunk_cnt) {
            cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
            if (lane == 0) chunk_cnt[(int64_t)w * (nchunks + 1) + c] = cnt;
        }
    }
    block_atomic_max(bmax, beta_norm_bits + w);
}

// Exclusive prefix of the chunk counts of each worker (one block per worker); writes nnz and flags
// messages that exceed the capacity (their tail is dropped).
__global__ void __launch_bounds__(kThreads)
chunk_scan_kernel(uint32_t* __restrict__ chunk_off, int64_t nchunks, int64_t cap, uint32_t* __restrict__ nnz,
                  int* __restrict__ status, uint8_t* __restrict__ clear_codes = nullptr /* [M][stride]: zeroed here if given */,
                  int64_t stride = 0)
{
    pdl_prologue();
    if (clear_codes) {
        uint4* row = reinterpret_cast<uint4*>(clear_codes + (int64_t)blockIdx.x * stride);      // stride is a multiple of 16
        for (int64_t q = threadIdx.x; q < (stride >> 4); q += blockDim.x) row[q] = make_uint4(0u, 0u, 0u, 0u);
    }
    uint32_t* off = chunk_off + (int64_t)blockIdx.x * (nchunks + 1);
    __shared__ uint32_t s_warp[kThreads / 32];
    // each thread owns a contiguous run of entries: local sum, one block-wide scan of the sums, local prefix
    const int64_t per = (nchunks + blockDim.x - 1) / blockDim.x;
    const int64_t i0 = (int64_t)threadIdx.x * per, i1 = min(i0 + per, nchunks);
    uint32_t sum = 0;
    for (int64_t i = i0; i < i1; ++i) sum += off[i];
    uint32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if ((threadIdx.x & 31) >= o) incl += t; }
    if ((threadIdx.x & 31) == 31) s_warp[threadIdx.x >> 5] = incl;
    __syncthreads();
    uint32_t run = incl - sum;
    for (int k = 0; k < (int)(threadIdx.x >> 5); ++k) run += s_warp[k];
    for (int64_t i = i0; i < i1; ++i) { const uint32_t c = off[i]; off[i] = run; run += c; }
    if (threadIdx.x == blockDim.x - 1) {
        uint32_t total = run;
        off[nchunks] = total;
        if ((int64_t)total > cap) { set_status(status, DQ_ERR_CAPACITY); total = (uint32_t)cap; }
        nnz[blockIdx.x] = total;
    }
}

// ---------------------------------------------------------------------------------------------------
// Sparsifier pass 2: redraw the mask, quantise the survivors with delta = ||beta||_inf / L (rounding draw
// keyed by the coordinate) and emit either the dense packed message (SPARSE_OUT = false) or the
// (position, code) list at the chunk's offset (SPARSE_OUT = true; codes OR-ed into a zeroed buffer).
// ---------------------------------------------------------------------------------------------------
template <int BITS, bool SPARSE_OUT>
__global__ void __launch_bounds__(kThreads)
sparsify_emit_kernel(const float* __restrict__ v, int64_t d, int vec_ok, const uint32_t* __restrict__ norm_bits,
                     const unsigned long long* __restrict__ l1_sum, float phi,
                     const __grid_constant__ PhiloxKeys K, uint32_t round,
                     const uint32_t* __restrict__ beta_norm_bits, const uint32_t* __restrict__ chunk_off,
                     int64_t nchunks, int64_t ngroups,
                     uint8_t* __restrict__ codes, int64_t stride, float* __restrict__ scale,
                     uint32_t* __restrict__ idx, int64_t cap, int* __restrict__ status, const RoundParams* __restrict__ rp,
                     GroupList gl, int iters,
                     const uint32_t* __restrict__ redo_flags = nullptr /* [M + 1]: per worker, any; NULL: do everything.
                        With sparse output only the chunks with more than kStash survivors are redone. */,
                     int M = 0)
{
    pdl_prologue();
    const int w = blockIdx.y, lane = threadIdx.x & 31;
    if (redo_flags && (redo_flags[M] == 0u || redo_flags[w] == 0u)) return;        // the staged path covered this worker
    if (rp) round = rp->round;
    const int64_t gpc = 32 * (int64_t)iters;
    const SparsifyScale sc = sparsify_scale(norm_bits[w], l1_sum[w], phi);
    const uint32_t bb = beta_norm_bits[w];
    const bool finite = bb < 0x7F800000u && norm_bits[w] < 0x7F800000u;
    const float bnrm = __uint_as_float(bb);
    const float inv = (finite && bb != 0u) ? __fdiv_rd((float)levels(BITS), bnrm) : 0.0f;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        scale[w] = (finite && bb != 0u) ? __fdiv_rn(bnrm, (float)levels(BITS)) : 0.0f;
        if (!finite) set_status(status, DQ_ERR_NONFINITE);
    }
    const float* row = v + (int64_t)w * d;
    uint8_t* out = codes + (int64_t)w * stride;
    uint32_t* oidx = SPARSE_OUT ? idx + (int64_t)w * cap : nullptr;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t nch_eff = (SPARSE_OUT && gl.groups) ? ((int64_t)gl.count[w] + gpc - 1) / gpc : nchunks;
    for (int64_t c = warp; c < nch_eff; c += nwarps) {
        uint32_t pos = SPARSE_OUT ? chunk_off[(int64_t)w * (nchunks + 1) + c] : 0u;
        if (SPARSE_OUT && redo_flags && chunk_off[(int64_t)w * (nchunks + 1) + c + 1] - pos <= (uint32_t)kStash) continue;
        for (int it = 0; it < iters; ++it) {
            const int64_t pos_g = c * gpc + it * 32 + lane;
            const int64_t g = SPARSE_OUT ? group_at(gl, w, pos_g, d) : pos_g, i0 = g << 3;
            uint32_t mask = 0;
            uint32_t s8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) s8[j] = 128u << 16;                        // code 0
            if (!sc.empty && g >= 0 && i0 < d) {
                float a[8], beta[8];
                if (vec_ok && i0 + 8 <= d) load8(row + i0, a); else load8_guarded(row, i0, d, a);
                uint32_t r[4];
                philox4x32_10((uint32_t)g, round, (uint32_t)w, kStreamMask, K, r);
                mask = sparsify8(a, sc.s, r, beta);
                if (mask) {
                    philox4x32_10((uint32_t)g, round, (uint32_t)w, kStreamGrad, K, r);
#pragma unroll
                    for (int j = 0; j < 8; ++j) if ((mask >> j) & 1u) s8[j] = round_fixed<BITS>(beta[j], inv, half16(r, j));
                }
            }
            if (!SPARSE_OUT) {
                if (g < ngroups) store_group<BITS>(out + g * BITS, pack8<BITS>(s8));
            } else {
                // ordered positions inside the warp: survivors of lower lanes come first
                const uint32_t cnt = __popc(mask);
                uint32_t incl = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t; }
                uint32_t p = pos + incl - cnt;
                pos += __shfl_sync(0xFFFFFFFFu, incl, 31);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if ((mask >> j) & 1u) {
                        if ((int64_t)p < cap) {
                            oidx[p] = (uint32_t)(i0 + j);
                            const uint32_t field = ((s8[j] >> 16) ^ (BITS == 8 ? 0x80u : 0u)) & ((1u << BITS) - 1u);
                            const int64_t bit = (int64_t)p * BITS;
                            atomicOr(reinterpret_cast<uint32_t*>(out) + (bit >> 5), field << (bit & 31));
                        }
                        ++p;
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// First list entry of every coordinate tile of kChunk coordinates in each worker's ascending index
// list (binary search; one thread per (tile boundary, worker)).
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
tile_ptr_kernel(const uint32_t* __restrict__ idx, int64_t cap, const uint32_t* __restrict__ nnz, int64_t ntiles,
                uint32_t* __restrict__ tile_ptr)
{
    pdl_prologue();
    const int w = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t > ntiles) return;
    const uint32_t* list = idx + (int64_t)w * cap;
    const uint64_t bound = (uint64_t)t * kChunk;
    uint32_t lo = 0, hi = nnz[w];
    while (lo < hi) { uint32_t mid = (lo + hi) >> 1; if ((uint64_t)list[mid] < bound) lo = mid + 1; else hi = mid; }
    tile_ptr[(int64_t)w * (ntiles + 1) + t] = lo;
}

// ---------------------------------------------------------------------------------------------------
// Master step: g = (1/M) sum_w code_w delta_w (fused multiply-adds in worker order), u = g + g_full,
// prox step on x (Algorithms 1/2) or on y with the momentum combination (Algorithm 3), ||x||_inf.
// ---------------------------------------------------------------------------------------------------
// Quantise + pack + master step in one kernel (dense messages, averaged master).  Between the workers'
// quantiser and the master's unpack the codes would only travel to memory and back.  A block owns a tile of
// kQmTile model coordinates: its threads first quantise the tile for every worker (one group of eight coordinates of
// one worker per task: same draws and codes as quantize_pack_kernel, written out as the packed messages of Section
// 3.1) and leave the codes in shared memory; then each thread takes one coordinate, adds code * delta in worker
// order and applies the prox step (Algorithm 1 steps 12 and 9; Algorithm 3 step 9).  norm_bits [M] are the
// workers' ||alpha_w||_inf.  grid = tiles covering the zero padding of the packed messages; M <= kQmMaxWorkers.
// ---------------------------------------------------------------------------------------------------
constexpr int kQmTile = 256;
constexpr int kQmMaxWorkers = 128;

template <int BITS, bool ACC>
__global__ void __launch_bounds__(kThreads)
quantize_master_kernel(const float* __restrict__ v, int64_t d, int M, int vec_ok, const uint32_t* __restrict__ norm_bits,
                       uint8_t* __restrict__ codes, int64_t stride, float* __restrict__ scale,
                       const __grid_constant__ PhiloxKeys K, uint32_t round, int64_t ngroups, int* __restrict__ status,
                       const float* __restrict__ g_full, float* __restrict__ x, float* __restrict__ y,
                       const float* __restrict__ xsnap, float* __restrict__ xsum, float eta, float theta, ProxParams pp,
                       uint32_t* __restrict__ normx_bits, const RoundParams* __restrict__ rp, BitsArgs ba)
{
    pdl_prologue();
    if (rp) { round = rp->round; eta = rp->eta; theta = rp->theta; }
    if (ba.down && blockIdx.x == 0 && threadIdx.x == 0) write_round_bits(ba, M, d);
    extern __shared__ float s_q[];                           // [M] 1/delta_w rounded toward zero, [M] delta_w, [M][kQmTile] codes
    float* s_inv = s_q; float* s_delta = s_q + M;
    int8_t* s_code = reinterpret_cast<int8_t*>(s_q + 2 * M);
    for (int w = threadIdx.x; w < M; w += blockDim.x) {
        const uint32_t nb = norm_bits[w];
        const bool ok = nb < 0x7F800000u && nb != 0u;
        s_inv[w] = ok ? __fdiv_rd((float)levels(BITS), __uint_as_float(nb)) : 0.0f;
        s_delta[w] = ok ? __fdiv_rn(__uint_as_float(nb), (float)levels(BITS)) : 0.0f;
        if (blockIdx.x == 0) { scale[w] = s_delta[w]; if (nb >= 0x7F800000u) set_status(status, DQ_ERR_NONFINITE); }
    }
    __syncthreads();
    constexpr int GT = kQmTile / 8;                          // groups per tile
    const int64_t g_first = (int64_t)blockIdx.x * GT;
    for (int task = threadIdx.x; task < M * GT; task += blockDim.x) {
        const int w = task / GT, gl = task - w * GT;
        const int64_t g = g_first + gl, i0 = g << 3;
        uint32_t s[8];
        if (g < ngroups) {
            float a[8];
            const float* row = v + (int64_t)w * d;
            if (vec_ok && i0 + 8 <= d) load8(row + i0, a); else load8_guarded(row, i0, d, a);
            uint32_t r[4];
            philox4x32_10((uint32_t)g, round, (uint32_t)w, kStreamGrad, K, r);
            const float inv = s_inv[w];
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = round_fixed<BITS>(a[j], inv, half16(r, j));
            if (norm_bits[w] >= 0x7F800000u) {               // NaN or Inf in the message: every code is 0
#pragma unroll
                for (int j = 0; j < 8; ++j) s[j] = 128u << 16;
            }
            store_group<BITS>(codes + (int64_t)w * stride + g * BITS, pack8<BITS>(s));
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = 128u << 16;
        }
        // the eight codes as bytes (code + 128 sits in byte 2 of each word)
        const uint32_t lo = __byte_perm(__byte_perm(s[0], s[1], 0x0062), __byte_perm(s[2], s[3], 0x0062), 0x5410) ^ 0x80808080u;
        const uint32_t hi = __byte_perm(__byte_perm(s[4], s[5], 0x0062), __byte_perm(s[6], s[7], 0x0062), 0x5410) ^ 0x80808080u;
        *reinterpret_cast<uint2*>(s_code + (int64_t)w * kQmTile + gl * 8) = make_uint2(lo, hi);
    }
    __syncthreads();
    const float inv_m = __fdiv_rn(1.0f, (float)M);
    const float thr = __fmul_rn(eta, pp.lambda1), den = __fadd_rn(1.0f, __fmul_rn(eta, pp.lambda2));
    uint32_t nmax = 0;
    const int64_t i = (int64_t)blockIdx.x * kQmTile + threadIdx.x;
    if (i < d) {
        float* target = ACC ? y : x;
        const float gf = g_full[i], cur = target[i];
        const float xs = ACC ? xsnap[i] : 0.0f;
        float sm = ACC ? xsum[i] : 0.0f, yo = 0.0f, acc = 0.0f;
#pragma unroll 4
        for (int w = 0; w < M; ++w) acc = __fmaf_rn((float)s_code[w * kQmTile + threadIdx.x], s_delta[w], acc);
        const float xo = master_update<ACC>(acc, inv_m, eta, theta, thr, den, pp, gf, cur, xs, yo, sm);
        x[i] = xo;
        if (ACC) { y[i] = yo; xsum[i] = sm; }
        nmax = __float_as_uint(xo) & 0x7FFFFFFFu;
    }
    block_atomic_max(nmax, normx_bits);
    finish_round(rp);
}

// ---------------------------------------------------------------------------------------------------
// acc[j] = fma(code_j, delta, acc[j]) for the 32/BITS codes of one packed word.  The integer-to-float
// conversion avoids the conversion pipe: the code, biased by 2^(BITS-1), is placed in the mantissa of 2^23
// (one byte permute) and the bias is subtracted exactly.
template <int BITS>
__device__ __forceinline__ void accumulate_word(uint32_t word, float dl, float (&acc)[32 / BITS])
{
    constexpr float kBias = 8388608.0f + (float)(1 << (BITS - 1));
    if (BITS == 8) {
        const uint32_t wb = word ^ 0x80808080u;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            acc[j] = __fmaf_rn(__fsub_rn(__uint_as_float(__byte_perm(wb, 0x4B000000u, 0x7540u | j)), kBias), dl, acc[j]);
    } else if (BITS == 4) {
        const uint32_t wb = word ^ 0x88888888u;
        const uint32_t ev = wb & 0x0F0F0F0Fu, od = (wb >> 4) & 0x0F0F0F0Fu;
#pragma unroll
        for (int j = 0; j < 8; ++j)
            acc[j] = __fmaf_rn(__fsub_rn(__uint_as_float(__byte_perm((j & 1) ? od : ev, 0x4B000000u, 0x7540u | (j >> 1))), kBias), dl, acc[j]);
    } else {
        const uint32_t wb = word ^ 0xAAAAAAAAu;
        uint32_t p[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) p[k] = (wb >> (2 * k)) & 0x03030303u;
#pragma unroll
        for (int j = 0; j < 16; ++j)
            acc[j] = __fmaf_rn(__fsub_rn(__uint_as_float(__byte_perm(p[j & 3], 0x4B000000u, 0x7540u | (j >> 2))), kBias), dl, acc[j]);
    }
}

// Dense messages.  Each thread owns the 32/BITS coordinates of one 32-bit code word per worker.
// BATCH: code words (workers) in flight per thread.  8 keeps four blocks per SM for models that stream from HBM; 32 is
// for models of a few thousand coordinates, where the kernel's time is the number of dependent batches of loads.
template <int BITS, bool ACC, int BATCH = 8>
__global__ void __launch_bounds__(kThreads, BATCH == 8 ? 4 : 2)
master_dense_kernel(const uint8_t* __restrict__ codes, int64_t stride, const float* __restrict__ scale, int M, int64_t d,
                    const float* __restrict__ g_full, float* __restrict__ x, float* __restrict__ y,
                    const float* __restrict__ xsnap, float* __restrict__ xsum, float eta, float theta, ProxParams pp,
                    int vec8_ok, uint32_t* __restrict__ normx_bits, const RoundParams* __restrict__ rp, BitsArgs ba)
{
    pdl_prologue();
    if (rp) { eta = rp->eta; theta = rp->theta; }
    if (ba.down && blockIdx.x == 0 && threadIdx.x == 0) write_round_bits(ba, M, d);
    constexpr int W = (BITS == 8) ? 2 : 1;                  // code words per worker and thread
    constexpr int CW = 32 / BITS;                           // coordinates per code word
    constexpr int C = W * CW;                               // coordinates per thread: 8, 8, 16 for 8, 4, 2 bits
    extern __shared__ float s_scale[];
    for (int i = threadIdx.x; i < M; i += blockDim.x) s_scale[i] = scale[i];
    __syncthreads();
    const float inv_m = __fdiv_rn(1.0f, (float)M);
    const float thr = __fmul_rn(eta, pp.lambda1), den = __fadd_rn(1.0f, __fmul_rn(eta, pp.lambda2));
    const int64_t nwords = (d + C - 1) / C;
    const int64_t wstride = stride >> 2;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(codes);
    uint32_t nmax = 0;
    const int64_t nth = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < nwords; t += nth) {
        float acc[W][CW];
#pragma unroll
        for (int j = 0; j < C; ++j) acc[j / CW][j % CW] = 0.0f;
        const int64_t i0 = t * C;
        const bool fast = C >= 8 && vec8_ok && i0 + C <= d;
        float gfp[C >= 8 ? C : 8], curp[C >= 8 ? C : 8];     // issued before the code words so that all loads overlap
        constexpr bool kEarly = BITS != 2;                   // sixteen coordinates per thread: loading early costs a block per SM
        if (fast && kEarly) {
#pragma unroll
            for (int q = 0; q < C / 8; ++q) {
                load8(g_full + i0 + q * 8, *reinterpret_cast<float(*)[8]>(gfp + q * 8));
                load8_rw((ACC ? y : x) + i0 + q * 8, *reinterpret_cast<float(*)[8]>(curp + q * 8));
            }
        }
        if (BITS == 4 && BATCH == 8) {      // the two loop shapes compute the same thing; each bit width uses the one that the
                              // compiler schedules better (measured: registers and load placement differ)
            const uint32_t* wp = words + t * W;
            int w0 = 0;
            for (; w0 + 8 <= M; w0 += 8) {                       // full batches: eight code words in flight, no predicates
                uint32_t wd[8][W];
    #pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (W == 2) { const uint2 u = __ldg(reinterpret_cast<const uint2*>(wp)); wd[k][0] = u.x; wd[k][W - 1] = u.y; }
                    else wd[k][0] = __ldg(wp);
                    wp += wstride;
                }
    #pragma unroll
                for (int k = 0; k < 8; ++k) {
    #pragma unroll
                    for (int q = 0; q < W; ++q) accumulate_word<BITS>(wd[k][q], s_scale[w0 + k], acc[q]);
                }
            }
            for (; w0 < M; ++w0) {                               // remaining workers
                uint32_t wd[W];
                if (W == 2) { const uint2 u = __ldg(reinterpret_cast<const uint2*>(wp)); wd[0] = u.x; wd[W - 1] = u.y; }
                else wd[0] = __ldg(wp);
                wp += wstride;
    #pragma unroll
                for (int q = 0; q < W; ++q) accumulate_word<BITS>(wd[q], s_scale[w0], acc[q]);
            }
        } else {
            for (int w0 = 0; w0 < M; w0 += BATCH) {         // batches of BATCH code words in flight; rows clamped, tail predicated
                uint32_t wd[BATCH][W];
    #pragma unroll
                for (int k = 0; k < BATCH; ++k) {
                    const uint32_t* wq = words + (int64_t)min(w0 + k, M - 1) * wstride;
                    if (W == 2) { const uint2 u = __ldg(reinterpret_cast<const uint2*>(wq) + t); wd[k][0] = u.x; wd[k][W - 1] = u.y; }
                    else wd[k][0] = __ldg(wq + t);
                }
    #pragma unroll
                for (int k = 0; k < BATCH; ++k) {
                    if (w0 + k < M) {
    #pragma unroll
                        for (int q = 0; q < W; ++q) accumulate_word<BITS>(wd[k][q], s_scale[w0 + k], acc[q]);
                    }
                }
            }
        }
        float* target = ACC ? y : x;
        if (fast && !kEarly) {
#pragma unroll
            for (int q = 0; q < C / 8; ++q) {
                load8(g_full + i0 + q * 8, *reinterpret_cast<float(*)[8]>(gfp + q * 8));
                load8_rw((ACC ? y : x) + i0 + q * 8, *reinterpret_cast<float(*)[8]>(curp + q * 8));
            }
        }
        if (fast) {                                          // 256-bit accesses: every 32-byte sector is used whole
#pragma unroll
            for (int q = 0; q < C / 8; ++q) {
                const int64_t i = i0 + q * 8;
                float xs[8], sm[8], yo[8], xo[8];
                const float* gf = gfp + q * 8; const float* cur = curp + q * 8;
                if (ACC) { load8(xsnap + i, xs); load8_rw(xsum + i, sm); }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (!ACC) { xs[j] = 0.0f; sm[j] = 0.0f; }
                    xo[j] = master_update<ACC>(acc[(q * 8 + j) / CW][(q * 8 + j) % CW], inv_m, eta, theta, thr, den, pp, gf[j], cur[j], xs[j], yo[j], sm[j]);
                    nmax = max(nmax, __float_as_uint(xo[j]) & 0x7FFFFFFFu);
                }
                store8(x + i, xo);
                if (ACC) { store8(y + i, yo); store8(xsum + i, sm); }
            }
        } else if (i0 + C <= d) {
#pragma unroll
            for (int q = 0; q < C / 4; ++q) {
                const int64_t i = i0 + q * 4;
                const float4 gf = *reinterpret_cast<const float4*>(g_full + i);
                const float4 cur = *reinterpret_cast<const float4*>(target + i);
                float4 xs = make_float4(0, 0, 0, 0), sm = make_float4(0, 0, 0, 0), yo, xo;
                if (ACC) { xs = *reinterpret_cast<const float4*>(xsnap + i); sm = *reinterpret_cast<const float4*>(xsum + i); }
                xo.x = master_update<ACC>(acc[(q * 4 + 0) / CW][(q * 4 + 0) % CW], inv_m, eta, theta, thr, den, pp, gf.x, cur.x, xs.x, yo.x, sm.x);
                xo.y = master_update<ACC>(acc[(q * 4 + 1) / CW][(q * 4 + 1) % CW], inv_m, eta, theta, thr, den, pp, gf.y, cur.y, xs.y, yo.y, sm.y);
                xo.z = master_update<ACC>(acc[(q * 4 + 2) / CW][(q * 4 + 2) % CW], inv_m, eta, theta, thr, den, pp, gf.z, cur.z, xs.z, yo.z, sm.z);
                xo.w = master_update<ACC>(acc[(q * 4 + 3) / CW][(q * 4 + 3) % CW], inv_m, eta, theta, thr, den, pp, gf.w, cur.w, xs.w, yo.w, sm.w);
                *reinterpret_cast<float4*>(x + i) = xo;
                if (ACC) { *reinterpret_cast<float4*>(y + i) = yo; *reinterpret_cast<float4*>(xsum + i) = sm; }
                nmax = max(nmax, max(max(__float_as_uint(xo.x) & 0x7FFFFFFFu, __float_as_uint(xo.y) & 0x7FFFFFFFu),
                                     max(__float_as_uint(xo.z) & 0x7FFFFFFFu, __float_as_uint(xo.w) & 0x7FFFFFFFu)));
            }
        } else {
#pragma unroll
            for (int j = 0; j < C; ++j) {
                const int64_t i = i0 + j;
                if (i >= d) break;
                float yo = 0.0f, sm = ACC ? xsum[i] : 0.0f;
                const float xo = master_update<ACC>(acc[j / CW][j % CW], inv_m, eta, theta, thr, den, pp, g_full[i], target[i],
                                                    ACC ? xsnap[i] : 0.0f, yo, sm);
                x[i] = xo;
                if (ACC) { y[i] = yo; xsum[i] = sm; }
                nmax = max(nmax, __float_as_uint(xo) & 0x7FFFFFFFu);
            }
        }
    }
    block_atomic_max(nmax, normx_bits);
    finish_round(rp);
}

// Sparse messages.  One block per tile of kChunk coordinates: the tile's sum is built in shared memory
// worker by worker (indices inside one message are distinct, so no two threads meet), then the prox.
template <int BITS, bool ACC>
__global__ void __launch_bounds__(kThreads)
master_sparse_kernel(const uint8_t* __restrict__ codes, int64_t stride, const float* __restrict__ scale,
                     const uint32_t* __restrict__ idx, int64_t cap, const uint32_t* __restrict__ tile_ptr, int64_t ntiles,
                     int M, int64_t d, const float* __restrict__ g_full, float* __restrict__ x, float* __restrict__ y,
                     const float* __restrict__ xsnap, float* __restrict__ xsum, float eta, float theta, ProxParams pp,
                     uint32_t* __restrict__ normx_bits, const RoundParams* __restrict__ rp, BitsArgs ba)
{
    pdl_prologue();
    if (rp) { eta = rp->eta; theta = rp->theta; }
    if (ba.down && blockIdx.x == 0 && threadIdx.x == 0) write_round_bits(ba, M, d);
    __shared__ float s_acc[kChunk];
    extern __shared__ uint32_t s_seg[];                          // [M][2] list segment of each worker in the tile
    const float inv_m = __fdiv_rn(1.0f, (float)M);
    const float thr = __fmul_rn(eta, pp.lambda1), den = __fadd_rn(1.0f, __fmul_rn(eta, pp.lambda2));
    uint32_t nmax = 0;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t lo = tile * kChunk;
        for (int i = threadIdx.x; i < kChunk; i += blockDim.x) s_acc[i] = 0.0f;
        for (int w = threadIdx.x; w < M; w += blockDim.x) {      // every worker's segment of this tile, fetched at once
            const uint32_t* tp = tile_ptr + (int64_t)w * (ntiles + 1) + tile;
            s_seg[2 * w] = tp[0]; s_seg[2 * w + 1] = tp[1];
        }
        __syncthreads();
        for (int w = 0; w < M; ++w) {                            // worker order is the oracle's order of the fused adds
            const uint32_t e0 = s_seg[2 * w], e1 = s_seg[2 * w + 1];
            if (e0 == e1) continue;                              // nothing from this worker here (uniform for the block)
            const uint32_t* list = idx + (int64_t)w * cap;
            const uint32_t* words = reinterpret_cast<const uint32_t*>(codes + (int64_t)w * stride);
            const float dl = scale[w];
            for (uint32_t e = e0 + threadIdx.x; e < e1; e += blockDim.x) {
                const int64_t bit = (int64_t)e * BITS;
                const int k = code_of<BITS>(__ldg(words + (bit >> 5)), (int)((bit & 31) / BITS));
                const int li = (int)((int64_t)list[e] - lo);
                if ((unsigned)li < (unsigned)kChunk) s_acc[li] = __fmaf_rn((float)k, dl, s_acc[li]);     // a list entry outside its tile is dropped, never followed
            }
            __syncthreads();
        }
        float* target = ACC ? y : x;
        for (int li = threadIdx.x; li < kChunk && lo + li < d; li += blockDim.x) {
            const int64_t i = lo + li;
            float yo = 0.0f, sm = ACC ? xsum[i] : 0.0f;
            const float xo = master_update<ACC>(s_acc[li], inv_m, eta, theta, thr, den, pp, g_full[i], target[i],
                                                ACC ? xsnap[i] : 0.0f, yo, sm);
            x[i] = xo;
            if (ACC) { y[i] = yo; xsum[i] = sm; }
            nmax = max(nmax, __float_as_uint(xo) & 0x7FFFFFFFu);
        }
        __syncthreads();
    }
    block_atomic_max(nmax, normx_bits);
    finish_round(rp);
}

// The 32/BITS codes of one packed word as floats (same conversion-free trick as accumulate_word).
template <int BITS>
__device__ __forceinline__ void codes_as_float(uint32_t word, float (&kf)[32 / BITS])
{
    constexpr float kBias = 8388608.0f + (float)(1 << (BITS - 1));
    if (BITS == 8) {
        const uint32_t wb = word ^ 0x80808080u;
#pragma unroll
        for (int j = 0; j < 4; ++j) kf[j] = __fsub_rn(__uint_as_float(__byte_perm(wb, 0x4B000000u, 0x7540u | j)), kBias);
    } else if (BITS == 4) {
        const uint32_t wb = word ^ 0x88888888u;
        const uint32_t ev = wb & 0x0F0F0F0Fu, od = (wb >> 4) & 0x0F0F0F0Fu;
#pragma unroll
        for (int j = 0; j < 8; ++j) kf[j] = __fsub_rn(__uint_as_float(__byte_perm((j & 1) ? od : ev, 0x4B000000u, 0x7540u | (j >> 1))), kBias);
    } else {
        const uint32_t wb = word ^ 0xAAAAAAAAu;
        uint32_t p[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) p[k] = (wb >> (2 * k)) & 0x03030303u;
#pragma unroll
        for (int j = 0; j < 16; ++j) kf[j] = __fsub_rn(__uint_as_float(__byte_perm(p[j & 3], 0x4B000000u, 0x7540u | (j >> 2))), kBias);
    }
}

// ---------------------------------------------------------------------------------------------------
// Sequential master (Algorithm 1 step 9 as written): one prox step per message, in worker order; message w
// meets a model that is w steps newer than the one it was computed on.  Same traffic as the averaged step,
// M times the update arithmetic.  Each thread owns the 32/BITS coordinates of one code word.
// ---------------------------------------------------------------------------------------------------
template <int BITS, bool ACC>
__global__ void __launch_bounds__(kThreads)
master_dense_seq_kernel(const uint8_t* __restrict__ codes, int64_t stride, const float* __restrict__ scale, int M, int64_t d,
                        const float* __restrict__ g_full, float* __restrict__ x, float* __restrict__ y,
                        const float* __restrict__ xsnap, float* __restrict__ xsum, float eta, float theta, ProxParams pp,
                        uint32_t* __restrict__ normx_bits, const RoundParams* __restrict__ rp, BitsArgs ba)
{
    pdl_prologue();
    if (rp) { eta = rp->eta; theta = rp->theta; }
    if (ba.down && blockIdx.x == 0 && threadIdx.x == 0) write_round_bits(ba, M, d);
    constexpr int C = 32 / BITS;
    extern __shared__ float s_scale[];
    for (int i = threadIdx.x; i < M; i += blockDim.x) s_scale[i] = scale[i];
    __syncthreads();
    const float thr = __fmul_rn(eta, pp.lambda1), den = __fadd_rn(1.0f, __fmul_rn(eta, pp.lambda2));
    const int64_t nwords = (d + C - 1) / C, wstride = stride >> 2;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(codes);
    float* target = ACC ? y : x;
    uint32_t nmax = 0;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < nwords; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i0 = t * C;
        float cur[C], g[C], xs[C], sm[C], xo[C];
        const bool full = i0 + C <= d;                       // whole group inside the vector: 16-byte accesses
        if (full) {
#pragma unroll
            for (int q = 0; q < C / 4; ++q) {
                const float4 c4 = *reinterpret_cast<const float4*>(target + i0 + 4 * q), g4 = *reinterpret_cast<const float4*>(g_full + i0 + 4 * q);
                cur[4 * q] = c4.x; cur[4 * q + 1] = c4.y; cur[4 * q + 2] = c4.z; cur[4 * q + 3] = c4.w;
                g[4 * q] = g4.x; g[4 * q + 1] = g4.y; g[4 * q + 2] = g4.z; g[4 * q + 3] = g4.w;
                if (ACC) {
                    const float4 s4 = *reinterpret_cast<const float4*>(xsnap + i0 + 4 * q), m4 = *reinterpret_cast<const float4*>(xsum + i0 + 4 * q);
                    xs[4 * q] = s4.x; xs[4 * q + 1] = s4.y; xs[4 * q + 2] = s4.z; xs[4 * q + 3] = s4.w;
                    sm[4 * q] = m4.x; sm[4 * q + 1] = m4.y; sm[4 * q + 2] = m4.z; sm[4 * q + 3] = m4.w;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < C; ++j) {
            if (!full) {
                const bool in = i0 + j < d;
                cur[j] = in ? target[i0 + j] : 0.0f; g[j] = in ? g_full[i0 + j] : 0.0f;
                xs[j] = (ACC && in) ? xsnap[i0 + j] : 0.0f; sm[j] = (ACC && in) ? xsum[i0 + j] : 0.0f;
            } else if (!ACC) { xs[j] = 0.0f; sm[j] = 0.0f; }
            xo[j] = cur[j];
        }
#pragma unroll 4
        for (int w = 0; w < M; ++w) {
            const uint32_t word = __ldg(words + (int64_t)w * wstride + t);
            const float dl = s_scale[w];
            float kf[C];
            codes_as_float<BITS>(word, kf);
#pragma unroll
            for (int j = 0; j < C; ++j) {
                float yo = 0.0f;
                xo[j] = master_update<ACC>(kf[j], dl, eta, theta, thr, den, pp, g[j], cur[j], xs[j], yo, sm[j]);
                cur[j] = ACC ? yo : xo[j];
            }
        }
        if (full) {
#pragma unroll
            for (int q = 0; q < C / 4; ++q) {
                *reinterpret_cast<float4*>(x + i0 + 4 * q) = make_float4(xo[4 * q], xo[4 * q + 1], xo[4 * q + 2], xo[4 * q + 3]);
                if (ACC) {
                    *reinterpret_cast<float4*>(y + i0 + 4 * q) = make_float4(cur[4 * q], cur[4 * q + 1], cur[4 * q + 2], cur[4 * q + 3]);
                    *reinterpret_cast<float4*>(xsum + i0 + 4 * q) = make_float4(sm[4 * q], sm[4 * q + 1], sm[4 * q + 2], sm[4 * q + 3]);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < C; ++j) {
            if (i0 + j < d) {
                if (!full) { x[i0 + j] = xo[j]; if (ACC) { y[i0 + j] = cur[j]; xsum[i0 + j] = sm[j]; } }
                nmax = max(nmax, __float_as_uint(xo[j]) & 0x7FFFFFFFu);
            }
        }
    }
    block_atomic_max(nmax, normx_bits);
    finish_round(rp);
}

// Sparse messages, sequential: per tile, every worker's (possibly empty) message is expanded into shared memory and
// followed by a prox sweep over the tile; each thread keeps its eight coordinates of the tile in registers.
template <int BITS, bool ACC>
__global__ void __launch_bounds__(kThreads)
master_sparse_seq_kernel(const uint8_t* __restrict__ codes, int64_t stride, const float* __restrict__ scale,
                         const uint32_t* __restrict__ idx, int64_t cap, const uint32_t* __restrict__ tile_ptr, int64_t ntiles,
                         int M, int64_t d, const float* __restrict__ g_full, float* __restrict__ x, float* __restrict__ y,
                         const float* __restrict__ xsnap, float* __restrict__ xsum, float eta, float theta, ProxParams pp,
                         uint32_t* __restrict__ normx_bits, const RoundParams* __restrict__ rp, BitsArgs ba)
{
    pdl_prologue();
    if (rp) { eta = rp->eta; theta = rp->theta; }
    if (ba.down && blockIdx.x == 0 && threadIdx.x == 0) write_round_bits(ba, M, d);
    constexpr int R = kChunk / kThreads;                       // coordinates of the tile per thread
    __shared__ float s_q[kChunk];
    extern __shared__ uint32_t s_seg[];
    const float thr = __fmul_rn(eta, pp.lambda1), den = __fadd_rn(1.0f, __fmul_rn(eta, pp.lambda2));
    float* target = ACC ? y : x;
    uint32_t nmax = 0;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t lo = tile * kChunk;
        for (int w = threadIdx.x; w < M; w += blockDim.x) {
            const uint32_t* tp = tile_ptr + (int64_t)w * (ntiles + 1) + tile;
            s_seg[2 * w] = tp[0]; s_seg[2 * w + 1] = tp[1];
        }
        float cur[R], g[R], xs[R], sm[R], xo[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int64_t i = lo + threadIdx.x + r * kThreads;
            const bool in = i < d;
            cur[r] = in ? target[i] : 0.0f; g[r] = in ? g_full[i] : 0.0f;
            xs[r] = (ACC && in) ? xsnap[i] : 0.0f; sm[r] = (ACC && in) ? xsum[i] : 0.0f;
            xo[r] = cur[r];
        }
        __syncthreads();
        for (int w = 0; w < M; ++w) {
#pragma unroll
            for (int r = 0; r < R; ++r) s_q[threadIdx.x + r * kThreads] = 0.0f;
            __syncthreads();
            const uint32_t e0 = s_seg[2 * w], e1 = s_seg[2 * w + 1];
            const uint32_t* list = idx + (int64_t)w * cap;
            const uint32_t* words = reinterpret_cast<const uint32_t*>(codes + (int64_t)w * stride);
            for (uint32_t e = e0 + threadIdx.x; e < e1; e += blockDim.x) {
                const int64_t bit = (int64_t)e * BITS;
                const int li = (int)((int64_t)list[e] - lo);
                if ((unsigned)li < (unsigned)kChunk)                               // a list entry outside its tile is dropped, never followed
                    s_q[li] = (float)code_of<BITS>(__ldg(words + (bit >> 5)), (int)((bit & 31) / BITS));
            }
            __syncthreads();
            const float dl = scale[w];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float yo = 0.0f;
                xo[r] = master_update<ACC>(s_q[threadIdx.x + r * kThreads], dl, eta, theta, thr, den, pp, g[r], cur[r], xs[r], yo, sm[r]);
                cur[r] = ACC ? yo : xo[r];
            }
            __syncthreads();
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int64_t i = lo + threadIdx.x + r * kThreads;
            if (i < d) {
                x[i] = xo[r];
                if (ACC) { y[i] = cur[r]; xsum[i] = sm[r]; }
                nmax = max(nmax, __float_as_uint(xo[r]) & 0x7FFFFFFFu);
            }
        }
        __syncthreads();
    }
    block_atomic_max(nmax, normx_bits);
    finish_round(rp);
}

// Test utility: dequantise one message into a dense fp32 vector.
template <int BITS>
__global__ void unpack_dense_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scale, int64_t d,
                                    float* __restrict__ out)
{
    pdl_prologue();
    const float dl = scale[0];
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t bit = i * BITS;
        out[i] = __fmul_rn((float)code_of<BITS>(reinterpret_cast<const uint32_t*>(codes)[bit >> 5], (int)((bit & 31) / BITS)), dl);
    }
}

template <int BITS>
__global__ void unpack_sparse_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scale,
                                     const uint32_t* __restrict__ idx, const uint32_t* __restrict__ nnz,
                                     int64_t d, float* __restrict__ out)
{
    pdl_prologue();
    const float dl = scale[0];
    const uint32_t n = nnz[0];
    for (uint32_t e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int64_t bit = (int64_t)e * BITS;
        if ((int64_t)idx[e] >= d) continue;                                        // a position beyond the vector is dropped
        out[idx[e]] = __fmul_rn((float)code_of<BITS>(reinterpret_cast<const uint32_t*>(codes)[bit >> 5], (int)((bit & 31) / BITS)), dl);
    }
}

// ---------------------------------------------------------------------------------------------------
// Sparse gradients.  The worker kernel marks every group of eight coordinates it adds to in a bitmap.
// build_group_list turns each worker's bitmap into the ascending list of those groups, clears the bitmap,
// turns the integer accumulator of the listed groups into alpha_w (one rounding to fp32; the accumulator is
// zeroed again) and folds ||alpha_w||_inf over them (all other coordinates are zero).
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
count_touched_kernel(const uint32_t* __restrict__ touched, int64_t bm_words, uint32_t* __restrict__ seg_count, int nseg)
{
    pdl_prologue();
    // grid (nseg, M): set bits of one segment of kThreads bitmap words
    const int w = blockIdx.y;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t c = (i < bm_words) ? __popc(touched[(int64_t)w * bm_words + i]) : 0u;
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    __shared__ uint32_t s_c[kThreads / 32];
    if ((threadIdx.x & 31) == 0) s_c[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (int k = 0; k < (int)(blockDim.x >> 5); ++k) t += s_c[k];
        seg_count[(int64_t)w * nseg + blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(kThreads)
build_group_list_kernel(uint32_t* __restrict__ touched, uint32_t* __restrict__ ptouched /* may be NULL */, int64_t bm_words, const uint32_t* __restrict__ seg_count, int nseg,
                        FixedAcc fa, float* __restrict__ alpha, int64_t d,
                        uint32_t* __restrict__ glist, int64_t cap, uint32_t* __restrict__ gcount, uint32_t* __restrict__ norm_bits)
{
    pdl_prologue();
    // grid (nseg, M): this segment's groups go to the list after those of the segments before it
    const int w = blockIdx.y;
    uint32_t* bm = touched + (int64_t)w * bm_words;
    uint32_t* list = glist + (int64_t)w * cap;
    float* row = alpha + (int64_t)w * d;
    long long* acc = fa.acc + (int64_t)w * d;
    __shared__ uint32_t s_warp[kThreads / 32];
    __shared__ uint32_t s_base[kThreads / 32];
    // base = sum of the earlier segments' counts (all threads help)
    uint32_t part = 0;
    for (int k = threadIdx.x; k < (int)blockIdx.x; k += blockDim.x) part += seg_count[(int64_t)w * nseg + k];
    part = __reduce_add_sync(0xFFFFFFFFu, part);
    if ((threadIdx.x & 31) == 0) s_base[threadIdx.x >> 5] = part;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t word = 0;
    if (i < bm_words) {
        word = bm[i]; if (word) bm[i] = 0u;
        if (ptouched) ptouched[(int64_t)w * bm_words + i] = word;      // kept for the kernel that works from bitmaps (sparse_message_kernel)
    }
    const uint32_t c = __popc(word);
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if ((threadIdx.x & 31) >= o) incl += t; }
    if ((threadIdx.x & 31) == 31) s_warp[threadIdx.x >> 5] = incl;
    __syncthreads();
    uint32_t pos = incl - c;
    for (int k = 0; k < (int)(blockDim.x >> 5); ++k) { pos += s_base[k]; if (k < (int)(threadIdx.x >> 5)) pos += s_warp[k]; }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == blockDim.x - 1) gcount[w] = pos + c;     // the last word closes the list
    uint32_t nmax = 0;
    while (word) {
        const int bit = __ffs(word) - 1; word &= word - 1;
        const int64_t g = (i << 5) + bit, i0 = g << 3;
        list[pos++] = (uint32_t)g;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (i0 + j < d) {
                const long long q = acc[i0 + j];
                if (q != 0) acc[i0 + j] = 0;
                const float a = (float)((double)q * fa.inv_scale);
                row[i0 + j] = a;
                nmax = max(nmax, __float_as_uint(a) & 0x7FFFFFFFu);
            }
        }
    }
    block_atomic_max(nmax, norm_bits + w);
}

// Puts back zeros in the groups listed by the previous round, so that alpha is all-zero again.  grid (blocks, M).
__global__ void __launch_bounds__(kThreads)
clear_listed_groups_kernel(float* __restrict__ alpha, int64_t d, const uint32_t* __restrict__ glist, int64_t cap,
                           const uint32_t* __restrict__ gcount)
{
    pdl_prologue();
    const int w = blockIdx.y;
    float* row = alpha + (int64_t)w * d;
    const int64_t n = gcount[w];
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < n; p += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i0 = (int64_t)glist[(int64_t)w * cap + p] << 3;
#pragma unroll
        for (int j = 0; j < 8; ++j) if (i0 + j < d) row[i0 + j] = 0.0f;
    }
}

// ---------------------------------------------------------------------------------------------------
// Sparse gradient -> sparse message in one kernel (CSR data, sparsifier of eq. (4), (position, code) messages).
// From the integer accumulator and the bitmap of touched groups that the worker kernel leaves behind to the
// finished message of Section 3.1 and the master's tile pointers; the steps are those of the stand-alone kernels
// (list of touched groups, alpha and ||alpha||_inf, integer-grid ||alpha||_1, survivor mask, ||beta||_inf, quantise
// and emit in ascending order) with the same draws and arithmetic.  A worker is served by a thread-block cluster
// of kMsgCluster blocks, each owning a range of the bitmap and the groups listed in it.  A round touches a few
// thousand groups per worker, so the kernel's time is a chain of memory round trips: a block keeps its groups'
// numbers in shared memory and (up to kMsgKeep groups per thread) their values in registers, so that only the
// accumulator is read from memory; the three points where a step needs a value over the whole worker (list length
// with ||alpha||_inf, ||alpha||_1, survivor counts with ||beta||_inf) are cluster barriers, with the blocks'
// partial values written into each other's shared memory.  A block with more groups than it can keep re-reads
// them (group numbers from a scratch list, values from alpha).
// grid (kMsgCluster, M), cluster (kMsgCluster, 1, 1), kMsgThreads threads.
// ---------------------------------------------------------------------------------------------------
constexpr int kMsgCluster = 4;
constexpr int kMsgThreads = 512;
constexpr int kMsgKeep = 2;                       // groups per thread whose values stay in registers

struct SparseMsg {
    uint32_t* touched; uint32_t* ptouched; int64_t bm_words;    // [M][bm_words] bitmaps of touched groups: this round's (cleared here) and
                                                  // the previous round's (whose groups get their zeros back; replaced by this round's)
    FixedAcc fa;                                  // integer accumulator (zeroed again here)
    float* alpha; int64_t d;                      // [M][d] receives alpha_w; zero outside the listed groups
    uint32_t* glist; uint32_t* gtmp; int64_t gcap; uint32_t* gcount;   // ascending list of touched groups (out), scratch of the same size
    uint32_t* norm_bits; unsigned long long* l1_sum; uint32_t* beta_norm_bits;     // [M] each, written here
    float phi; uint32_t round; const RoundParams* rp;
    uint8_t* codes; int64_t stride; float* scale; uint32_t* idx; int64_t cap; uint32_t* nnz;    // the messages
    uint32_t* tile_ptr; int64_t ntiles;           // [M][ntiles + 1] first list entry of every tile of kChunk coordinates
    int* status;
};

template <int BITS>
__global__ void __launch_bounds__(kMsgThreads, 1)
sparse_message_kernel(const __grid_constant__ SparseMsg A, const __grid_constant__ PhiloxKeys K)
{
    pdl_prologue();
    constexpr int NW = kMsgThreads / 32, kKeepCap = kMsgKeep * kMsgThreads;
    const int w = blockIdx.y, r = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ uint32_t s_scan[NW];
    __shared__ unsigned long long s_red[NW];
    __shared__ uint32_t s_list[kKeepCap];
    __shared__ __align__(16) unsigned long long s_ex[3][kMsgCluster][2];      // written by the cluster's blocks, one pair each
    const uint32_t round = A.rp ? A.rp->round : A.round;
    const int64_t d = A.d;
    uint32_t* bm = A.touched + (int64_t)w * A.bm_words;
    uint32_t* pbm = A.ptouched + (int64_t)w * A.bm_words;
    float* row = A.alpha + (int64_t)w * d;
    long long* acc = A.fa.acc + (int64_t)w * d;
    const bool vec = (d & 7) == 0;                            // every group of a row starts on a 32-byte boundary

    // sum or maximum of one value per thread over the block (every thread gets the result)
    auto block_reduce = [&](unsigned long long v, bool is_max) -> unsigned long long {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const unsigned long long t = __shfl_xor_sync(0xFFFFFFFFu, v, o); v = is_max ? (t > v ? t : v) : v + t; }
        if (lane == 0) s_red[warp] = v;
        __syncthreads();
        unsigned long long tot = 0;
        for (int k = 0; k < NW; ++k) tot = is_max ? (s_red[k] > tot ? s_red[k] : tot) : tot + s_red[k];
        __syncthreads();
        return tot;
    };
    // exclusive prefix of one count per thread in thread order, and the block's total
    auto block_scan = [&](uint32_t c, uint32_t& total) -> uint32_t {
        uint32_t incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t; }
        if (lane == 31) s_scan[warp] = incl;
        __syncthreads();
        uint32_t base = 0, tot = 0;
        for (int k = 0; k < NW; ++k) { const uint32_t t = s_scan[k]; if (k < warp) base += t; tot += t; }
        __syncthreads();
        total = tot;
        return base + incl - c;
    };
    // every block hands its pair (v0, v1) to all blocks of the cluster (slot = which of the three meetings)
    unsigned long long all0[kMsgCluster], all1[kMsgCluster];
    auto exchange = [&](int slot, unsigned long long v0, unsigned long long v1) {
        if (tid < kMsgCluster) {
            const uint32_t local = (uint32_t)__cvta_generic_to_shared(&s_ex[slot][r][0]);
            uint32_t remote;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(tid));
            asm volatile("st.shared::cluster.v2.u64 [%0], {%1, %2};" :: "r"(remote), "l"(v0), "l"(v1) : "memory");
        }
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
#pragma unroll
        for (int k = 0; k < kMsgCluster; ++k) { all0[k] = s_ex[slot][k][0]; all1[k] = s_ex[slot][k][1]; }
    };
    // alpha is written in this kernel: no read-only path for its loads
    auto load_group = [&](int64_t i0, float (&a)[8]) {
        if (vec) { load8_rw(row + i0, a); return; }
#pragma unroll
        for (int j = 0; j < 8; ++j) a[j] = (i0 + j < d) ? *reinterpret_cast<volatile float*>(row + i0 + j) : 0.0f;
    };

    // ---- 0: zero this worker's code words; in this block's range of the bitmaps: zeros back into the groups of the
    //         previous round, this round's groups to the block's list, bitmaps rolled over
    {
        uint4* c16 = reinterpret_cast<uint4*>(A.codes + (int64_t)w * A.stride);            // stride is a multiple of 16
        for (int64_t q = (int64_t)r * kMsgThreads + tid; q < (A.stride >> 4); q += kMsgCluster * kMsgThreads) c16[q] = make_uint4(0u, 0u, 0u, 0u);
    }
    const int64_t wpb = (A.bm_words + kMsgCluster - 1) / kMsgCluster;
    const int64_t w0 = (int64_t)r * wpb, w1 = min(A.bm_words, w0 + wpb);
    uint32_t* tmp = A.gtmp + (int64_t)w * A.gcap + (w0 << 5);           // this block's scratch list: it has at most 32 groups per word
    uint32_t cl = 0;                                          // groups listed by this block
    for (int64_t i = w0; i < w1; i += kMsgThreads) {
        const int64_t wi = i + tid;
        uint32_t word = 0, old = 0;
        if (wi < w1) { word = bm[wi]; old = pbm[wi]; }
        if (word != old) pbm[wi] = word;
        if (word) bm[wi] = 0u;
        while (old) {
            const int bit = __ffs(old) - 1; old &= old - 1;
            const int64_t i0 = ((wi << 5) + bit) << 3;
            if (vec) { float4* q = reinterpret_cast<float4*>(row + i0); q[0] = make_float4(0.f, 0.f, 0.f, 0.f); q[1] = make_float4(0.f, 0.f, 0.f, 0.f); }
            else for (int j = 0; j < 8; ++j) if (i0 + j < d) row[i0 + j] = 0.0f;
        }
        uint32_t total;
        uint32_t pos = cl + block_scan(__popc(word), total);
        while (word) {
            const int bit = __ffs(word) - 1; word &= word - 1;
            const uint32_t g = (uint32_t)((wi << 5) + bit);
            if (pos < (uint32_t)kKeepCap) s_list[pos] = g;
            tmp[pos++] = g;
        }
        cl += total;
    }
    __syncthreads();                                          // the zeros are in place before alpha is stored; the list is complete
    const bool keep = cl <= (uint32_t)kKeepCap;               // this block's groups fit shared memory and registers
    const uint32_t g_last = cl ? (keep ? s_list[cl - 1] : __ldcg(tmp + cl - 1)) : 0u;
    auto group_at_entry = [&](uint32_t e) -> uint32_t { return keep ? s_list[e] : __ldcg(tmp + e); };

    // ---- 1: accumulator -> alpha (one rounding to fp32), accumulator zeroed, ||alpha||_inf
    float ka[kMsgKeep][8];
    uint32_t kg[kMsgKeep], kmask[kMsgKeep];
    uint32_t amax = 0;
    auto make_alpha = [&](uint32_t g, float (&a)[8]) {
        const int64_t i0 = (int64_t)g << 3;
        long long q[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) q[j] = (i0 + j < d) ? acc[i0 + j] : 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            a[j] = 0.0f;
            if (q[j] != 0) {                                  // (most coordinates of a touched group are untouched)
                acc[i0 + j] = 0;
                a[j] = (float)((double)q[j] * A.fa.inv_scale);
                amax = max(amax, __float_as_uint(a[j]) & 0x7FFFFFFFu);
            }
        }
        if (vec) {
            float4* o = reinterpret_cast<float4*>(row + i0);
            o[0] = make_float4(a[0], a[1], a[2], a[3]); o[1] = make_float4(a[4], a[5], a[6], a[7]);
        } else {
            for (int j = 0; j < 8; ++j) if (i0 + j < d) row[i0 + j] = a[j];
        }
    };
    if (keep) {
#pragma unroll
        for (int k = 0; k < kMsgKeep; ++k) {
            const uint32_t e = tid + k * kMsgThreads;
            kg[k] = 0; kmask[k] = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) ka[k][j] = 0.0f;
            if (e < cl) { kg[k] = s_list[e]; make_alpha(kg[k], ka[k]); }
        }
    } else {
        for (uint32_t e = tid; e < cl; e += kMsgThreads) { float a[8]; make_alpha(__ldcg(tmp + e), a); }
    }
    exchange(0, ((unsigned long long)cl << 32) | block_reduce(amax, true), g_last);
    uint32_t base = 0, count = 0, nb = 0;
    int64_t t_before = -1;                                    // tile of the last group listed by a block before this one
    bool last_block = true;                                   // no block after this one lists a group
#pragma unroll
    for (int k = 0; k < kMsgCluster; ++k) {
        const uint32_t c = (uint32_t)(all0[k] >> 32);
        if (k < r) { base += c; if (c) t_before = (int64_t)((uint32_t)all1[k] >> 8); }
        if (k > r && c) last_block = false;
        count += c; nb = max(nb, (uint32_t)all0[k]);
    }
    {   // the worker's list: this block's groups after those of the blocks before it
        uint32_t* list = A.glist + (int64_t)w * A.gcap + base;
        for (uint32_t e = tid; e < cl; e += kMsgThreads) list[e] = group_at_entry(e);
        if (r == 0 && tid == 0) { A.gcount[w] = count; A.norm_bits[w] = nb; }
    }

    // ---- 2: ||alpha||_1 on the integer grid of ||alpha||_inf's exponent
    unsigned long long l1 = 0;
    if (nb != 0u && nb < 0x7F800000u) {
        int ee; (void)frexpf(__uint_as_float(nb), &ee);
        if (keep) {
#pragma unroll
            for (int k = 0; k < kMsgKeep; ++k)
#pragma unroll
                for (int j = 0; j < 8; ++j) l1 += l1_term(ka[k][j], ee);              // (entries beyond the list hold zeros)
        } else {
            for (uint32_t e = tid; e < cl; e += kMsgThreads) {
                float a[8]; load_group((int64_t)__ldcg(tmp + e) << 3, a);
#pragma unroll
                for (int j = 0; j < 8; ++j) l1 += l1_term(a[j], ee);
            }
        }
    }
    exchange(1, block_reduce(l1, false), 0ull);
    l1 = 0;
#pragma unroll
    for (int k = 0; k < kMsgCluster; ++k) l1 += all0[k];
    if (r == 0 && tid == 0) A.l1_sum[w] = l1;
    const SparsifyScale sc = sparsify_scale(nb, l1, A.phi);

    // ---- 3: survivor mask of every listed group: survivors and ||beta||_inf
    uint32_t nsurv = 0, bmax = 0;
    auto draw_mask = [&](uint32_t g, const float (&a)[8], float (&beta)[8]) -> uint32_t {
        uint32_t rr[4];
        philox4x32_10(g, round, (uint32_t)w, kStreamMask, K, rr);
        return sparsify8(a, sc.s, rr, beta);
    };
    auto count_mask = [&](uint32_t mask, const float (&beta)[8]) {
        if (mask) {
            nsurv += __popc(mask);
#pragma unroll
            for (int j = 0; j < 8; ++j) bmax = max(bmax, __float_as_uint(beta[j]) & 0x7FFFFFFFu);
        }
    };
    if (!sc.empty) {
        if (keep) {
#pragma unroll
            for (int k = 0; k < kMsgKeep; ++k) {
                if (tid + k * kMsgThreads < cl) {
                    float beta[8];
                    kmask[k] = draw_mask(kg[k], ka[k], beta);
                    count_mask(kmask[k], beta);
#pragma unroll
                    for (int j = 0; j < 8; ++j) ka[k][j] = beta[j];               // from here on the registers hold beta
                }
            }
        } else {
            for (uint32_t e = tid; e < cl; e += kMsgThreads) {
                const uint32_t g = __ldcg(tmp + e);
                float a[8], beta[8]; load_group((int64_t)g << 3, a);
                count_mask(draw_mask(g, a, beta), beta);
            }
        }
    }
    exchange(2, (block_reduce(nsurv, false) << 32) | block_reduce(bmax, true), 0ull);
    uint32_t offset = 0, total = 0, bb = 0;
#pragma unroll
    for (int k = 0; k < kMsgCluster; ++k) {
        const uint32_t c = (uint32_t)(all0[k] >> 32);
        if (k < r) offset += c;
        total += c; bb = max(bb, (uint32_t)all0[k]);
    }
    const bool finite = bb < 0x7F800000u && nb < 0x7F800000u;
    const float bnrm = __uint_as_float(bb);
    const float inv = (finite && bb != 0u) ? __fdiv_rd((float)levels(BITS), bnrm) : 0.0f;
    const uint32_t nnzc = (int64_t)total > A.cap ? (uint32_t)A.cap : total;
    if (r == 0 && tid == 0) {
        A.beta_norm_bits[w] = bb;
        A.scale[w] = (finite && bb != 0u) ? __fdiv_rn(bnrm, (float)levels(BITS)) : 0.0f;
        A.nnz[w] = nnzc;
        if (!finite) set_status(A.status, DQ_ERR_NONFINITE);
        if ((int64_t)total > A.cap) set_status(A.status, DQ_ERR_CAPACITY);
    }

    // ---- 4: quantise the survivors (delta = ||beta||_inf / L, rounding draw keyed by the coordinate) and emit
    //         (position, code) in ascending order; the master's tile pointers from neighbouring groups
    uint8_t* out = A.codes + (int64_t)w * A.stride;
    uint32_t* oidx = A.idx + (int64_t)w * A.cap;
    uint32_t* tp = A.tile_ptr + (int64_t)w * (A.ntiles + 1);
    constexpr int kTileShift = 8;                             // kChunk coordinates = 256 groups
    static_assert(kChunk == 8 << kTileShift, "tile of kChunk coordinates");
    if (count == 0) {
        for (int64_t t = (int64_t)r * kMsgThreads + tid; t <= A.ntiles; t += kMsgCluster * kMsgThreads) tp[t] = 0u;
        return;
    }
    auto emit = [&](uint32_t e, uint32_t g, uint32_t mask, const float (&beta)[8], uint32_t p) {
        // tiles that begin between the previous group and this one start at this group's first survivor
        const int64_t t_cur = g >> kTileShift, t_prev = e > 0 ? (int64_t)(group_at_entry(e - 1) >> kTileShift) : t_before;
        const uint32_t pc = p < nnzc ? p : nnzc;
        for (int64_t t = t_prev + 1; t <= t_cur; ++t) tp[t] = pc;
        if (last_block && e == cl - 1) for (int64_t t = t_cur + 1; t <= A.ntiles; ++t) tp[t] = nnzc;
        if (!mask) return;
        uint32_t rr[4];
        philox4x32_10(g, round, (uint32_t)w, kStreamGrad, K, rr);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if ((mask >> j) & 1u) {
                if ((int64_t)p < A.cap) {
                    const uint32_t s8 = round_fixed<BITS>(beta[j], inv, half16(rr, j));
                    oidx[p] = (g << 3) + (uint32_t)j;
                    const uint32_t field = ((s8 >> 16) ^ (BITS == 8 ? 0x80u : 0u)) & ((1u << BITS) - 1u);
                    const int64_t bit = (int64_t)p * BITS;
                    atomicOr(reinterpret_cast<uint32_t*>(out) + (bit >> 5), field << (bit & 31));
                }
                ++p;
            }
        }
    };
    uint32_t run = offset;
    if (keep) {
#pragma unroll
        for (int k = 0; k < kMsgKeep; ++k) {
            if ((uint32_t)(k * kMsgThreads) >= cl) break;             // (the same for the whole block)
            const uint32_t e = tid + k * kMsgThreads;
            uint32_t tile_total;
            const uint32_t p = run + block_scan(__popc(kmask[k]), tile_total);
            run += tile_total;
            if (e < cl) emit(e, kg[k], kmask[k], ka[k], p);
        }
    } else {
        for (uint32_t eb = 0; eb < cl; eb += kMsgThreads) {
            const uint32_t e = eb + tid;
            uint32_t g = 0, mask = 0;
            float beta[8];
            if (e < cl) {
                g = __ldcg(tmp + e);
                if (!sc.empty) { float a[8]; load_group((int64_t)g << 3, a); mask = draw_mask(g, a, beta); }
            }
            uint32_t tile_total;
            const uint32_t p = run + block_scan(__popc(mask), tile_total);
            run += tile_total;
            if (e < cl) emit(e, g, mask, beta, p);
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// Model precision, condition (3): sums of frac (1 - frac) of x / delta_b for b = 2..11 (the expected squared
// error of rule (i) in units of delta_b^2; the widths of Table 1) and ||x - xsnap||^2, in double.
// stats [kWidths + 1] must be zero on entry.
// ---------------------------------------------------------------------------------------------------
constexpr int kWidths = 10;          // candidate widths 2..11

__global__ void __launch_bounds__(kThreads)
model_precision_kernel(const float* __restrict__ x, const float* __restrict__ xsnap, int64_t d, const uint32_t* __restrict__ norm_bits,
                       double* __restrict__ stats)
{
    pdl_prologue();
    const float nrm = __uint_as_float(norm_bits[0]);
    double inv[kWidths];
#pragma unroll
    for (int k = 0; k < kWidths; ++k) inv[k] = nrm > 0.0f ? 1.0 / (double)__fdiv_rn(nrm, (float)levels(k + 2)) : 0.0;
    // The kernel is bound by the double-precision pipe, so the fraction costs as few of its operations as exactness
    // allows: with M = 1.5 * 2^52, x inv + M rounded toward -inf is M + floor(x inv) (one fused operation), M minus that
    // is -floor exactly, a second fused operation gives frac = x inv - floor rounded once, and frac (1 - frac) is
    // accumulated as sum frac - sum frac^2: five operations per width.
    const double kMagic = 6755399441055744.0;
    double s1[kWidths], s2[kWidths], dist = 0.0;
#pragma unroll
    for (int k = 0; k < kWidths; ++k) { s1[k] = 0.0; s2[k] = 0.0; }
    auto one = [&](float xf, float sf) {
        const double xi = (double)xf, df = xi - (double)sf;
#pragma unroll
        for (int k = 0; k < kWidths; ++k) {
            const double nfl = kMagic - __fma_rd(xi, inv[k], kMagic);
            const double fr = fma(xi, inv[k], nfl);
            s1[k] += fr; s2[k] = fma(fr, fr, s2[k]);
        }
        dist = fma(df, df, dist);
    };
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, nth = (int64_t)gridDim.x * blockDim.x;
    const bool vec = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(xsnap)) & 15) == 0;
    const int64_t nq = vec ? (d >> 2) : 0;
    for (int64_t q = tid; q < nq; q += nth) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(x) + q), b = __ldg(reinterpret_cast<const float4*>(xsnap) + q);
        one(a.x, b.x); one(a.y, b.y); one(a.z, b.z); one(a.w, b.w);
    }
    for (int64_t i = (nq << 2) + tid; i < d; i += nth) one(x[i], xsnap[i]);
    double acc[kWidths + 1];
#pragma unroll
    for (int k = 0; k < kWidths; ++k) acc[k] = s1[k] - s2[k];
    acc[kWidths] = dist;
    __shared__ double s_part[kThreads / 32][kWidths + 1];
#pragma unroll
    for (int k = 0; k <= kWidths; ++k) {
        double v = acc[k];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5][k] = v;
    }
    __syncthreads();
    if (threadIdx.x <= kWidths) {
        double t = 0.0;
        for (int k = 0; k < (int)(blockDim.x >> 5); ++k) t += s_part[k][threadIdx.x];
        atomicAdd(stats + threadIdx.x, t);
    }
}

// Smallest width whose expected error is within mu ||x - xsnap||^2 (Algorithm 3: theta mu), 11 if none.
__global__ void select_bits_kernel(double* __restrict__ stats, const uint32_t* __restrict__ norm_bits, float mu, int accelerated,
                                   float theta, const RoundParams* __restrict__ rp, int32_t* __restrict__ bits)
{
    pdl_prologue();
    if (rp) theta = rp->theta;
    const float nrm = __uint_as_float(norm_bits[0]);
    const double mu_eff = accelerated ? (double)__fmul_rn(theta, mu) : (double)mu;
    int chosen = kWidths + 1;
    for (int b = kWidths + 1; b >= 2; --b) {
        const double delta = nrm > 0.0f ? (double)__fdiv_rn(nrm, (float)levels(b)) : 0.0;
        const double e = stats[b - 2] * delta * delta;
        stats[b - 2] = e;
        if (e <= mu_eff * stats[kWidths]) chosen = b;
    }
    *bits = chosen;
}

// ---------------------------------------------------------------------------------------------------
// Q_(delta,b) + pack for any width 2..11 (the model widths of Table 1 that do not divide eight: 3, 5, 6, 7, and
// 9..11 bits).  The fixed-point position is r = fl(v inv + 1.5 2^e), e = 8 up to 8-bit codes and b beyond, whose
// significand holds (t + 2^(e-1)) 2^(23-e); the top 23-e bits of the coordinate's draw are added and the fraction
// dropped (15 fractional bits up to 8-bit codes, then 14, 13, 12).  A group of eight coordinates is b bytes of
// the message, the codes laid end to end.  One vector (the model); width = *bits_dev if given (then the kernel
// leaves 2, 4 and 8 bits to the kernels specialised for them), else bits_fixed.  With diff also writes
// code * delta - ref and clears the next stages' accumulators, like quantize_pack_kernel<.., true>.
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
quantize_pack_any_kernel(const float* __restrict__ v, int64_t d, const uint32_t* __restrict__ norm_bits, uint8_t* __restrict__ codes,
                         float* __restrict__ scale, const __grid_constant__ PhiloxKeys K, uint32_t round, uint32_t worker,
                         uint32_t stream, int* __restrict__ status, const RoundParams* __restrict__ rp,
                         const float* __restrict__ ref, float* __restrict__ diff, float* __restrict__ zero_f, int64_t zero_n,
                         uint32_t* __restrict__ zero_u, int zero_un, int bits_fixed, const int32_t* __restrict__ bits_dev, int ring)
{
    pdl_prologue();
    const int bits = bits_dev ? *bits_dev : bits_fixed;
    if (bits < 2 || bits > 11 || (bits_dev && (bits == 2 || bits == 4 || bits == 8))) return;
    if (rp) round = rp->round;
    if (diff && rp && ring > 1) diff += (int64_t)(rp->t_epoch % (uint32_t)ring) * d;
    const int64_t nth = (int64_t)gridDim.x * blockDim.x, tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (diff) {
        for (int64_t i = tid; i < zero_n; i += nth) zero_f[i] = 0.0f;
        for (int64_t i = tid; i < zero_un; i += nth) zero_u[i] = 0u;
    }
    const uint32_t nb = norm_bits[0];
    const float nrm = __uint_as_float(nb);
    const bool ok = nb < 0x7F800000u && nb != 0u;
    const float Lf = (float)levels(bits);
    const float inv = ok ? __fdiv_rd(Lf, nrm) : 0.0f;
    const float delta = ok ? __fdiv_rn(nrm, Lf) : 0.0f;
    if (tid == 0) { scale[0] = delta; if (nb >= 0x7F800000u) set_status(status, DQ_ERR_NONFINITE); }
    const int e = bits <= 8 ? 8 : bits, fb = 23 - e;
    const float off = 1.5f * (float)(1 << e);
    const int half = 1 << (e - 1);
    const uint32_t mask = (1u << bits) - 1u;
    const int64_t nbytes = ((d * bits + 7) / 8 + 15) / 16 * 16;
    const int64_t ngroups = (d + 7) >> 3;
    for (int64_t g = tid; g < ngroups; g += nth) {
        float a[8];
        const int64_t i0 = g << 3;
        load8_guarded(v, i0, d, a);
        uint32_t r[4];
        philox4x32_10((uint32_t)g, round, worker, stream, K, r);
        unsigned long long lo = 0, hi = 0;                    // the group's 8 b <= 88 bits
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t F = __float_as_uint(__fmaf_rn(a[j], inv, off)) & 0x007FFFFFu;
            const int code = ok ? (int)((F + (half16(r, j) >> (16 - fb))) >> fb) - half : 0;    // zero or non-finite norm: code 0
            const unsigned long long field = (unsigned long long)((uint32_t)code & mask);
            const int pos = j * bits;
            if (pos < 64) { lo |= field << pos; if (pos + bits > 64) hi |= field >> (64 - pos); }
            else hi |= field << (pos - 64);
            if (diff && i0 + j < d) diff[i0 + j] = __fsub_rn(__fmul_rn((float)code, delta), ref ? ref[i0 + j] : 0.0f);
        }
        for (int k = 0; k < bits; ++k) {
            const int64_t p = g * bits + k;
            if (p < nbytes) codes[p] = (uint8_t)((k < 8 ? lo >> (8 * k) : hi >> (8 * (k - 8))) & 0xFFu);
        }
    }
    for (int64_t p = ngroups * bits + tid; p < nbytes; p += nth) codes[p] = 0;     // padding behind the last group
}

// code * delta - ref for packed codes of any width (see quantize_pack_any_kernel for the layout).
__global__ void __launch_bounds__(kThreads)
dequant_diff_any_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ delta_x, const float* __restrict__ ref, int64_t d,
                        float* __restrict__ diff, int bits)
{
    pdl_prologue();
    const float dl = *delta_x;
    const int64_t nbytes = ((d * bits + 7) / 8 + 15) / 16 * 16;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t bit = i * bits, p = bit >> 3;
        uint32_t w = codes[p];
        if (p + 1 < nbytes) w |= (uint32_t)codes[p + 1] << 8;
        if (p + 2 < nbytes) w |= (uint32_t)codes[p + 2] << 16;
        const int k = ((int)((w >> (bit & 7)) << (32 - bits))) >> (32 - bits);
        diff[i] = __fsub_rn(__fmul_rn((float)k, dl), ref ? ref[i] : 0.0f);
    }
}

// ---------------------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------------------
static inline int grid_for(int64_t items_per_thread_units, int sm_count, int per_sm = 8)
{
    int64_t need = (items_per_thread_units + kThreads - 1) / kThreads;
    int64_t cap = (int64_t)sm_count * per_sm;
    if (need < 1) need = 1;
    return (int)(need < cap ? need : cap);
}

static inline int vec_ok_for(const float* v, int64_t d) { return ((reinterpret_cast<uintptr_t>(v) & 31) == 0 && (d & 7) == 0) ? 1 : 0; }

void launch_norm_inf(dq_ctx* ctx, const float* v, int64_t d, int M, uint32_t* norm_bits, cudaStream_t st)
{
    if (!ctx->ninf_zeroed) cudaMemsetAsync(norm_bits, 0, sizeof(uint32_t) * M, st);
    dim3 grid(grid_for((d + 7) / 8, ctx->sm_count), M);
    launch_k(norm_inf_kernel, grid, kThreads, 0, st, v, d, vec_ok_for(v, d), norm_bits);
    ctx->launches += 1;
}

void launch_quantize_pack(dq_ctx* ctx, const float* v, int64_t d, int M, int bits, const uint32_t* norm_bits,
                          uint8_t* codes, int64_t stride, float* scale, uint32_t round, uint32_t worker_base,
                          uint32_t stream_id, cudaStream_t st, const float* ref, float* diff, float* zero_f, int64_t zero_n,
                          uint32_t* zero_u, int zero_un, const int32_t* bits_gate)
{
    if (bits != 2 && bits != 4 && bits != 8) {                 // a width that does not divide eight: one vector, general kernel
        launch_k(quantize_pack_any_kernel, grid_for((d + 7) / 8, ctx->sm_count), kThreads, 0, st, v, d, norm_bits, codes, scale, ctx->keys,
                 round, worker_base, stream_id, ctx->status, ctx->rp_active, ref, diff, zero_f, zero_n, zero_u, zero_un, bits, bits_gate, ctx->diff_ring);
        ctx->launches += 1;
        return;
    }
    const int64_t ngroups = dq_packed_bytes(d, bits) / bits;
    dim3 grid(grid_for(ngroups, ctx->sm_count), M);
    if (diff) {
        grid.x = max(grid.x, (unsigned)grid_for(zero_n / 4, ctx->sm_count));   // enough blocks for the clearing loop too
        DQ_DISPATCH_BITS(bits, (launch_k(quantize_pack_kernel<BITS_, true>, grid, kThreads, 0, st, v, d, vec_ok_for(v, d), norm_bits, codes, stride, scale, ctx->keys, round, worker_base, stream_id, ngroups, ctx->status,
            ctx->rp_active, ref, diff, zero_f, zero_n, zero_u, zero_un, bits_gate, ctx->diff_ring)));
        ctx->launches += 1;
        return;
    }
    DQ_DISPATCH_BITS(bits, (launch_k(quantize_pack_kernel<BITS_>, grid, kThreads, 0, st, v, d, vec_ok_for(v, d), norm_bits, codes, stride, scale, ctx->keys, round, worker_base, stream_id, ngroups, ctx->status, ctx->rp_active, nullptr, nullptr, nullptr, 0, nullptr, 0, nullptr, 0)));
    ctx->launches += 1;
}

void launch_select_bits(dq_ctx* ctx, const float* x, const float* xsnap, const uint32_t* norm_bits, float mu, int accelerated,
                        float theta, int32_t* bits, double* stats, cudaStream_t st)
{
    cudaMemsetAsync(stats, 0, sizeof(double) * (kWidths + 1), st);
    launch_k(model_precision_kernel, grid_for(ctx->cfg.d / 2 + 1, ctx->sm_count, 4), kThreads, 0, st, x, xsnap, ctx->cfg.d, norm_bits, stats);
    launch_k(select_bits_kernel, 1, 1, 0, st, stats, norm_bits, mu, accelerated, theta, ctx->rp_active, bits);
    ctx->launches += 2;
}

void launch_dequant_diff_any(dq_ctx* ctx, const uint8_t* codes, const float* delta_x, const float* ref, float* diff, int bits, cudaStream_t st)
{
    launch_k(dequant_diff_any_kernel, grid_for(ctx->cfg.d, ctx->sm_count), kThreads, 0, st, codes, delta_x, ref, ctx->cfg.d, diff, bits);
    ctx->launches += 1;
}

void launch_clear_listed(dq_ctx* ctx, cudaStream_t st)
{
    dim3 grid(16, ctx->cfg.M);
    launch_k(clear_listed_groups_kernel, grid, kThreads, 0, st, ctx->alpha, ctx->cfg.d, ctx->glist, ctx->glist_cap, ctx->gcount);
    ctx->launches += 1;
}

void launch_build_group_list(dq_ctx* ctx, uint32_t* norm_bits, cudaStream_t st)
{
    const dq_config& c = ctx->cfg;
    if (!ctx->ninf_zeroed) cudaMemsetAsync(norm_bits, 0, sizeof(uint32_t) * c.M, st);
    const int nseg = (int)((ctx->bm_words + kThreads - 1) / kThreads);
    dim3 grid(nseg, c.M);
    launch_k(count_touched_kernel, grid, kThreads, 0, st, ctx->touched, ctx->bm_words, ctx->seg_count, nseg);
    const FixedAcc fa = {ctx->acc64, ctx->acc_scale, ctx->acc_inv};
    launch_k(build_group_list_kernel, grid, kThreads, 0, st, ctx->touched, ctx->ptouched, ctx->bm_words, ctx->seg_count, nseg, fa, ctx->alpha, c.d,
                                                        ctx->glist, ctx->glist_cap, ctx->gcount, norm_bits);
    ctx->launches += 2;
}

void launch_sparsify_pack(dq_ctx* ctx, const float* v, int64_t d, int M, int bits, const uint32_t* norm_bits,
                          uint32_t round, const dq_msgs* out, bool sparse_out, cudaStream_t st)
{
    const int vec_ok = vec_ok_for(v, d);
    const bool list = ctx->list_ready && sparse_out && v == ctx->alpha;     // only the listed groups can be nonzero
    const GroupList gl = list ? GroupList{ctx->glist, ctx->gcount, ctx->glist_cap} : GroupList{nullptr, nullptr, 0};
    // a chunk is what one warp compacts on its own: 8 steps of 32 groups when streaming the whole vector, a single
    // step in list mode, where the work is small and parallelism matters more than the size of the offset table
    const int iters = list ? 1 : kChunk / 256;
    const int64_t nchunks = list ? (ctx->glist_cap + 31) / 32 : (d + kChunk - 1) / kChunk;
    if (!(ctx->sp_norms_zeroed && v == ctx->alpha))           // both live in one block behind ninf: one clear covers them
        cudaMemsetAsync(ctx->beta_norm_bits, 0, sizeof(uint32_t) * M + sizeof(unsigned long long) * M, st);
    ctx->sp_norms_zeroed = false;
    if (list) {
        launch_k(norm_l1_list_kernel, dim3(16, M), kThreads, 0, st, v, d, vec_ok, gl, norm_bits, ctx->l1_sum);
    } else {
        dim3 grid_l1(grid_for((d + 7) / 8, ctx->sm_count), M);
        launch_k(norm_l1_kernel, grid_l1, kThreads, 0, st, v, d, vec_ok, norm_bits, ctx->l1_sum);
    }
    dim3 grid_c(list ? 64 : grid_for(nchunks * 32, ctx->sm_count), M);
    const int64_t ngroups = dq_packed_bytes(d, bits) / bits;
    if (list) {
        launch_k(sparsify_count_kernel, grid_c, kThreads, 0, st, v, d, vec_ok, norm_bits, ctx->l1_sum, ctx->cfg.phi, ctx->keys, round,
                                                           ctx->beta_norm_bits, ctx->chunk_off, nchunks, ctx->rp_active, gl, iters);
        launch_k(chunk_scan_kernel, M, kThreads, 0, st, ctx->chunk_off, nchunks, out->cap, out->nnz, ctx->status, out->codes, out->stride);
        DQ_DISPATCH_BITS(bits, (launch_k(sparsify_emit_kernel<BITS_, true>, grid_c, kThreads, 0, st, v, d, vec_ok, norm_bits, ctx->l1_sum, ctx->cfg.phi, ctx->keys, round, ctx->beta_norm_bits, ctx->chunk_off,
            nchunks, 0, out->codes, out->stride, out->scale, out->idx, out->cap, ctx->status, ctx->rp_active, gl, iters, nullptr, 0)));
        ctx->launches += 4;
        return;
    }
    // whole-vector mode: the mask pass stages the survivors; the steps after it touch the vector again only for
    // the chunks (or workers) whose survivors did not fit the staging area
    uint32_t* flags = ctx->stage_ctrl;
    const StageBufs sb{ctx->stage_idx, ctx->stage_val, flags};
    cudaMemsetAsync(flags, 0, sizeof(uint32_t) * ((size_t)M + 1), st);
    launch_k(sparsify_stage_kernel, grid_c, kThreads, 0, st, v, d, vec_ok, norm_bits, ctx->l1_sum, ctx->cfg.phi, ctx->keys, round,
                                                       ctx->beta_norm_bits, ctx->chunk_off, nchunks, ctx->rp_active, sb, M);
    cudaMemsetAsync(out->codes, 0, (size_t)out->stride * M, st);
    ctx->launches += 2;
    dim3 grid_f(grid_for(nchunks * 8, ctx->sm_count), M);
    if (sparse_out) {
        launch_k(chunk_scan_kernel, M, kThreads, 0, st, ctx->chunk_off, nchunks, out->cap, out->nnz, ctx->status, nullptr, 0);
        DQ_DISPATCH_BITS(bits, (launch_k(sparsify_finish_sparse_kernel<BITS_>, grid_f, kThreads, 0, st, norm_bits, ctx->beta_norm_bits, ctx->keys, round, ctx->chunk_off, nchunks, sb, out->codes, out->stride, out->scale,
            out->idx, out->cap, ctx->status, ctx->rp_active)));
        DQ_DISPATCH_BITS(bits, (launch_k(sparsify_emit_kernel<BITS_, true>, grid_c, kThreads, 0, st, v, d, vec_ok, norm_bits, ctx->l1_sum, ctx->cfg.phi, ctx->keys, round, ctx->beta_norm_bits, ctx->chunk_off,
            nchunks, 0, out->codes, out->stride, out->scale, out->idx, out->cap, ctx->status, ctx->rp_active, gl, iters,
            flags, M)));
        ctx->launches += 3;
    } else {
        DQ_DISPATCH_BITS(bits, (launch_k(sparsify_scatter_dense_kernel<BITS_>, grid_f, kThreads, 0, st, norm_bits, ctx->beta_norm_bits, ctx->keys, round, ctx->chunk_off, nchunks, sb, out->codes, out->stride, out->scale,
            ctx->status, ctx->rp_active)));
        DQ_DISPATCH_BITS(bits, (launch_k(sparsify_emit_kernel<BITS_, false>, grid_c, kThreads, 0, st, v, d, vec_ok, norm_bits, ctx->l1_sum, ctx->cfg.phi, ctx->keys, round, ctx->beta_norm_bits, nullptr,
            nchunks, ngroups, out->codes, out->stride, out->scale, nullptr, 0, ctx->status, ctx->rp_active, gl, iters,
            flags, M)));
        ctx->launches += 2;
    }
}

// One cluster kernel from the CSR worker kernel's accumulator to the sparse messages and the master's tile pointers.
void sparse_message_setup(dq_ctx* ctx)
{
    ctx->msg_cluster = false;
    const dq_config& c = ctx->cfg;
    if (!ctx->list_mode || c.no_fused || (c.b != 2 && c.b != 4 && c.b != 8)) return;
    const size_t bm_bytes = sizeof(uint32_t) * (size_t)c.M * ctx->bm_words, list_bytes = sizeof(uint32_t) * (size_t)c.M * ctx->glist_cap;
    if (cudaMalloc(&ctx->ptouched, bm_bytes) != cudaSuccess || cudaMalloc(&ctx->gtmp, list_bytes) != cudaSuccess ||
        cudaMemset(ctx->ptouched, 0, bm_bytes) != cudaSuccess) {
        cudaFree(ctx->ptouched); cudaFree(ctx->gtmp); ctx->ptouched = nullptr; ctx->gtmp = nullptr; cudaGetLastError(); return;
    }
    cudaLaunchConfig_t cfg = cudaLaunchConfig_t{}; cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kMsgCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(kMsgCluster, (unsigned)c.M); cfg.blockDim = dim3(kMsgThreads); cfg.attrs = attr; cfg.numAttrs = 1;
    int nclusters = 0;
    cudaError_t e = cudaErrorInvalidValue;
    DQ_DISPATCH_BITS(c.b, (e = cudaOccupancyMaxActiveClusters(&nclusters, sparse_message_kernel<BITS_>, &cfg)));
    if (e == cudaSuccess && nclusters >= 1) ctx->msg_cluster = true; else cudaGetLastError();
}

bool sparse_message_applies(const dq_ctx* ctx) { return ctx->msg_cluster && ctx->list_mode && ctx->cfg.sparsify && ctx->msgs.idx != nullptr; }

void launch_sparse_message(dq_ctx* ctx, uint32_t round, const dq_msgs* out, cudaStream_t st)
{
    const dq_config& c = ctx->cfg;
    SparseMsg A;
    A.touched = ctx->touched; A.ptouched = ctx->ptouched; A.bm_words = ctx->bm_words; A.fa = FixedAcc{ctx->acc64, ctx->acc_scale, ctx->acc_inv};
    A.alpha = ctx->alpha; A.d = c.d; A.glist = ctx->glist; A.gtmp = ctx->gtmp; A.gcap = ctx->glist_cap; A.gcount = ctx->gcount;
    A.norm_bits = reinterpret_cast<uint32_t*>(ctx->ninf); A.l1_sum = ctx->l1_sum; A.beta_norm_bits = ctx->beta_norm_bits;
    A.phi = c.phi; A.round = round; A.rp = ctx->rp_active;
    A.codes = out->codes; A.stride = out->stride; A.scale = out->scale; A.idx = out->idx; A.cap = out->cap; A.nnz = out->nnz;
    A.tile_ptr = ctx->tile_ptr; A.ntiles = ctx->nchunks; A.status = ctx->status;
    cudaLaunchConfig_t cfg = cudaLaunchConfig_t{}; cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kMsgCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(kMsgCluster, (unsigned)c.M); cfg.blockDim = dim3(kMsgThreads); cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 2;
    DQ_DISPATCH_BITS(c.b, (cudaLaunchKernelEx(&cfg, sparse_message_kernel<BITS_>, A, ctx->keys)));
    ctx->launches += 1;
}

// Quantiser and master step of a round in one kernel (dense messages, averaged master): the context's message buffers
// receive the packed codes and scales as from launch_quantize_pack followed by launch_master.
bool quantize_master_applies(const dq_ctx* ctx)
{
    const dq_config& c = ctx->cfg;
    // the tile's codes of all workers sit in shared memory; very large models gain nothing from sharing a kernel
    return !c.sparsify && !c.sequential && !c.no_fused && c.M <= kQmMaxWorkers && c.d <= ((int64_t)1 << 22);
}

void launch_quantize_master(dq_ctx* ctx, const float* v, const uint32_t* norm_bits, uint32_t round, const dq_msgs* msgs, dq_state* s,
                            float eta, float theta, cudaStream_t st, const BitsArgs* bits)
{
    BitsArgs ba = {nullptr, nullptr, nullptr, 0, 0, 0, 0};
    if (bits) ba = *bits;
    const dq_config& c = ctx->cfg;
    const int64_t d = c.d;
    ProxParams pp{c.lambda1, c.lambda2, c.box_lo, c.box_hi};
    uint32_t* nx = reinterpret_cast<uint32_t*>(s->norm_x);
    if (!ctx->normx_zeroed) cudaMemsetAsync(nx, 0, sizeof(uint32_t), st);
    const int64_t ngroups = dq_packed_bytes(d, c.b) / c.b;
    const int grid = (int)((ngroups * 8 + kQmTile - 1) / kQmTile);
    const size_t smem = sizeof(float) * 2 * c.M + (size_t)c.M * kQmTile;
    if (c.accelerated) {
        DQ_DISPATCH_BITS(c.b, (launch_k(quantize_master_kernel<BITS_, true>, grid, kThreads, smem, st, v, d, c.M, vec_ok_for(v, d), norm_bits,
            msgs->codes, msgs->stride, msgs->scale, ctx->keys, round, ngroups, ctx->status, s->g_full, s->x, s->y, s->x_snap, s->x_sum,
            eta, theta, pp, nx, ctx->rp_active, ba)));
    } else {
        DQ_DISPATCH_BITS(c.b, (launch_k(quantize_master_kernel<BITS_, false>, grid, kThreads, smem, st, v, d, c.M, vec_ok_for(v, d), norm_bits,
            msgs->codes, msgs->stride, msgs->scale, ctx->keys, round, ngroups, ctx->status, s->g_full, s->x, s->y, s->x_snap, s->x_sum,
            eta, theta, pp, nx, ctx->rp_active, ba)));
    }
    ctx->launches += 1;
}

void launch_master(dq_ctx* ctx, const dq_msgs* msgs, bool sparse_msgs, dq_state* s, float eta, float theta, cudaStream_t st,
                   const BitsArgs* bits)
{
    BitsArgs ba = {nullptr, nullptr, nullptr, 0, 0, 0, 0};
    if (bits) ba = *bits;
    const dq_config& c = ctx->cfg;
    const int64_t d = c.d;
    ProxParams pp{c.lambda1, c.lambda2, c.box_lo, c.box_hi};
    uint32_t* nx = reinterpret_cast<uint32_t*>(s->norm_x);
    if (!ctx->normx_zeroed) cudaMemsetAsync(nx, 0, sizeof(uint32_t), st);
    if (c.sequential && !sparse_msgs) {
        const int64_t nw = (d + (32 / c.b) - 1) / (32 / c.b);
        const int grid = grid_for(nw, ctx->sm_count);
        const size_t smem = sizeof(float) * c.M;
        if (c.accelerated) {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_dense_seq_kernel<BITS_, true>, grid, kThreads, smem, st, msgs->codes, msgs->stride, msgs->scale, c.M, d, s->g_full, s->x, s->y, s->x_snap, s->x_sum, eta, theta, pp, nx, ctx->rp_active, ba)));
        } else {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_dense_seq_kernel<BITS_, false>, grid, kThreads, smem, st, msgs->codes, msgs->stride, msgs->scale, c.M, d, s->g_full, s->x, s->y, s->x_snap, s->x_sum, eta, theta, pp, nx, ctx->rp_active, ba)));
        }
        ctx->launches += 1;
        return;
    }
    if (!sparse_msgs) {
        const int64_t cpt = c.b == 2 ? 16 : 8;               // coordinates per thread of master_dense_kernel
        const int64_t nwords = (d + cpt - 1) / cpt;
        const int grid = grid_for(nwords, ctx->sm_count);
        const size_t smem = sizeof(float) * c.M;
        auto al32 = [](const void* p) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & 31) == 0; };
        const int vec8_ok = al32(s->x) && al32(s->g_full) && al32(s->y) && al32(s->x_snap) && al32(s->x_sum);
        const bool small = nwords <= (int64_t)ctx->sm_count * kThreads && c.M > 8;     // less than a block per SM: latency, not bandwidth
        if (small && c.accelerated) {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_dense_kernel<BITS_, true, 32>, grid, kThreads, smem, st, msgs->codes, msgs->stride, msgs->scale, c.M, d, s->g_full, s->x, s->y, s->x_snap, s->x_sum, eta, theta, pp, vec8_ok, nx, ctx->rp_active, ba)));
        } else if (small) {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_dense_kernel<BITS_, false, 32>, grid, kThreads, smem, st, msgs->codes, msgs->stride, msgs->scale, c.M, d, s->g_full, s->x, s->y, s->x_snap, s->x_sum, eta, theta, pp, vec8_ok, nx, ctx->rp_active, ba)));
        } else if (c.accelerated) {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_dense_kernel<BITS_, true>, grid, kThreads, smem, st, msgs->codes, msgs->stride, msgs->scale, c.M, d, s->g_full, s->x, s->y, s->x_snap, s->x_sum, eta, theta, pp, vec8_ok, nx, ctx->rp_active, ba)));
        } else {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_dense_kernel<BITS_, false>, grid, kThreads, smem, st, msgs->codes, msgs->stride, msgs->scale, c.M, d, s->g_full, s->x, s->y, s->x_snap, s->x_sum, eta, theta, pp, vec8_ok, nx, ctx->rp_active, ba)));
        }
        ctx->launches += 1;
    } else {
        const int64_t ntiles = (d + kChunk - 1) / kChunk;
        dim3 grid_t((unsigned)((ntiles + 1 + kThreads - 1) / kThreads), c.M);
        const int tp_launch = ctx->tile_ptr_ready ? 0 : 1;      // the message kernel may have written the tile pointers already
        if (tp_launch) launch_k(tile_ptr_kernel, grid_t, kThreads, 0, st, msgs->idx, msgs->cap, msgs->nnz, ntiles, ctx->tile_ptr);
        if (c.sequential) {
            const int grid = (int)(ntiles < (int64_t)ctx->sm_count * 8 ? ntiles : (int64_t)ctx->sm_count * 8);
            if (c.accelerated) {
                DQ_DISPATCH_BITS(c.b, (launch_k(master_sparse_seq_kernel<BITS_, true>, grid, kThreads, sizeof(uint32_t) * 2 * c.M, st, msgs->codes, msgs->stride, msgs->scale, msgs->idx, msgs->cap, ctx->tile_ptr, ntiles, c.M, d, s->g_full, s->x,
                    s->y, s->x_snap, s->x_sum, eta, theta, pp, nx, ctx->rp_active, ba)));
            } else {
                DQ_DISPATCH_BITS(c.b, (launch_k(master_sparse_seq_kernel<BITS_, false>, grid, kThreads, sizeof(uint32_t) * 2 * c.M, st, msgs->codes, msgs->stride, msgs->scale, msgs->idx, msgs->cap, ctx->tile_ptr, ntiles, c.M, d, s->g_full, s->x,
                    s->y, s->x_snap, s->x_sum, eta, theta, pp, nx, ctx->rp_active, ba)));
            }
            ctx->launches += 1 + tp_launch;
            return;
        }
        const int grid = (int)(ntiles < (int64_t)ctx->sm_count * 8 ? ntiles : (int64_t)ctx->sm_count * 8);
        if (c.accelerated) {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_sparse_kernel<BITS_, true>, grid, kThreads, sizeof(uint32_t) * 2 * c.M, st, msgs->codes, msgs->stride, msgs->scale, msgs->idx, msgs->cap, ctx->tile_ptr, ntiles, c.M, d, s->g_full, s->x,
                s->y, s->x_snap, s->x_sum, eta, theta, pp, nx, ctx->rp_active, ba)));
        } else {
            DQ_DISPATCH_BITS(c.b, (launch_k(master_sparse_kernel<BITS_, false>, grid, kThreads, sizeof(uint32_t) * 2 * c.M, st, msgs->codes, msgs->stride, msgs->scale, msgs->idx, msgs->cap, ctx->tile_ptr, ntiles, c.M, d, s->g_full, s->x,
                s->y, s->x_snap, s->x_sum, eta, theta, pp, nx, ctx->rp_active, ba)));
        }
        ctx->launches += 1 + tp_launch;
    }
}

void launch_unpack(dq_ctx* ctx, const dq_msgs* msgs, bool sparse_msgs, int w, float* out, cudaStream_t st)
{
    const dq_config& c = ctx->cfg;
    const uint8_t* codes = msgs->codes + (int64_t)w * msgs->stride;
    if (!sparse_msgs) {
        DQ_DISPATCH_BITS(c.b, (launch_k(unpack_dense_kernel<BITS_>, grid_for(c.d, ctx->sm_count), kThreads, 0, st, codes, msgs->scale + w, c.d, out)));
    } else {
        cudaMemsetAsync(out, 0, sizeof(float) * c.d, st);
        DQ_DISPATCH_BITS(c.b, (launch_k(unpack_sparse_kernel<BITS_>, grid_for(msgs->cap, ctx->sm_count), kThreads, 0, st, codes, msgs->scale + w, msgs->idx + (int64_t)w * msgs->cap, msgs->nnz + w, c.d, out)));
    }
    ctx->launches += 1;
}

}  // namespace dq

// ---------------------------------------------------------------------------------------------------
// dq_quantize_pack_static: dense quantise + pack for callers that cannot allocate device memory.
// The per-message norm words that the other entry points keep in a context's scratch live here in a
// file-scope device array instead.  Host code must not hand the array's name to a kernel (on the
// host that name is only a handle); the device address is looked up once per device below.
// ---------------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxMessages = DQ_STATIC_MAX_MESSAGES;
constexpr int kStaticMaxDevices = 64;

// [0, kStaticMaxMessages): ||v_w||_inf bit patterns; [kStaticMaxMessages]: non-finite flag of the last call.
static __device__ __align__(256) uint32_t g_static_scratch[kStaticMaxMessages + 64];

struct StaticSlot { uint32_t* ptr; int sm_count; std::atomic<int> ready; };
StaticSlot g_static_slot[kStaticMaxDevices];

// Looks up the device address of the scratch array for the current device (first call on that device).  Two host
// threads may make that first call together: both look the address up and store the same values; `ready` is
// published with release order after the values and read with acquire order before them, so no thread sees the flag
// without the values.
int static_scratch_for_current_device(uint32_t** ptr, int* sm_count)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return DQ_ERR_CUDA;
    StaticSlot& s = g_static_slot[dev];
    if (s.ready.load(std::memory_order_acquire) == 0) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) { cudaGetLastError(); return DQ_ERR_CUDA; }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return DQ_ERR_CUDA;
        s.ptr = static_cast<uint32_t*>(p); s.sm_count = sms;
        s.ready.store(1, std::memory_order_release);
    }
    *ptr = s.ptr; *sm_count = s.sm_count;
    return DQ_OK;
}

}  // namespace

extern "C" int dq_quantize_pack_static(const float* v, int64_t d, int M, int b, uint64_t seed, uint32_t round,
                                       uint8_t* codes, int64_t stride, float* scale, void* stream)
{
    using namespace dq;
    if (!v || !codes || !scale || d < 1 || M < 1) return DQ_ERR_ARG;
    if (b != 2 && b != 4 && b != 8) return DQ_ERR_BITS;
    if (M > kStaticMaxMessages) return DQ_ERR_SHAPE;                       // beyond the fixed scratch
    if (d > ((int64_t)1 << 32)) return DQ_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(codes) & 15) || (stride & 15) || (reinterpret_cast<uintptr_t>(v) & 3) ||
        (reinterpret_cast<uintptr_t>(scale) & 3)) return DQ_ERR_ARG;
    if (stride < dq_packed_bytes(d, b)) return DQ_ERR_SHAPE;
    uint32_t* scratch = nullptr; int sms = 0;
    int rc = static_scratch_for_current_device(&scratch, &sms);
    if (rc != DQ_OK) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // the array keeps the previous call's norms: the maxima must start from zero again
    if (cudaMemsetAsync(scratch, 0, sizeof(uint32_t) * (kStaticMaxMessages + 1), st) != cudaSuccess) return DQ_ERR_CUDA;
    const int vec_ok = vec_ok_for(v, d);
    dim3 grid_n(grid_for((d + 7) / 8, sms), M);
    if (launch_k(norm_inf_kernel, grid_n, kThreads, 0, st, v, d, vec_ok, scratch) != cudaSuccess) return DQ_ERR_CUDA;
    const int64_t ngroups = dq_packed_bytes(d, b) / b;
    dim3 grid_q(grid_for(ngroups, sms), M);
    const PhiloxKeys keys = expand_keys(seed);
    int* flag = reinterpret_cast<int*>(scratch + kStaticMaxMessages);
    cudaError_t err = cudaSuccess;             // this launch's own result, not whatever error an earlier call left behind
    DQ_DISPATCH_BITS(b, (err = launch_k(quantize_pack_kernel<BITS_, false>, grid_q, kThreads, 0, st, v, d, vec_ok, scratch, codes, stride, scale, keys, round, 0u, kStreamGrad, ngroups, flag, nullptr, nullptr, nullptr, nullptr, 0, nullptr, 0, nullptr, 0)));
    return err == cudaSuccess ? DQ_OK : DQ_ERR_CUDA;
}
