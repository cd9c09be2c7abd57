// Internal declarations shared by the translation units of libdat.so (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "dat.h"

// Elements per tile of the per-layer tiling (tiles never cross a layer boundary; they start
// on 4-element boundaries of the flat vector so that float4 accesses stay 16-byte aligned).
#define DAT_TILE 4096
#define DAT_THREADS 256

struct GradPtrs {
    const float *p[DAT_MAX_WORKERS];
};

// The ten round keys of Philox4x32-10 for one (seed, step): the same for every thread.
struct PhiloxKeys {
    uint32_t k0[10];
    uint32_t k1[10];
    uint32_t seed_hi;   // fourth counter word
};

struct PipeSchedule;    // dat_pipeline.cu

// LAMB (Algorithm A2): what the kernels need of the hyper-parameters at iteration t.
struct LambConst {
    float beta1, beta2, om1, om2, bc1, bc2, zeta, wd;
};
LambConst dat_lamb_const(const dat_lamb_hparams_t *hp, int64_t t);   // dat_plan.cu

struct dat_plan {
    int device = 0;
    int64_t h = 0, d = 0;
    int M = 0, bits = 0, scale_mode = 0, rng_bits = 16;
    int64_t elem_base = 0;             // global index of the plan's element 0 and of its worker 0 in the random
    uint32_t worker_base = 0;          // streams (dat_plan_set_origin: a plan that covers a slice of a larger problem)
    uint32_t S = 0;
    std::vector<int64_t> offsets;      // host copy, h+1
    std::vector<int64_t> tile_base;    // host copy, h+1: first per-layer tile of each layer
    int64_t n_tiles = 0;               // per-layer tiles in total
    int64_t level_bytes = 0, sign_bytes = 0;

    // device workspace (one allocation, carved up)
    char *ws = nullptr;
    size_t ws_bytes = 0;
    int64_t *d_offsets = nullptr;      // h+1
    int64_t *d_tile_base = nullptr;    // h+1
    double *d_partials = nullptr;      // n_tiles * max(M,2)
    float *d_worker_norms = nullptr;   // M*h
    float *d_scales = nullptr;         // h     nu_l (fused path / scratch)
    float *d_qmul = nullptr;           // h (shared scale) or M*h (per-worker scales): S/nu (0 if nu = 0)
    float *d_dq = nullptr;             // h     nu_l/(S*M)
    float *d_step_a = nullptr;         // h     lr * tau/||u||
    float *d_norms = nullptr;          // 2h
    uint32_t *d_status = nullptr;      // 1

    PipeSchedule *pipe = nullptr;      // work items and tables of dat_step_pipelined, built with the plan

    // dat_step_passes: per-layer tiles that start on multiples of 8 elements, and their partial sums
    int64_t *d_tile_base8 = nullptr;   // h+1
    double *d_partials8 = nullptr;     // 2 per tile
    int64_t n_tiles8 = 0;

    // staging buffers of dat_step_host
    float *stage = nullptr;

    int sm_count = 0;
    int64_t launches = 0;
    int last_cuda = 0;
};

// ---- host helpers (dat_plan.cu) -------------------------------------------------------------
int dat_check_plan(dat_plan_t *plan);                       // device current, non-null
int dat_cuda_fail(dat_plan_t *plan, cudaError_t e);          // records e, returns DAT_ERR_CUDA
bool dat_aligned16(const void *p);
int dat_check_grads(const dat_plan_t *plan, const float *const *grads, GradPtrs *out);
PhiloxKeys dat_make_keys(uint64_t seed, uint64_t step);
int dat_pipe_build(dat_plan_t *plan);                        // dat_pipeline.cu (device current)
void dat_pipe_destroy(dat_plan_t *plan);
cudaError_t dat_pipe_reset(dat_plan_t *plan, cudaStream_t s);

#define DAT_CUDA(plan, call)                                              \
    do {                                                                  \
        cudaError_t e__ = (call);                                         \
        if (e__ != cudaSuccess) return dat_cuda_fail((plan), e__);        \
    } while (0)

#define DAT_LAUNCHED(plan)                                                \
    do {                                                                  \
        cudaError_t e__ = cudaGetLastError();                             \
        if (e__ != cudaSuccess) return dat_cuda_fail((plan), e__);        \
        (plan)->launches++;                                               \
    } while (0)

// ---- device helpers ---------------------------------------------------------------------------
#ifdef __CUDACC__

// One Philox4x32-10 block (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and
// two three-way XORs; round keys precomputed on the host.
__device__ __forceinline__ void dat_philox(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                           const PhiloxKeys &k, uint32_t out[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The random words of the four elements 4q .. 4q+3 of `worker`.
__device__ __forceinline__ void dat_random_words(uint64_t q, uint32_t worker, const PhiloxKeys &k,
                                                 uint32_t out[4])
{
    dat_philox((uint32_t)q, (uint32_t)(q >> 32), worker, k.seed_hi, k, out);
}

// The quantizer's random number u1 = 1 + u in [1, 2), u uniform on a 2^-23 grid: the low 23 bits
// of a random word become the mantissa.
__device__ __forceinline__ float dat_u1_from_word(uint32_t w)
{
    return __uint_as_float(0x3F800000u | (w & 0x007FFFFFu));
}

// The same on a 2^-16 grid, from a 16-bit half word: 1 + half / 2^16.
__device__ __forceinline__ float dat_u1_from_half(uint32_t half)
{
    return __uint_as_float(0x3F800000u | (half << 7));
}

// u1 of the four elements e0 .. e0+3 (e0 a multiple of 4) of `worker`.  rng16 = false: one
// Philox block per four elements, word j for element e0+j.  rng16 = true: one block per EIGHT
// elements (counter e/8); element e takes word (e/2) mod 4, low half if e is even, high if odd.
__device__ __forceinline__ void dat_u1x4(uint64_t e0, uint32_t worker, const PhiloxKeys &k, bool rng16, float u1[4])
{
    uint32_t w[4];
    if (!rng16) {
        dat_random_words(e0 >> 2, worker, k, w);
#pragma unroll
        for (int j = 0; j < 4; ++j) u1[j] = dat_u1_from_word(w[j]);
    } else {
        dat_random_words(e0 >> 3, worker, k, w);
        const uint32_t wa = (e0 & 4u) ? w[2] : w[0], wb = (e0 & 4u) ? w[3] : w[1];
        u1[0] = dat_u1_from_half(wa & 0xFFFFu);
        u1[1] = dat_u1_from_half(wa >> 16);
        u1[2] = dat_u1_from_half(wb & 0xFFFFu);
        u1[3] = dat_u1_from_half(wb >> 16);
    }
}

// Stochastic level of one element (Eq. xi): level = min(floor(|g|*qmul + u), S) with u uniform
// on [0,1).  With u1 = 1 + u in [1,2), y = fma(|g|, qmul, u1) is clamped to S+1 and
// level = floor(y) - 1.  y lies in [1, 65537): adding 2^23 - 1 with rounding toward -inf leaves
// floor(y) - 1 in the low mantissa bits.  Returns those float bits, 0x4B000000 + level.
__device__ __forceinline__ uint32_t dat_level_bits_u1(float g, float qmul, float S1_f, float u1)
{
    const float y = fminf(__fmaf_rn(fabsf(g), qmul, u1), S1_f);
    return __float_as_uint(__fadd_rd(y, 8388607.0f));
}

__device__ __forceinline__ uint32_t dat_level_u1(float g, float qmul, float S1_f, float u1)
{
    return dat_level_bits_u1(g, qmul, S1_f, u1) & 0x007FFFFFu;
}

// sum += sign(g) * level, from the bits of dat_level_bits: with sm = 0 or -1 (all ones) for
// g's sign bit, (level ^ sm) - sm is level or -level.  (-0.0 has level 0, so its sign is moot.)
__device__ __forceinline__ int dat_add_signed_level(int sum, float g, uint32_t level_bits)
{
    const int sm = (int)__float_as_uint(g) >> 31;
    return sum + (int)((level_bits & 0x007FFFFFu) ^ (uint32_t)sm) - sm;
}

// Largest l in [0, h) with table[l] <= x (table[0] <= x < table[h] assumed).
__device__ __forceinline__ int dat_find(const int64_t *__restrict__ table, int h, int64_t x)
{
    int lo = 0, hi = h;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(table + mid) <= x) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ double dat_warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sum over a block of DAT_THREADS threads in a fixed order; result valid in thread 0.
// `scratch` holds at least DAT_THREADS/32 doubles; safe to call repeatedly.
__device__ __forceinline__ double dat_block_sum(double v, double *scratch)
{
    v = dat_warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < DAT_THREADS / 32; ++w) r += scratch[w];
    }
    return r;
}

// ------------------------------------------------------------------------------------------
// Per-layer tiling shared by the norm kernels: tile t belongs to layer l = find(tile_base, t);
// it covers the flat elements [a + k*DAT_TILE, a + (k+1)*DAT_TILE) ∩ [lo, hi) where
// lo/hi are the layer's bounds, a = lo rounded down to a multiple of 4 and k = t - tile_base[l].
// ------------------------------------------------------------------------------------------
struct TileRange {
    int layer;
    int64_t lo, hi;        // layer bounds
    int64_t begin, end;    // begin is a multiple of 4; elements outside [lo, hi) are masked
};

__device__ __forceinline__ TileRange dat_tile_range(const int64_t *__restrict__ off,
                                                    const int64_t *__restrict__ tile_base, int h,
                                                    int64_t tile)
{
    TileRange r;
    r.layer = dat_find(tile_base, h, tile);
    r.lo = __ldg(off + r.layer);
    r.hi = __ldg(off + r.layer + 1);
    r.begin = (r.lo & ~(int64_t)3) + (tile - __ldg(tile_base + r.layer)) * DAT_TILE;
    r.end = min(r.begin + (int64_t)DAT_TILE, r.hi);
    return r;
}

// Loads the four elements e0..e0+3 (e0 a multiple of 4) that lie in [lo, hi); others read 0.
__device__ __forceinline__ void dat_load4(const float *__restrict__ p, int64_t e0, int64_t lo,
                                          int64_t hi, float v[4])
{
    if (e0 >= lo && e0 + 4 <= hi) {
        const float4 f = *reinterpret_cast<const float4 *>(p + e0);
        v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (e0 + j >= lo && e0 + j < hi) ? p[e0 + j] : 0.0f;
    }
}

__device__ __forceinline__ void dat_store4(float *__restrict__ p, int64_t e0, int64_t lo,
                                           int64_t hi, const float v[4])
{
    if (e0 >= lo && e0 + 4 <= hi) {
        *reinterpret_cast<float4 *>(p + e0) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (e0 + j >= lo && e0 + j < hi) p[e0 + j] = v[j];
    }
}

// The LAMB direction of one element from the stored moments: u = m^/(sqrt(v^) + zeta) + wd*theta with the
// bias-corrected m^ = m'/(1 - beta1^t), v^ = v'/(1 - beta2^t) (Algorithm A2; one rounding per operation).
__device__ __forceinline__ float dat_lamb_direction(const LambConst &c, float m_new, float v_new, float theta)
{
    const float m_hat = m_new / c.bc1;
    const float v_hat = v_new / c.bc2;
    return __fmaf_rn(c.wd, theta, m_hat / (sqrtf(v_hat) + c.zeta));
}

// ------------------------------------------------------------------------------------------
// 16-byte global loads and stores that stay out of L1 and carry an L2 eviction priority.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t dat_policy_evict_last()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t dat_policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t dat_policy_evict_normal()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ float4 dat_ld4_hint(const float *p, uint64_t pol)
{
    float4 v;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.f32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ void dat_st4_hint(float *p, float4 v, uint64_t pol)
{
    asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1,%2,%3,%4}, %5;"
                 :: "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "l"(pol) : "memory");
}

// ------------------------------------------------------------------------------------------
// Levels and signed sum over the workers for one thread's group of eight consecutive elements
// (Eq. xi, Eq. grad_agg), shared by the kernels that keep codes and sums in registers.
// ------------------------------------------------------------------------------------------
#define DAT_QU_THREADS 256
#ifndef DAT_QU_GROUPS
#define DAT_QU_GROUPS 2                          // groups of 8 elements per thread
#endif
#ifndef DAT_QU_UNROLL
#define DAT_QU_UNROLL 2                          // workers whose loads and Philox blocks are in flight together
#endif
#ifndef DAT_QU_MINB
#define DAT_QU_MINB 4                            // resident CTAs per SM asked for (64 registers per thread): this pass lives on many warps
#endif
#define DAT_QU_TILE (DAT_QU_THREADS * 8 * DAT_QU_GROUPS)
#define DAT_QU_PRAGMA(x) _Pragma(#x)
#define DAT_QU_UNROLL_N(n) DAT_QU_PRAGMA(unroll n)

struct QuConst {
    float t, ts, two_b, c0, c1;
    uint32_t ubits;
};

// The M gradient rows of one group of eight elements: levels and signed sum.  FULL: the group lies
// inside the layer (16-byte loads); PLAIN: the layer's scale is outside the range of the scaled
// form.  The common case (FULL, not PLAIN) is inlined, the others are calls.
template <bool RNG16, bool FULL, bool PLAIN>
__device__ __forceinline__ void qu_rows_body(const GradPtrs &gp, const PhiloxKeys &keys, const QuConst &qc, int M, int64_t e0,
                                             int64_t lo, int64_t hi, float acc[8])
{
#ifndef DAT_QU_POLICY
#define DAT_QU_POLICY dat_policy_evict_first
#endif
    const uint64_t pol = DAT_QU_POLICY();             // a gradient is dead once its level is drawn
    DAT_QU_UNROLL_N(DAT_QU_UNROLL)
    for (int i = 0; i < M; ++i) {
        float v[8];
        if (FULL) {
            const float4 a0 = dat_ld4_hint(gp.p[i] + e0, pol), a1 = dat_ld4_hint(gp.p[i] + e0 + 4, pol);
            v[0] = a0.x; v[1] = a0.y; v[2] = a0.z; v[3] = a0.w; v[4] = a1.x; v[5] = a1.y; v[6] = a1.z; v[7] = a1.w;
        } else {
            dat_load4(gp.p[i], e0, lo, hi, v);
            dat_load4(gp.p[i], e0 + 4, lo, hi, v + 4);
        }
        uint32_t w[8];
        if (RNG16) {
            dat_random_words((uint64_t)e0 >> 3, (uint32_t)i, keys, w);
        } else {
            dat_random_words((uint64_t)e0 >> 2, (uint32_t)i, keys, w);
            dat_random_words(((uint64_t)e0 >> 2) + 1, (uint32_t)i, keys, w + 4);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (!PLAIN) {
                float u1s;
                if (RNG16) u1s = __fmaf_rn(__uint_as_float(__byte_perm(w[j >> 1], 0x4B000000u, (j & 1) ? 0x7632 : 0x7610)), qc.c0, qc.c1);
                else u1s = __uint_as_float(qc.ubits | (w[j] & 0x007FFFFFu));
                const float ys = __saturatef(__fmaf_rn(fabsf(v[j]), qc.ts, u1s));
                const float lf = __fmaf_rz(ys, qc.two_b, 8388607.0f) - 8388608.0f;
                const float sg = __uint_as_float((__float_as_uint(v[j]) & 0x80000000u) | 0x3F800000u);
                acc[j] = __fmaf_rn(lf, sg, acc[j]);
            } else {
                const float u1 = RNG16 ? dat_u1_from_half((j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xFFFFu)) : dat_u1_from_word(w[j]);
                const float lf = (float)dat_level_u1(v[j], qc.t, qc.two_b, u1);
                acc[j] += (v[j] < 0.0f) ? -lf : lf;
            }
        }
    }
}
template <bool RNG16, bool FULL, bool PLAIN>
__device__ __noinline__ void qu_rows_call(const GradPtrs &gp, const PhiloxKeys &keys, const QuConst &qc, int M, int64_t e0,
                                          int64_t lo, int64_t hi, float acc[8])
{
    qu_rows_body<RNG16, FULL, PLAIN>(gp, keys, qc, M, e0, lo, hi, acc);
}
template <bool RNG16, bool FULL, bool PLAIN>
__device__ __forceinline__ void qu_rows(const GradPtrs &gp, const PhiloxKeys &keys, const QuConst &qc, int M, int64_t e0,
                                        int64_t lo, int64_t hi, float acc[8])
{
    if (FULL && !PLAIN) qu_rows_body<RNG16, FULL, PLAIN>(gp, keys, qc, M, e0, lo, hi, acc);
    else qu_rows_call<RNG16, FULL, PLAIN>(gp, keys, qc, M, e0, lo, hi, acc);
}

#endif  // __CUDACC__
