// The three steps as separate calls: dat_quantize (Algorithm A1 Step 7), dat_aggregate /
// dat_average (Step 9, Eq. grad_agg) and dat_lalr_step (Step 12, Eq. 3).  Codes, scales and
// g_hat are materialised in device memory between the calls.
#include <cmath>

#include "dat_internal.cuh"

// ------------------------------------------------------------------------------------------
// S1: quantizer norms.  Pass A: one fp64 partial sum of squares per (tile, worker).
// Pass B: per layer, fixed-order sum of the partials, nu_l = max_i sqrt(.), S/nu_l.
// Squares of fp32 values are exact in fp64, so the result does not depend on the tiling
// beyond the last bits of an fp64 sum.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DAT_THREADS)
k_sumsq_partial(GradPtrs gp, const int64_t *__restrict__ off, const int64_t *__restrict__ tile_base,
                int h, int M, double *__restrict__ partials)
{
    __shared__ double scratch[DAT_THREADS / 32];
    const int64_t tile = blockIdx.x;
    const int worker = blockIdx.y;
    const TileRange r = dat_tile_range(off, tile_base, h, tile);
    const float *__restrict__ g = gp.p[worker];
    double acc = 0.0;
    constexpr int ITERS = DAT_TILE / 4 / DAT_THREADS;
    float v[ITERS][4];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {          // every load of the thread is in flight before the first is used
        const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
        if (e0 < r.end) dat_load4(g, e0, r.lo, r.hi, v[it]);
        else v[it][0] = v[it][1] = v[it][2] = v[it][3] = 0.0f;
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
#pragma unroll
        for (int j = 0; j < 4; ++j) acc = fma((double)v[it][j], (double)v[it][j], acc);
    }
    const double s = dat_block_sum(acc, scratch);
    if (threadIdx.x == 0) partials[tile * M + worker] = s;
}

__global__ void __launch_bounds__(DAT_THREADS)
k_scales_finalize(const int64_t *__restrict__ tile_base, int h, int M, float S_f,
                  const double *__restrict__ partials, float *__restrict__ worker_norms,
                  float *__restrict__ scales, float *__restrict__ qmul, uint32_t *status, bool per_worker)
{
    __shared__ float s_norm[DAT_MAX_WORKERS];
    const int l = blockIdx.x;
    const int64_t t0 = tile_base[l], t1 = tile_base[l + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = warp; i < M; i += DAT_THREADS / 32) {
        double acc = 0.0;
        for (int64_t t = t0 + lane; t < t1; t += 32) acc += partials[t * M + i];
        acc = dat_warp_sum(acc);
        if (lane == 0) {
            const float nrm = (float)sqrt(acc);
            s_norm[i] = nrm;
            worker_norms[(int64_t)i * h + l] = nrm;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float nu = s_norm[0];
        bool bad = !isfinite(nu);
        for (int i = 1; i < M; ++i) {
            bad |= !isfinite(s_norm[i]);
            nu = (s_norm[i] > nu) ? s_norm[i] : nu;
        }
        if (per_worker) {
            // every worker keeps its own norm (Eq. rand_q as written): index i*h + l
            for (int i = 0; i < M; ++i) {
                scales[(int64_t)i * h + l] = s_norm[i];
                qmul[(int64_t)i * h + l] = (s_norm[i] == 0.0f) ? 0.0f : S_f / s_norm[i];
            }
        } else {
            scales[l] = nu;
            qmul[l] = (nu == 0.0f) ? 0.0f : S_f / nu;
        }
        if (bad) atomicOr(status, DAT_STATUS_NONFINITE);
    }
}

// qmul from caller-supplied norms.
__global__ void k_qmul_from_scales(int h, float S_f, const float *__restrict__ scales,
                                   float *__restrict__ qmul, uint32_t *status)
{
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= h) return;
    const float nu = scales[l];
    qmul[l] = (nu == 0.0f) ? 0.0f : S_f / nu;
    if (!isfinite(nu)) atomicOr(status, DAT_STATUS_NONFINITE);
}

// ------------------------------------------------------------------------------------------
// S2 + S3: stochastic levels and the packed planes.  Tiles are DAT_TILE consecutive elements of
// the FLAT vector (they may span layers); thread t of iteration k owns the aligned group of four
// elements 4*(k*256+t).., which is exactly one Philox block.  The packed bits of a tile are
// assembled in shared memory and written out with 128-bit stores.
// ------------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(DAT_THREADS)
k_quantize(GradPtrs gp, PhiloxKeys keys, const int64_t *__restrict__ off, int h, int64_t d,
           const float *__restrict__ qmul_all, uint8_t *__restrict__ levels, uint8_t *__restrict__ signs,
           int64_t level_bytes, int64_t sign_bytes, bool rng16, bool per_worker, uint32_t stream_base, int64_t elem_base)
{
    constexpr int GROUPS = DAT_TILE / 4;                     // aligned groups per tile
    constexpr int LEVEL_TILE_BYTES = DAT_TILE * BITS / 8;
    constexpr int SIGN_TILE_BYTES = DAT_TILE / 8;
    __shared__ uint4 s_level[LEVEL_TILE_BYTES / 16];
    __shared__ uint4 s_sign[SIGN_TILE_BYTES / 16];
    __shared__ int s_first;

    const int64_t tile = blockIdx.x;
    const int worker = blockIdx.y;
    const int64_t e_tile = tile * DAT_TILE;
    const float *__restrict__ g = gp.p[worker];
    const float *__restrict__ qmul = qmul_all + (per_worker ? (int64_t)worker * h : 0);
    const float S1_f = (float)(1u << BITS);                  // S + 1

    if (threadIdx.x == 0) s_first = dat_find(off, h, e_tile);
    __syncthreads();
    int l = s_first;
    int64_t l_hi = __ldg(off + l + 1);
    float t = __ldg(qmul + l);

    float gall[GROUPS / DAT_THREADS][4];
#pragma unroll
    for (int it = 0; it < GROUPS / DAT_THREADS; ++it)      // every load of the thread is in flight before the first is used
        dat_load4(g, e_tile + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x), 0, d, gall[it]);
#pragma unroll
    for (int it = 0; it < GROUPS / DAT_THREADS; ++it) {
        const int v = it * DAT_THREADS + threadIdx.x;
        const int64_t e0 = e_tile + 4 * (int64_t)v;
        const float *gv = gall[it];
        float u1[4];
        dat_u1x4((uint64_t)(e0 + elem_base), stream_base + (uint32_t)worker, keys, rng16, u1);     // the worker's random stream
        uint32_t lev[4], neg = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t e = e0 + j;
            while (e >= l_hi && l + 1 < h) {     // advance to the element's layer
                ++l;
                l_hi = __ldg(off + l + 1);
                t = __ldg(qmul + l);
            }
            lev[j] = (e < d) ? dat_level_u1(gv[j], t, S1_f, u1[j]) : 0u;
            neg |= (uint32_t)(gv[j] < 0.0f) << j;
        }
        // pack the group's level bits
        if (BITS == 16) {
            reinterpret_cast<uint2 *>(s_level)[v] = make_uint2(lev[0] | (lev[1] << 16), lev[2] | (lev[3] << 16));
        } else if (BITS == 8) {
            reinterpret_cast<uint32_t *>(s_level)[v] = lev[0] | (lev[1] << 8) | (lev[2] << 16) | (lev[3] << 24);
        } else if (BITS == 4) {
            reinterpret_cast<uint16_t *>(s_level)[v] = (uint16_t)(lev[0] | (lev[1] << 4) | (lev[2] << 8) | (lev[3] << 12));
        } else if (BITS == 2) {
            reinterpret_cast<uint8_t *>(s_level)[v] = (uint8_t)(lev[0] | (lev[1] << 2) | (lev[2] << 4) | (lev[3] << 6));
        } else {   // BITS == 1: two neighbouring groups share a byte
            const uint32_t nib = lev[0] | (lev[1] << 1) | (lev[2] << 2) | (lev[3] << 3);
            const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, nib, 1);
            if ((threadIdx.x & 1) == 0) reinterpret_cast<uint8_t *>(s_level)[v >> 1] = (uint8_t)(nib | (other << 4));
        }
        const uint32_t other_neg = __shfl_xor_sync(0xFFFFFFFFu, neg, 1);
        if ((threadIdx.x & 1) == 0) reinterpret_cast<uint8_t *>(s_sign)[v >> 1] = (uint8_t)(neg | (other_neg << 4));
    }
    __syncthreads();

    // 128-bit stores of the finished tile (planes are padded to 16 bytes, so whole uint4 fit)
    {
        const int64_t base = tile * LEVEL_TILE_BYTES;
        const int64_t left = level_bytes - base;
        const int n16 = (int)((left < LEVEL_TILE_BYTES ? left : LEVEL_TILE_BYTES) / 16);
        uint4 *dst = reinterpret_cast<uint4 *>(levels + (int64_t)worker * level_bytes + base);
        for (int k = threadIdx.x; k < n16; k += DAT_THREADS) dst[k] = s_level[k];
    }
    {
        const int64_t base = tile * SIGN_TILE_BYTES;
        const int64_t left = sign_bytes - base;
        const int n16 = (int)((left < SIGN_TILE_BYTES ? left : SIGN_TILE_BYTES) / 16);
        uint4 *dst = reinterpret_cast<uint4 *>(signs + (int64_t)worker * sign_bytes + base);
        for (int k = threadIdx.x; k < n16; k += DAT_THREADS) dst[k] = s_sign[k];
    }
}

extern "C" int dat_quantize(dat_plan_t *plan, const float *const *grads, uint64_t seed, uint64_t step,
                            uint8_t *levels, uint8_t *signs, float *scales, const float *scales_in,
                            void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (plan->bits == 32) return DAT_ERR_BITS;
    if (!levels || !signs || !scales) return DAT_ERR_ARG;
    if (step >> 32) return DAT_ERR_ARG;
    if (!dat_aligned16(levels) || !dat_aligned16(signs) || !dat_aligned16(scales)) return DAT_ERR_ALIGN;
    if (scales_in && !dat_aligned16(scales_in)) return DAT_ERR_ALIGN;
    GradPtrs gp;
    rc = dat_check_grads(plan, grads, &gp);
    if (rc != DAT_OK) return rc;

    cudaStream_t s = (cudaStream_t)stream;
    const int h = (int)plan->h;
    const float S_f = (float)plan->S;
    const bool per_worker = (plan->scale_mode == DAT_SCALE_PER_WORKER);
    const int n_scales = per_worker ? h * plan->M : h;
    if (scales_in) {
        if (scales_in != scales)
            DAT_CUDA(plan, cudaMemcpyAsync(scales, scales_in, (size_t)n_scales * 4, cudaMemcpyDeviceToDevice, s));
        k_qmul_from_scales<<<(n_scales + 255) / 256, 256, 0, s>>>(n_scales, S_f, scales, plan->d_qmul, plan->d_status);
        DAT_LAUNCHED(plan);
    } else {
        dim3 grid((unsigned)plan->n_tiles, (unsigned)plan->M);
        k_sumsq_partial<<<grid, DAT_THREADS, 0, s>>>(gp, plan->d_offsets, plan->d_tile_base, h, plan->M,
                                                     plan->d_partials);
        DAT_LAUNCHED(plan);
        k_scales_finalize<<<h, DAT_THREADS, 0, s>>>(plan->d_tile_base, h, plan->M, S_f, plan->d_partials,
                                                    plan->d_worker_norms, scales, plan->d_qmul, plan->d_status, per_worker);
        DAT_LAUNCHED(plan);
    }
    const PhiloxKeys keys = dat_make_keys(seed, step);
    const int64_t flat_tiles = (plan->d + DAT_TILE - 1) / DAT_TILE;
    dim3 grid((unsigned)flat_tiles, (unsigned)plan->M);
#define DAT_Q(B)                                                                                           \
    k_quantize<B><<<grid, DAT_THREADS, 0, s>>>(gp, keys, plan->d_offsets, h, plan->d, plan->d_qmul, levels, \
                                               signs, plan->level_bytes, plan->sign_bytes, plan->rng_bits == 16, per_worker, plan->worker_base, plan->elem_base)
    switch (plan->bits) {
    case 1: DAT_Q(1); break;
    case 2: DAT_Q(2); break;
    case 4: DAT_Q(4); break;
    case 8: DAT_Q(8); break;
    default: DAT_Q(16); break;
    }
#undef DAT_Q
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

// S1 by itself: the quantizer norm of every (worker, layer), nu_{i,l} = ||g_l^(i)||_2 (Eq. rand_q).
extern "C" int dat_worker_norms(dat_plan_t *plan, const float *const *grads, float *norms_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!norms_out) return DAT_ERR_ARG;
    if (!dat_aligned16(norms_out)) return DAT_ERR_ALIGN;
    GradPtrs gp;
    rc = dat_check_grads(plan, grads, &gp);
    if (rc != DAT_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    const int h = (int)plan->h;
    dim3 grid((unsigned)plan->n_tiles, (unsigned)plan->M);
    k_sumsq_partial<<<grid, DAT_THREADS, 0, s>>>(gp, plan->d_offsets, plan->d_tile_base, h, plan->M, plan->d_partials);
    DAT_LAUNCHED(plan);
    k_scales_finalize<<<h, DAT_THREADS, 0, s>>>(plan->d_tile_base, h, plan->M, (float)plan->S, plan->d_partials,
                                                plan->d_worker_norms, plan->d_scales, plan->d_qmul, plan->d_status, false);
    DAT_LAUNCHED(plan);
    DAT_CUDA(plan, cudaMemcpyAsync(norms_out, plan->d_worker_norms, (size_t)plan->M * h * 4, cudaMemcpyDeviceToDevice, s));
    return DAT_OK;
}

// ------------------------------------------------------------------------------------------
// S4 + S5: unpack, integer sum over workers, one scaling.  Each thread owns 8 consecutive
// elements (b bytes of levels and one sign byte per worker).
// ------------------------------------------------------------------------------------------
__global__ void k_dq_from_scales(int h, float SM_f, const float *__restrict__ scales, float *__restrict__ dq)
{
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= h) return;
    const float nu = scales[l];
    dq[l] = (nu == 0.0f) ? 0.0f : nu / SM_f;
}

template <int BITS>
__device__ __forceinline__ void dat_unpack8(const uint8_t *__restrict__ plane, int64_t e0, uint32_t lev[8])
{
    const uint8_t *p = plane + e0 * BITS / 8;
    if (BITS == 16) {
        const uint4 q = *reinterpret_cast<const uint4 *>(p);
        lev[0] = q.x & 0xFFFF; lev[1] = q.x >> 16; lev[2] = q.y & 0xFFFF; lev[3] = q.y >> 16;
        lev[4] = q.z & 0xFFFF; lev[5] = q.z >> 16; lev[6] = q.w & 0xFFFF; lev[7] = q.w >> 16;
    } else if (BITS == 8) {
        const uint2 q = *reinterpret_cast<const uint2 *>(p);
#pragma unroll
        for (int j = 0; j < 4; ++j) { lev[j] = (q.x >> (8 * j)) & 0xFF; lev[4 + j] = (q.y >> (8 * j)) & 0xFF; }
    } else {
        uint32_t q;
        if (BITS == 4) q = *reinterpret_cast<const uint32_t *>(p);
        else if (BITS == 2) q = *reinterpret_cast<const uint16_t *>(p);
        else q = *p;
#pragma unroll
        for (int j = 0; j < 8; ++j) lev[j] = (q >> (BITS * j)) & ((1u << BITS) - 1u);
    }
}

// Where the M workers' planes are: one buffer with worker i at i * level_bytes (what dat_quantize writes), or
// one pointer per worker -- this GPU's memory or a peer's mapped into the process, read with plain loads:
// the owner of a layer range pulls the other ranks' planes itself instead of waiting for them to be sent.
struct PlanesFlat {
    const uint8_t *levels, *signs;
    int64_t level_bytes, sign_bytes;
    __device__ __forceinline__ const uint8_t *lv(int i) const { return levels + (int64_t)i * level_bytes; }
    __device__ __forceinline__ const uint8_t *sg(int i) const { return signs + (int64_t)i * sign_bytes; }
};
struct PlanesTable {
    const uint8_t *levels[DAT_MAX_WORKERS], *signs[DAT_MAX_WORKERS];
    __device__ __forceinline__ const uint8_t *lv(int i) const { return levels[i]; }
    __device__ __forceinline__ const uint8_t *sg(int i) const { return signs[i]; }
};

template <int BITS, class SRC>
__global__ void __launch_bounds__(DAT_THREADS)
k_aggregate(const __grid_constant__ SRC src, int M, const int64_t *__restrict__ off, int h, int64_t d,
            const float *__restrict__ dq, int32_t *__restrict__ code_sum, float *__restrict__ g_hat)
{
    __shared__ int s_first;
    const int64_t e_blk = (int64_t)blockIdx.x * (DAT_THREADS * 8);
    if (threadIdx.x == 0) s_first = dat_find(off, h, e_blk);
    __syncthreads();
    const int64_t e0 = e_blk + 8 * (int64_t)threadIdx.x;
    if (e0 >= d) return;
    int sum[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) sum[j] = 0;
#pragma unroll 4
    for (int i = 0; i < M; ++i) {                // four workers' loads in flight at a time
        uint32_t lev[8];
        dat_unpack8<BITS>(src.lv(i), e0, lev);
        const uint32_t sg = src.sg(i)[e0 >> 3];
#pragma unroll
        for (int j = 0; j < 8; ++j) sum[j] += ((sg >> j) & 1u) ? -(int)lev[j] : (int)lev[j];
    }
    int l = s_first;
    int64_t l_hi = __ldg(off + l + 1);
    float f = __ldg(dq + l);
    float out[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int64_t e = e0 + j;
        while (e >= l_hi && l + 1 < h) {
            ++l;
            l_hi = __ldg(off + l + 1);
            f = __ldg(dq + l);
        }
        out[j] = (float)sum[j] * f;
    }
    if (e0 + 8 <= d) {
        reinterpret_cast<float4 *>(g_hat + e0)[0] = make_float4(out[0], out[1], out[2], out[3]);
        reinterpret_cast<float4 *>(g_hat + e0)[1] = make_float4(out[4], out[5], out[6], out[7]);
        if (code_sum) {
            reinterpret_cast<int4 *>(code_sum + e0)[0] = make_int4(sum[0], sum[1], sum[2], sum[3]);
            reinterpret_cast<int4 *>(code_sum + e0)[1] = make_int4(sum[4], sum[5], sum[6], sum[7]);
        }
    } else {
        for (int j = 0; j < 8 && e0 + j < d; ++j) {
            g_hat[e0 + j] = out[j];
            if (code_sum) code_sum[e0 + j] = sum[j];
        }
    }
}

// The same with one norm per worker (Eq. grad_agg as written): no integer sum exists;
// g_hat = (sum_i nu_{i,l} * signed level_i) / (S*M), accumulated in fp32 with one fused
// multiply-add per worker, in ascending worker order.
template <int BITS, class SRC>
__global__ void __launch_bounds__(DAT_THREADS)
k_aggregate_per_worker(const __grid_constant__ SRC src, int M, const int64_t *__restrict__ off, int h, int64_t d,
                       const float *__restrict__ scales, float SM_f, float *__restrict__ g_hat)
{
    __shared__ int s_first;
    const int64_t e_blk = (int64_t)blockIdx.x * (DAT_THREADS * 8);
    if (threadIdx.x == 0) s_first = dat_find(off, h, e_blk);
    __syncthreads();
    const int64_t e0 = e_blk + 8 * (int64_t)threadIdx.x;
    if (e0 >= d) return;
    int lidx[8];
    {
        int l = s_first;
        int64_t l_hi = __ldg(off + l + 1);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            while (e0 + j >= l_hi && l + 1 < h) {
                ++l;
                l_hi = __ldg(off + l + 1);
            }
            lidx[j] = l;
        }
    }
    const bool one_layer = (lidx[0] == lidx[7]);
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
#pragma unroll 1
    for (int i = 0; i < M; ++i) {
        uint32_t lev[8];
        dat_unpack8<BITS>(src.lv(i), e0, lev);
        const uint32_t sg = src.sg(i)[e0 >> 3];
        const float *__restrict__ nu_i = scales + (int64_t)i * h;
        const float nu0 = __ldg(nu_i + lidx[0]);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            // (float)level without the conversion unit: 2^23 + level is exact, the sign bit goes on afterwards
            const float mag = __uint_as_float(0x4B000000u | lev[j]) - 8388608.0f;
            const float code = __uint_as_float(__float_as_uint(mag) | (((sg >> j) & 1u) << 31));
            const float nu = one_layer ? nu0 : __ldg(nu_i + lidx[j]);
            acc[j] = __fmaf_rn(nu, code, acc[j]);
        }
    }
    float out[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) out[j] = acc[j] / SM_f;
    if (e0 + 8 <= d) {
        reinterpret_cast<float4 *>(g_hat + e0)[0] = make_float4(out[0], out[1], out[2], out[3]);
        reinterpret_cast<float4 *>(g_hat + e0)[1] = make_float4(out[4], out[5], out[6], out[7]);
    } else {
        for (int j = 0; j < 8 && e0 + j < d; ++j) g_hat[e0 + j] = out[j];
    }
}

// ------------------------------------------------------------------------------------------
// Algorithm A1 Step 10 (two-sided quantisation): g_hat <- Q(g_hat) at the server.  The same
// kernels as Steps 7 and 9 on ONE vector: norm per layer, levels on the random stream of index M
// (the first one no worker uses), packed message, and the receiver's value nu_l * sign * level / S.
// ------------------------------------------------------------------------------------------
extern "C" int dat_requantize(dat_plan_t *plan, float *g_hat, uint64_t seed, uint64_t step,
                              uint8_t *levels, uint8_t *signs, float *scales, const float *scales_in,
                              void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (plan->bits == 32) return DAT_ERR_BITS;
    if (!g_hat || !levels || !signs || !scales) return DAT_ERR_ARG;
    if (step >> 32) return DAT_ERR_ARG;
    if (!dat_aligned16(g_hat) || !dat_aligned16(levels) || !dat_aligned16(signs) || !dat_aligned16(scales) ||
        (scales_in && !dat_aligned16(scales_in)))
        return DAT_ERR_ALIGN;
    GradPtrs gp;
    for (int i = 0; i < DAT_MAX_WORKERS; ++i) gp.p[i] = nullptr;
    gp.p[0] = g_hat;

    cudaStream_t s = (cudaStream_t)stream;
    const int h = (int)plan->h;
    const float S_f = (float)plan->S;
    if (scales_in) {
        if (scales_in != scales)
            DAT_CUDA(plan, cudaMemcpyAsync(scales, scales_in, (size_t)h * 4, cudaMemcpyDeviceToDevice, s));
        k_qmul_from_scales<<<(h + 255) / 256, 256, 0, s>>>(h, S_f, scales, plan->d_qmul, plan->d_status);
        DAT_LAUNCHED(plan);
    } else {
        dim3 grid((unsigned)plan->n_tiles, 1u);
        k_sumsq_partial<<<grid, DAT_THREADS, 0, s>>>(gp, plan->d_offsets, plan->d_tile_base, h, 1, plan->d_partials);
        DAT_LAUNCHED(plan);
        k_scales_finalize<<<h, DAT_THREADS, 0, s>>>(plan->d_tile_base, h, 1, S_f, plan->d_partials,
                                                    plan->d_worker_norms, scales, plan->d_qmul, plan->d_status, false);
        DAT_LAUNCHED(plan);
    }
    const PhiloxKeys keys = dat_make_keys(seed, step);
    const int64_t flat_tiles = (plan->d + DAT_TILE - 1) / DAT_TILE;
    dim3 qgrid((unsigned)flat_tiles, 1u);
    const unsigned agrid = (unsigned)((plan->d + DAT_THREADS * 8 - 1) / (DAT_THREADS * 8));
    k_dq_from_scales<<<(h + 255) / 256, 256, 0, s>>>(h, S_f, scales, plan->d_dq);      // nu / (S * 1)
    DAT_LAUNCHED(plan);
#define DAT_RQ(B)                                                                                                   \
    do {                                                                                                            \
        k_quantize<B><<<qgrid, DAT_THREADS, 0, s>>>(gp, keys, plan->d_offsets, h, plan->d, plan->d_qmul, levels,    \
                                                    signs, plan->level_bytes, plan->sign_bytes,                     \
                                                    plan->rng_bits == 16, false, plan->worker_base + (uint32_t)plan->M, plan->elem_base); \
        DAT_LAUNCHED(plan);                                                                                         \
        k_aggregate<B, PlanesFlat><<<agrid, DAT_THREADS, 0, s>>>(PlanesFlat{levels, signs, plan->level_bytes, plan->sign_bytes}, 1, \
                                                                 plan->d_offsets, h, plan->d, plan->d_dq, nullptr, g_hat); \
    } while (0)
    switch (plan->bits) {
    case 1: DAT_RQ(1); break;
    case 2: DAT_RQ(2); break;
    case 4: DAT_RQ(4); break;
    case 8: DAT_RQ(8); break;
    default: DAT_RQ(16); break;
    }
#undef DAT_RQ
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

template <class SRC>
static int aggregate_launch(dat_plan_t *plan, const SRC &src, const float *scales, int32_t *code_sum, float *g_hat, void *stream)
{
    cudaStream_t s = (cudaStream_t)stream;
    const int h = (int)plan->h;
    const float SM_f = (float)((uint64_t)plan->S * (uint64_t)plan->M);
    const unsigned grid = (unsigned)((plan->d + DAT_THREADS * 8 - 1) / (DAT_THREADS * 8));
    if (plan->scale_mode == DAT_SCALE_PER_WORKER) {
        if (code_sum) return DAT_ERR_ARG;        // differently scaled codes have no integer sum
#define DAT_APW(B)                                                                                                  \
    k_aggregate_per_worker<B, SRC><<<grid, DAT_THREADS, 0, s>>>(src, plan->M, plan->d_offsets, h, plan->d, scales, SM_f, g_hat)
        switch (plan->bits) {
        case 1: DAT_APW(1); break;
        case 2: DAT_APW(2); break;
        case 4: DAT_APW(4); break;
        case 8: DAT_APW(8); break;
        default: DAT_APW(16); break;
        }
#undef DAT_APW
        DAT_LAUNCHED(plan);
        return DAT_OK;
    }
    k_dq_from_scales<<<(h + 255) / 256, 256, 0, s>>>(h, SM_f, scales, plan->d_dq);
    DAT_LAUNCHED(plan);
#define DAT_A(B)                                                                                         \
    k_aggregate<B, SRC><<<grid, DAT_THREADS, 0, s>>>(src, plan->M, plan->d_offsets, h, plan->d, plan->d_dq, code_sum, g_hat)
    switch (plan->bits) {
    case 1: DAT_A(1); break;
    case 2: DAT_A(2); break;
    case 4: DAT_A(4); break;
    case 8: DAT_A(8); break;
    default: DAT_A(16); break;
    }
#undef DAT_A
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

extern "C" int dat_aggregate(dat_plan_t *plan, const uint8_t *levels, const uint8_t *signs,
                             const float *scales, int32_t *code_sum, float *g_hat, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (plan->bits == 32) return DAT_ERR_BITS;
    if (!levels || !signs || !scales || !g_hat) return DAT_ERR_ARG;
    if (!dat_aligned16(levels) || !dat_aligned16(signs) || !dat_aligned16(scales) || !dat_aligned16(g_hat) ||
        (code_sum && !dat_aligned16(code_sum)))
        return DAT_ERR_ALIGN;
    return aggregate_launch(plan, PlanesFlat{levels, signs, plan->level_bytes, plan->sign_bytes}, scales, code_sum, g_hat, stream);
}

extern "C" int dat_aggregate_gather(dat_plan_t *plan, const uint8_t *const *level_planes, const uint8_t *const *sign_planes,
                                    const float *scales, int32_t *code_sum, float *g_hat, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (plan->bits == 32) return DAT_ERR_BITS;
    if (!level_planes || !sign_planes || !scales || !g_hat) return DAT_ERR_ARG;
    if (!dat_aligned16(scales) || !dat_aligned16(g_hat) || (code_sum && !dat_aligned16(code_sum))) return DAT_ERR_ALIGN;
    PlanesTable t;
    for (int i = 0; i < DAT_MAX_WORKERS; ++i) { t.levels[i] = nullptr; t.signs[i] = nullptr; }
    for (int i = 0; i < plan->M; ++i) {
        if (!level_planes[i] || !sign_planes[i]) return DAT_ERR_ARG;
        if (!dat_aligned16(level_planes[i]) || !dat_aligned16(sign_planes[i])) return DAT_ERR_ALIGN;
        t.levels[i] = level_planes[i];
        t.signs[i] = sign_planes[i];
    }
    return aggregate_launch(plan, t, scales, code_sum, g_hat, stream);
}

// Eq. grad_agg with Q = identity: ordered fp32 sum over workers, then one division by M.
__global__ void __launch_bounds__(DAT_THREADS)
k_average(GradPtrs gp, int M, int64_t d, float *__restrict__ g_hat)
{
    const int64_t e0 = 4 * ((int64_t)blockIdx.x * DAT_THREADS + threadIdx.x);
    if (e0 >= d) return;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int i = 0; i < M; ++i) {
        float v[4];
        dat_load4(gp.p[i], e0, 0, d, v);
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j] += v[j];
    }
    const float Mf = (float)M;
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[j] = acc[j] / Mf;
    dat_store4(g_hat, e0, 0, d, acc);
}

extern "C" int dat_average(dat_plan_t *plan, const float *const *grads, float *g_hat, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!g_hat) return DAT_ERR_ARG;
    if (!dat_aligned16(g_hat)) return DAT_ERR_ALIGN;
    GradPtrs gp;
    rc = dat_check_grads(plan, grads, &gp);
    if (rc != DAT_OK) return rc;
    const unsigned grid = (unsigned)((plan->d + DAT_THREADS * 4 - 1) / (DAT_THREADS * 4));
    k_average<<<grid, DAT_THREADS, 0, (cudaStream_t)stream>>>(gp, plan->M, plan->d, g_hat);
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

// ------------------------------------------------------------------------------------------
// S6-S8: LALR (Eq. 3).  Pass 1 (per-layer tiles): m' and the fp64 partial sums of theta^2 and
// m'^2.  Finalize: per layer, a_l = lr * tau(||theta_l||)/||u_l||.  Pass 2: theta -= a_l * m'.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DAT_THREADS)
k_lalr_pass1(const float *__restrict__ theta, float *__restrict__ mom, const float *__restrict__ g_hat,
             const int64_t *__restrict__ off, const int64_t *__restrict__ tile_base, int h, float mu, float wd,
             double *__restrict__ partials)
{
    __shared__ double scratch[DAT_THREADS / 32];
    const int64_t tile = blockIdx.x;
    const TileRange r = dat_tile_range(off, tile_base, h, tile);
    double ss_theta = 0.0, ss_u = 0.0;
#pragma unroll
    for (int it = 0; it < DAT_TILE / 4 / DAT_THREADS; ++it) {
        const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
        if (e0 < r.end) {
            float th[4], m[4], g[4];
            dat_load4(theta, e0, r.lo, r.hi, th);
            dat_load4(mom, e0, r.lo, r.hi, m);
            dat_load4(g_hat, e0, r.lo, r.hi, g);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                m[j] = __fmaf_rn(mu, m[j], __fmaf_rn(wd, th[j], g[j]));
                ss_theta = fma((double)th[j], (double)th[j], ss_theta);
                ss_u = fma((double)m[j], (double)m[j], ss_u);
            }
            dat_store4(mom, e0, r.lo, r.hi, m);
        }
    }
    const double a = dat_block_sum(ss_theta, scratch);
    const double b = dat_block_sum(ss_u, scratch);
    if (threadIdx.x == 0) { partials[2 * tile] = a; partials[2 * tile + 1] = b; }
}

__global__ void __launch_bounds__(DAT_THREADS)
k_lalr_finalize(const int64_t *__restrict__ tile_base, const double *__restrict__ partials,
                float lr, float c_l, float c_u, float *__restrict__ step_a,
                float *__restrict__ norms_out, uint32_t *status)
{
    __shared__ double scratch[DAT_THREADS / 32];
    const int l = blockIdx.x;
    const int64_t t0 = tile_base[l], t1 = tile_base[l + 1];
    double a = 0.0, b = 0.0;
    for (int64_t t = t0 + threadIdx.x; t < t1; t += DAT_THREADS) { a += partials[2 * t]; b += partials[2 * t + 1]; }
    a = dat_block_sum(a, scratch);
    b = dat_block_sum(b, scratch);
    if (threadIdx.x == 0) {
        const float n_theta = (float)sqrt(a), n_u = (float)sqrt(b);
        const float tau = fminf(fmaxf(n_theta, c_l), c_u);
        const float ratio = (n_u == 0.0f) ? 0.0f : tau / n_u;
        step_a[l] = lr * ratio;
        if (norms_out) { norms_out[2 * l] = n_theta; norms_out[2 * l + 1] = n_u; }
        if (!isfinite(n_theta) || !isfinite(n_u)) atomicOr(status, DAT_STATUS_NONFINITE);
    }
}

__global__ void __launch_bounds__(DAT_THREADS)
k_lalr_pass2(float *__restrict__ theta, const float *__restrict__ mom, const int64_t *__restrict__ off,
             const int64_t *__restrict__ tile_base, int h, const float *__restrict__ step_a)
{
    const int64_t tile = blockIdx.x;
    const TileRange r = dat_tile_range(off, tile_base, h, tile);
    const float na = -__ldg(step_a + r.layer);
#pragma unroll
    for (int it = 0; it < DAT_TILE / 4 / DAT_THREADS; ++it) {
        const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
        if (e0 < r.end) {
            float th[4], m[4];
            dat_load4(theta, e0, r.lo, r.hi, th);
            dat_load4(mom, e0, r.lo, r.hi, m);
#pragma unroll
            for (int j = 0; j < 4; ++j) th[j] = __fmaf_rn(na, m[j], th[j]);
            dat_store4(theta, e0, r.lo, r.hi, th);
        }
    }
}

extern "C" int dat_lalr_step(dat_plan_t *plan, float *theta, float *mom, const float *g_hat,
                             const dat_hparams_t *hp, float *layer_norms_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !g_hat || !hp) return DAT_ERR_ARG;
    if (!dat_aligned16(theta) || !dat_aligned16(mom) || !dat_aligned16(g_hat) ||
        (layer_norms_out && !dat_aligned16(layer_norms_out)))
        return DAT_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    const int h = (int)plan->h;
    k_lalr_pass1<<<(unsigned)plan->n_tiles, DAT_THREADS, 0, s>>>(theta, mom, g_hat, plan->d_offsets,
                                                                 plan->d_tile_base, h, hp->momentum,
                                                                 hp->weight_decay, plan->d_partials);
    DAT_LAUNCHED(plan);
    k_lalr_finalize<<<h, DAT_THREADS, 0, s>>>(plan->d_tile_base, plan->d_partials, hp->lr, hp->c_l, hp->c_u,
                                              plan->d_step_a, layer_norms_out, plan->d_status);
    DAT_LAUNCHED(plan);
    k_lalr_pass2<<<(unsigned)plan->n_tiles, DAT_THREADS, 0, s>>>(theta, mom, plan->d_offsets, plan->d_tile_base,
                                                                 h, plan->d_step_a);
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

// ------------------------------------------------------------------------------------------
// LAMB (Algorithm A2) with the update of Eq. upth = Eq. 3.  Pass 1: the moments m', v' are stored,
// the direction u = m^/(sqrt(v^) + zeta) + wd*theta is formed on the fly for the fp64 partial sums
// of theta^2 and u^2.  Finalize as for LALR.  Pass 2 forms u again from the stored moments (the same
// fp32 operations give the same bits) and moves theta.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DAT_THREADS)
k_lamb_pass1(const float *__restrict__ theta, float *__restrict__ mom, float *__restrict__ var,
             const float *__restrict__ g_hat, const int64_t *__restrict__ off,
             const int64_t *__restrict__ tile_base, int h, LambConst c, double *__restrict__ partials)
{
    __shared__ double scratch[DAT_THREADS / 32];
    const int64_t tile = blockIdx.x;
    const TileRange r = dat_tile_range(off, tile_base, h, tile);
    double ss_theta = 0.0, ss_u = 0.0;
#pragma unroll
    for (int it = 0; it < DAT_TILE / 4 / DAT_THREADS; ++it) {
        const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
        if (e0 < r.end) {
            float th[4], m[4], v[4], g[4];
            dat_load4(theta, e0, r.lo, r.hi, th);
            dat_load4(mom, e0, r.lo, r.hi, m);
            dat_load4(var, e0, r.lo, r.hi, v);
            dat_load4(g_hat, e0, r.lo, r.hi, g);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                m[j] = __fmaf_rn(c.beta1, m[j], __fmul_rn(c.om1, g[j]));
                v[j] = __fmaf_rn(c.beta2, v[j], __fmul_rn(c.om2, __fmul_rn(g[j], g[j])));
                const bool inside = (e0 + j >= r.lo && e0 + j < r.hi);
                const float u = inside ? dat_lamb_direction(c, m[j], v[j], th[j]) : 0.0f;
                ss_theta = fma((double)th[j], (double)th[j], ss_theta);
                ss_u = fma((double)u, (double)u, ss_u);
            }
            dat_store4(mom, e0, r.lo, r.hi, m);
            dat_store4(var, e0, r.lo, r.hi, v);
        }
    }
    const double a = dat_block_sum(ss_theta, scratch);
    const double b = dat_block_sum(ss_u, scratch);
    if (threadIdx.x == 0) { partials[2 * tile] = a; partials[2 * tile + 1] = b; }
}

__global__ void __launch_bounds__(DAT_THREADS)
k_lamb_pass2(float *__restrict__ theta, const float *__restrict__ mom, const float *__restrict__ var,
             const int64_t *__restrict__ off, const int64_t *__restrict__ tile_base, int h, LambConst c,
             const float *__restrict__ step_a)
{
    const int64_t tile = blockIdx.x;
    const TileRange r = dat_tile_range(off, tile_base, h, tile);
    const float na = -__ldg(step_a + r.layer);
#pragma unroll
    for (int it = 0; it < DAT_TILE / 4 / DAT_THREADS; ++it) {
        const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
        if (e0 < r.end) {
            float th[4], m[4], v[4];
            dat_load4(theta, e0, r.lo, r.hi, th);
            dat_load4(mom, e0, r.lo, r.hi, m);
            dat_load4(var, e0, r.lo, r.hi, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool inside = (e0 + j >= r.lo && e0 + j < r.hi);
                const float u = inside ? dat_lamb_direction(c, m[j], v[j], th[j]) : 0.0f;
                th[j] = __fmaf_rn(na, u, th[j]);
            }
            dat_store4(theta, e0, r.lo, r.hi, th);
        }
    }
}

extern "C" int dat_lamb_step(dat_plan_t *plan, float *theta, float *mom, float *var, const float *g_hat,
                             const dat_lamb_hparams_t *hp, int64_t t, float *layer_norms_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !var || !g_hat || !hp || t < 1) return DAT_ERR_ARG;
    if (!(hp->beta1 > 0.0f && hp->beta1 < 1.0f && hp->beta2 > 0.0f && hp->beta2 < 1.0f)) return DAT_ERR_ARG;
    if (!dat_aligned16(theta) || !dat_aligned16(mom) || !dat_aligned16(var) || !dat_aligned16(g_hat) ||
        (layer_norms_out && !dat_aligned16(layer_norms_out)))
        return DAT_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    const int h = (int)plan->h;
    const LambConst c = dat_lamb_const(hp, t);
    k_lamb_pass1<<<(unsigned)plan->n_tiles, DAT_THREADS, 0, s>>>(theta, mom, var, g_hat, plan->d_offsets,
                                                                 plan->d_tile_base, h, c, plan->d_partials);
    DAT_LAUNCHED(plan);
    k_lalr_finalize<<<h, DAT_THREADS, 0, s>>>(plan->d_tile_base, plan->d_partials, hp->lr, hp->c_l, hp->c_u,
                                              plan->d_step_a, layer_norms_out, plan->d_status);
    DAT_LAUNCHED(plan);
    k_lamb_pass2<<<(unsigned)plan->n_tiles, DAT_THREADS, 0, s>>>(theta, mom, var, plan->d_offsets,
                                                                 plan->d_tile_base, h, c, plan->d_step_a);
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

// ------------------------------------------------------------------------------------------
// dat_lalr_step_static: the LALR update for callers that cannot allocate device memory.
// No plan, no cudaMalloc: the layer table, the per-tile partial sums and the per-layer step
// lengths live in one fixed array that is part of the library image on every device.
// ------------------------------------------------------------------------------------------
struct StaticScratch {
    int64_t off[DAT_STATIC_MAX_LAYERS + 1];
    int64_t tile_base[DAT_STATIC_MAX_LAYERS + 1];
    double partials[2 * DAT_STATIC_MAX_TILES];
    float step_a[DAT_STATIC_MAX_LAYERS];
    uint32_t status;
};

static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

// In host code `g_static_scratch` is only a handle; the device address has to be asked for,
// once per device, with that device current.
#define DAT_STATIC_MAX_DEVICES 64
static StaticScratch *g_static_ptr[DAT_STATIC_MAX_DEVICES];

extern "C" int dat_lalr_step_static(int64_t num_layers, const int64_t *layer_offsets, float *theta, float *mom,
                                    const float *g_hat, const dat_hparams_t *hp, float *layer_norms_out,
                                    void *stream)
{
    if (!layer_offsets || !theta || !mom || !g_hat || !hp) return DAT_ERR_ARG;
    if (num_layers < 1) return DAT_ERR_ARG;
    if (num_layers > DAT_STATIC_MAX_LAYERS) return DAT_ERR_TOO_LARGE;
    if (!dat_aligned16(theta) || !dat_aligned16(mom) || !dat_aligned16(g_hat) ||
        (layer_norms_out && !dat_aligned16(layer_norms_out)))
        return DAT_ERR_ALIGN;
    if (layer_offsets[0] != 0) return DAT_ERR_LAYOUT;
    int64_t tile_base[DAT_STATIC_MAX_LAYERS + 1];              // host stack, 32 KB
    int64_t nt = 0;
    for (int64_t l = 0; l < num_layers; ++l) {
        if (layer_offsets[l + 1] <= layer_offsets[l]) return DAT_ERR_LAYOUT;
        tile_base[l] = nt;
        const int64_t a = layer_offsets[l] & ~(int64_t)3;
        nt += (layer_offsets[l + 1] - a + DAT_TILE - 1) / DAT_TILE;
        if (nt > DAT_STATIC_MAX_TILES) return DAT_ERR_TOO_LARGE;
    }
    tile_base[num_layers] = nt;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return DAT_ERR_CUDA; }
    if (dev < 0 || dev >= DAT_STATIC_MAX_DEVICES) return DAT_ERR_UNSUPPORTED;
    if (!g_static_ptr[dev]) {
        StaticScratch *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_static_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return DAT_ERR_CUDA;
        }
        g_static_ptr[dev] = p;
    }
    StaticScratch *sc = g_static_ptr[dev];
    cudaStream_t s = (cudaStream_t)stream;
    // the tables are copied from host memory (one of them from this function's stack) on every call:
    // a captured graph would replay those copies from dead memory
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) { (void)cudaGetLastError(); return DAT_ERR_CUDA; }
    if (cap != cudaStreamCaptureStatusNone) return DAT_ERR_UNSUPPORTED;
    const size_t table = (size_t)(num_layers + 1) * sizeof(int64_t);
    cudaError_t e = cudaMemcpyAsync(sc->off, layer_offsets, table, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sc->tile_base, tile_base, table, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(&sc->status, 0, sizeof(uint32_t), s);   // the one word that must start at zero
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DAT_ERR_CUDA; }
    const int h = (int)num_layers;
    k_lalr_pass1<<<(unsigned)nt, DAT_THREADS, 0, s>>>(theta, mom, g_hat, sc->off, sc->tile_base, h, hp->momentum,
                                                      hp->weight_decay, sc->partials);
    k_lalr_finalize<<<h, DAT_THREADS, 0, s>>>(sc->tile_base, sc->partials, hp->lr, hp->c_l, hp->c_u, sc->step_a,
                                              layer_norms_out, &sc->status);
    k_lalr_pass2<<<(unsigned)nt, DAT_THREADS, 0, s>>>(theta, mom, sc->off, sc->tile_base, h, sc->step_a);
    if (cudaGetLastError() != cudaSuccess) return DAT_ERR_CUDA;
    return DAT_OK;
}

// ------------------------------------------------------------------------------------------
// dat_step_passes: Steps 7, 9 and 12 of Algorithm A1 as three streaming passes without the
// packed message -- norms; levels, signed sum over the workers, g_hat, m' and the layer sums
// in one kernel (codes, sums and g_hat stay in registers); theta update.  The same arithmetic
// as dat_step, element by element; what differs is that the gradients are read from memory
// twice by construction and that the passes are separate launches.
// ------------------------------------------------------------------------------------------
template <bool RNG16>
__global__ void __launch_bounds__(DAT_QU_THREADS, DAT_QU_MINB)
k_quant_update(const __grid_constant__ GradPtrs gp, const __grid_constant__ PhiloxKeys keys, const int64_t *__restrict__ off, const int64_t *__restrict__ tile_base8,
               int h, int M, const float *__restrict__ qmul, const float *__restrict__ dq, const float *__restrict__ theta,
               float *__restrict__ mom, float S_f, float mu, float wd, double *__restrict__ partials,
               int32_t *__restrict__ code_sum)
{
    __shared__ double scratch[DAT_THREADS / 32];
    const int64_t tile = blockIdx.x;
    const int layer = dat_find(tile_base8, h, tile);
    const int64_t lo = __ldg(off + layer), hi = __ldg(off + layer + 1);
    const int64_t begin = (lo & ~(int64_t)7) + (tile - __ldg(tile_base8 + layer)) * DAT_QU_TILE;
    const float t = __ldg(qmul + layer), f = __ldg(dq + layer);
    const float two_b = S_f + 1.0f, inv_two_b = 1.0f / two_b;
    // scaled form of Eq. xi (see dat_step.cu): valid while t 2^-b is a normal number
    const bool plain = (t != 0.0f) && !(t >= 1.17549435e-38f * two_b && t <= 3.402823466e38f);
    const float ts = t * inv_two_b;
    const float c0 = inv_two_b * (1.0f / 65536.0f), c1 = -127.0f * inv_two_b;
    const uint32_t ubits = __float_as_uint(inv_two_b);
    double ss_theta = 0.0, ss_u = 0.0;
#pragma unroll 1
    for (int k = 0; k < DAT_QU_GROUPS; ++k) {
        const int64_t e0 = begin + 8 * (int64_t)(k * DAT_QU_THREADS + threadIdx.x);
        if (e0 >= hi) continue;
        const bool full = (e0 >= lo && e0 + 8 <= hi);
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
        const QuConst qc = {t, ts, two_b, c0, c1, ubits};
        if (full && !plain) qu_rows<RNG16, true, false>(gp, keys, qc, M, e0, lo, hi, acc);       // nearly always
        else if (full) qu_rows<RNG16, true, true>(gp, keys, qc, M, e0, lo, hi, acc);
        else if (!plain) qu_rows<RNG16, false, false>(gp, keys, qc, M, e0, lo, hi, acc);
        else qu_rows<RNG16, false, true>(gp, keys, qc, M, e0, lo, hi, acc);
        // theta and m only now: registers are what limits the number of resident warps here
        float th[8], m[8];
        if (full) {
            const float4 t0 = __ldcg(reinterpret_cast<const float4 *>(theta + e0)), t1 = __ldcg(reinterpret_cast<const float4 *>(theta + e0) + 1);
            const float4 m0 = __ldcs(reinterpret_cast<const float4 *>(mom + e0)), m1 = __ldcs(reinterpret_cast<const float4 *>(mom + e0) + 1);
            th[0] = t0.x; th[1] = t0.y; th[2] = t0.z; th[3] = t0.w; th[4] = t1.x; th[5] = t1.y; th[6] = t1.z; th[7] = t1.w;
            m[0] = m0.x; m[1] = m0.y; m[2] = m0.z; m[3] = m0.w; m[4] = m1.x; m[5] = m1.y; m[6] = m1.z; m[7] = m1.w;
        } else {
            dat_load4(theta, e0, lo, hi, th);
            dat_load4(theta, e0 + 4, lo, hi, th + 4);
            dat_load4(mom, e0, lo, hi, m);
            dat_load4(mom, e0 + 4, lo, hi, m + 4);
        }
        if (code_sum) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (e0 + j >= lo && e0 + j < hi) code_sum[e0 + j] = (int)acc[j];
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            m[j] = __fmaf_rn(mu, m[j], __fmaf_rn(wd, th[j], acc[j] * f));
            ss_theta = fma((double)th[j], (double)th[j], ss_theta);
            ss_u = fma((double)m[j], (double)m[j], ss_u);
        }
        dat_store4(mom, e0, lo, hi, m);
        dat_store4(mom, e0 + 4, lo, hi, m + 4);
    }
    const double a = dat_block_sum(ss_theta, scratch);
    const double b = dat_block_sum(ss_u, scratch);
    if (threadIdx.x == 0) { partials[2 * tile] = a; partials[2 * tile + 1] = b; }
}

extern "C" int dat_step_passes(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                               uint64_t seed, uint64_t step, const dat_hparams_t *hp,
                               int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !hp) return DAT_ERR_ARG;
    if (plan->bits == 32 || plan->scale_mode != DAT_SCALE_SHARED_MAX || plan->elem_base || plan->worker_base) return DAT_ERR_UNSUPPORTED;
    if (step >> 32) return DAT_ERR_ARG;
    if (!dat_aligned16(theta) || !dat_aligned16(mom) || (code_sum_out && !dat_aligned16(code_sum_out)) ||
        (layer_norms_out && !dat_aligned16(layer_norms_out)) || (scales_out && !dat_aligned16(scales_out)))
        return DAT_ERR_ALIGN;
    GradPtrs gp;
    rc = dat_check_grads(plan, grads, &gp);
    if (rc != DAT_OK) return rc;
    const int h = (int)plan->h;
    if (!plan->d_tile_base8) {      // first call: the tiling of the second pass (synchronous)
        std::vector<int64_t> tb((size_t)h + 1);
        int64_t nt = 0;
        for (int l = 0; l < h; ++l) {
            tb[l] = nt;
            nt += (plan->offsets[l + 1] - (plan->offsets[l] & ~(int64_t)7) + DAT_QU_TILE - 1) / DAT_QU_TILE;
        }
        tb[h] = nt;
        cudaError_t e = cudaMalloc((void **)&plan->d_tile_base8, ((size_t)h + 1) * 8);
        if (e == cudaSuccess) e = cudaMalloc((void **)&plan->d_partials8, (size_t)nt * 16);
        if (e == cudaSuccess) e = cudaMemcpy(plan->d_tile_base8, tb.data(), ((size_t)h + 1) * 8, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            if (plan->d_tile_base8) cudaFree(plan->d_tile_base8);
            if (plan->d_partials8) cudaFree(plan->d_partials8);
            plan->d_tile_base8 = nullptr;
            plan->d_partials8 = nullptr;
            plan->last_cuda = (int)e;
            (void)cudaGetLastError();
            return DAT_ERR_NOMEM;
        }
        plan->n_tiles8 = nt;
    }
    cudaStream_t s = (cudaStream_t)stream;
    const float S_f = (float)plan->S;
    const float SM_f = (float)((uint64_t)plan->S * (uint64_t)plan->M);
    dim3 ngrid((unsigned)plan->n_tiles, (unsigned)plan->M);
    k_sumsq_partial<<<ngrid, DAT_THREADS, 0, s>>>(gp, plan->d_offsets, plan->d_tile_base, h, plan->M, plan->d_partials);
    DAT_LAUNCHED(plan);
    k_scales_finalize<<<h, DAT_THREADS, 0, s>>>(plan->d_tile_base, h, plan->M, S_f, plan->d_partials, plan->d_worker_norms,
                                                plan->d_scales, plan->d_qmul, plan->d_status, false);
    DAT_LAUNCHED(plan);
    k_dq_from_scales<<<(h + 255) / 256, 256, 0, s>>>(h, SM_f, plan->d_scales, plan->d_dq);
    DAT_LAUNCHED(plan);
    if (scales_out) DAT_CUDA(plan, cudaMemcpyAsync(scales_out, plan->d_scales, (size_t)h * 4, cudaMemcpyDeviceToDevice, s));
    const PhiloxKeys keys = dat_make_keys(seed, step);
    if (plan->rng_bits == 16)
        k_quant_update<true><<<(unsigned)plan->n_tiles8, DAT_QU_THREADS, 0, s>>>(gp, keys, plan->d_offsets, plan->d_tile_base8, h, plan->M,
                                                                                 plan->d_qmul, plan->d_dq, theta, mom, S_f, hp->momentum,
                                                                                 hp->weight_decay, plan->d_partials8, code_sum_out);
    else
        k_quant_update<false><<<(unsigned)plan->n_tiles8, DAT_QU_THREADS, 0, s>>>(gp, keys, plan->d_offsets, plan->d_tile_base8, h, plan->M,
                                                                                  plan->d_qmul, plan->d_dq, theta, mom, S_f, hp->momentum,
                                                                                  hp->weight_decay, plan->d_partials8, code_sum_out);
    DAT_LAUNCHED(plan);
    k_lalr_finalize<<<h, DAT_THREADS, 0, s>>>(plan->d_tile_base8, plan->d_partials8, hp->lr, hp->c_l, hp->c_u, plan->d_step_a,
                                              layer_norms_out, plan->d_status);
    DAT_LAUNCHED(plan);
    k_lalr_pass2<<<(unsigned)plan->n_tiles, DAT_THREADS, 0, s>>>(theta, mom, plan->d_offsets, plan->d_tile_base, h, plan->d_step_a);
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

// ------------------------------------------------------------------------------------------
// dat_step: one call for Steps 7, 9 and 12 -- the single pipelined launch of dat_pipeline.cu.
// ------------------------------------------------------------------------------------------
extern "C" int dat_step(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                        uint64_t seed, uint64_t step, const dat_hparams_t *hp,
                        int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream)
{
    return dat_step_pipelined(plan, theta, mom, grads, seed, step, hp, code_sum_out, layer_norms_out, scales_out, stream);
}
