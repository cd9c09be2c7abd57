// dat_step: Steps 7, 9 and 12 of Algorithm A1 in ONE persistent kernel.
//
// The flat vector is cut into per-layer tiles (DAT_TILE elements).  Every tile passes through
// three stages, each a work item:
//   N  read the M gradient tiles, fp64 partial sums of squares per worker; the CTA that
//      completes a layer's last N item reduces the partials and publishes nu_l, S/nu_l and
//      nu_l/(S*M)                                                     [||g||_2 of Eq. rand_q]
//   Q  (needs nu_l) re-read the gradient tiles -- by construction still in L2 for layers that
//      fit -- draw the stochastic levels (Eq. xi), sum the signed codes over workers and scale
//      (Eq. grad_agg), form m' = mu*m + g_hat + wd*theta, store m', fp64 partial sums of
//      theta^2 and m'^2; the CTA completing a layer's last Q item publishes
//      a_l = lr * tau(||theta_l||)/||u_l||                              [Eq. 3]
//   U  (needs a_l) theta -= a_l * m'                                     [Eq. 3]
// Items are laid out on the host as a software pipeline: the N items of a window of layers are
// interleaved with the Q items of the previous window and the U items of the one before, so
// that HBM streaming (N) overlaps the L2/ALU-bound work (Q, U) and a layer's dependency is met
// long before its consumers are reached.  CTA c executes items c, c+G, c+2G, ... in order; an
// item depends only on items earlier in the list and all CTAs are co-resident (cooperative
// launch), so the list cannot deadlock.  Every wait is bounded all the same: when it runs out the
// CTA sets DAT_STATUS_TIMEOUT and leaves; the other CTAs see the bit and leave too.
#include <algorithm>
#include <new>

#include "dat_internal.cuh"

enum { ITEM_N = 0u, ITEM_Q = 1u, ITEM_U = 2u };
#define ITEM_TILE_MASK 0x3FFFFFFFu
#define DAT_SPIN_LIMIT (1u << 22)

struct FusedSchedule {
    uint32_t *d_items = nullptr;
    int64_t n_items = 0;
    uint32_t *d_sync = nullptr;     // cnt_n[h] cnt_q[h] flag_n[h] flag_q[h] done[1]
    double *d_qpart = nullptr;      // 2 per tile
    uint32_t epoch = 0;
    int grid = 0;
    int64_t window_bytes = 0;
    int ctas_per_sm = 0;
};

struct FusedArgs {
    GradPtrs gp;
    PhiloxKeys keys;
    float *theta, *mom;
    const int64_t *off, *tile_base;
    const uint32_t *items;
    int64_t n_items;
    double *npart, *qpart;
    uint32_t *cnt_n, *cnt_q, *flag_n, *flag_q, *done, *status;
    float *worker_norms, *scales, *qmul, *dq, *step_a;
    int32_t *code_sum;
    float *norms_out, *scales_out;
    int h, M;
    uint32_t epoch;
    float S_f, SM_f, lr, mu, wd, c_l, c_u;
};

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_release(uint32_t *p, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Thread 0 waits (bounded) until *flag == epoch; returns false for the whole CTA on time-out.
__device__ __forceinline__ bool wait_flag(const uint32_t *flag, uint32_t epoch, uint32_t *status, int *s_ok)
{
    if (threadIdx.x == 0) {
        int ok = 1;
        uint32_t spins = 0;
        while (ld_acquire(flag) != epoch) {
            __nanosleep(40);
            ++spins;
            if (spins > DAT_SPIN_LIMIT || ((spins & 255u) == 0 && (ld_acquire(status) & DAT_STATUS_TIMEOUT))) {
                atomicOr(status, DAT_STATUS_TIMEOUT);
                ok = 0;
                break;
            }
        }
        *s_ok = ok;
    }
    __syncthreads();
    const bool ok = (*s_ok != 0);
    __syncthreads();
    return ok;
}

// After all threads' results for an item are stored: returns true in every thread of the CTA
// that completed the layer's last item (and resets the counter for the next call).
__device__ __forceinline__ bool arrive_is_last(uint32_t *cnt, uint32_t n_tiles_layer, int *s_last)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t old = atomicAdd(cnt, 1u);
        const int last = (old == n_tiles_layer - 1u);
        if (last) { *cnt = 0u; __threadfence(); }
        *s_last = last;
    }
    __syncthreads();
    const bool last = (*s_last != 0);
    __syncthreads();
    return last;
}

// ---- N: partial sums of squares of one tile, all workers ---------------------------------------
__device__ __forceinline__ void item_norm(const FusedArgs &a, const TileRange &r, int64_t tile,
                                          double (*s_red)[DAT_MAX_WORKERS], int *s_flag)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int ITERS = DAT_TILE / 4 / DAT_THREADS;
    for (int i = 0; i < a.M; i += 2) {
        const float *__restrict__ g0 = a.gp.p[i];
        const bool two = (i + 1 < a.M);
        const float *__restrict__ g1 = a.gp.p[two ? i + 1 : i];
        float v0[ITERS][4], v1[ITERS][4];
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
            if (e0 < r.end) {
                dat_load4(g0, e0, r.lo, r.hi, v0[it]);
                dat_load4(g1, e0, r.lo, r.hi, v1[it]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) { v0[it][j] = 0.0f; v1[it][j] = 0.0f; }
            }
        }
        double acc0 = 0.0, acc1 = 0.0;
#pragma unroll
        for (int it = 0; it < ITERS; ++it)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc0 = fma((double)v0[it][j], (double)v0[it][j], acc0);
                acc1 = fma((double)v1[it][j], (double)v1[it][j], acc1);
            }
        acc0 = dat_warp_sum(acc0);
        acc1 = dat_warp_sum(acc1);
        if (lane == 0) {
            s_red[warp][i] = acc0;
            if (two) s_red[warp][i + 1] = acc1;
        }
    }
    __syncthreads();
    if (threadIdx.x < a.M) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < DAT_THREADS / 32; ++w) s += s_red[w][threadIdx.x];
        a.npart[tile * a.M + threadIdx.x] = s;
    }
    const int64_t t0 = __ldg(a.tile_base + r.layer), t1 = __ldg(a.tile_base + r.layer + 1);
    if (!arrive_is_last(a.cnt_n + r.layer, (uint32_t)(t1 - t0), s_flag)) return;

    // this CTA completed the layer: reduce the partials in a fixed order and publish the scale
    float *s_norm = reinterpret_cast<float *>(&s_red[0][0]);
    for (int i = warp; i < a.M; i += DAT_THREADS / 32) {
        double acc = 0.0;
        for (int64_t t = t0 + lane; t < t1; t += 32) acc += __ldcg(a.npart + t * a.M + i);
        acc = dat_warp_sum(acc);
        if (lane == 0) {
            const float nrm = (float)sqrt(acc);
            s_norm[i] = nrm;
            a.worker_norms[(int64_t)i * a.h + r.layer] = nrm;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float nu = s_norm[0];
        bool bad = !isfinite(nu);
        for (int i = 1; i < a.M; ++i) {
            bad |= !isfinite(s_norm[i]);
            nu = (s_norm[i] > nu) ? s_norm[i] : nu;
        }
        a.scales[r.layer] = nu;
        a.qmul[r.layer] = (nu == 0.0f) ? 0.0f : a.S_f / nu;
        a.dq[r.layer] = (nu == 0.0f) ? 0.0f : nu / a.SM_f;
        if (a.scales_out) a.scales_out[r.layer] = nu;
        if (bad) atomicOr(a.status, DAT_STATUS_NONFINITE);
        st_release(a.flag_n + r.layer, a.epoch);
    }
    __syncthreads();
}

// ---- Q: quantize + aggregate + direction of one tile ------------------------------------------
template <bool IDENTITY>
__device__ __forceinline__ bool item_quant(const FusedArgs &a, const TileRange &r, int64_t tile,
                                           double *s_scratch, int *s_flag)
{
    float qmul = 0.0f, dq = 0.0f;
    if (!IDENTITY) {
        if (!wait_flag(a.flag_n + r.layer, a.epoch, a.status, s_flag)) return false;
        qmul = __ldcg(a.qmul + r.layer);
        dq = __ldcg(a.dq + r.layer);
    }
    const float Mf = (float)a.M;
    double ss_theta = 0.0, ss_u = 0.0;
#pragma unroll 1
    for (int it = 0; it < DAT_TILE / 4 / DAT_THREADS; ++it) {
        const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
        if (e0 >= r.end) break;
        float th[4], m[4], ghat[4];
        dat_load4(a.theta, e0, r.lo, r.hi, th);
        dat_load4(a.mom, e0, r.lo, r.hi, m);
        if (IDENTITY) {
            float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            for (int i0 = 0; i0 < a.M; i0 += 4) {
                float gv[4][4];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (i0 + k < a.M) dat_load4(a.gp.p[i0 + k], e0, r.lo, r.hi, gv[k]);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (i0 + k < a.M) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) acc[j] += gv[k][j];
                    }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) ghat[j] = acc[j] / Mf;
        } else {
            int sum[4] = {0, 0, 0, 0};
            for (int i0 = 0; i0 < a.M; i0 += 4) {
                float gv[4][4];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (i0 + k < a.M) dat_load4(a.gp.p[i0 + k], e0, r.lo, r.hi, gv[k]);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (i0 + k < a.M) {
                        uint32_t w[4];
                        dat_random_words((uint64_t)e0 >> 2, (uint32_t)(i0 + k), a.keys, w);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int lev = (int)dat_level(gv[k][j], qmul, a.S_f, w[j]);
                            sum[j] += (gv[k][j] < 0.0f) ? -lev : lev;
                        }
                    }
            }
            if (a.code_sum) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (e0 + j >= r.lo && e0 + j < r.hi) a.code_sum[e0 + j] = sum[j];
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) ghat[j] = (float)sum[j] * dq;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            m[j] = __fmaf_rn(a.mu, m[j], __fmaf_rn(a.wd, th[j], ghat[j]));
            ss_theta = fma((double)th[j], (double)th[j], ss_theta);
            ss_u = fma((double)m[j], (double)m[j], ss_u);
        }
        dat_store4(a.mom, e0, r.lo, r.hi, m);
    }
    const double st = dat_block_sum(ss_theta, s_scratch);
    const double su = dat_block_sum(ss_u, s_scratch);
    if (threadIdx.x == 0) { a.qpart[2 * tile] = st; a.qpart[2 * tile + 1] = su; }
    const int64_t t0 = __ldg(a.tile_base + r.layer), t1 = __ldg(a.tile_base + r.layer + 1);
    if (!arrive_is_last(a.cnt_q + r.layer, (uint32_t)(t1 - t0), s_flag)) return true;

    double x = 0.0, y = 0.0;
    for (int64_t t = t0 + threadIdx.x; t < t1; t += DAT_THREADS) { x += __ldcg(a.qpart + 2 * t); y += __ldcg(a.qpart + 2 * t + 1); }
    x = dat_block_sum(x, s_scratch);
    y = dat_block_sum(y, s_scratch);
    if (threadIdx.x == 0) {
        const float n_theta = (float)sqrt(x), n_u = (float)sqrt(y);
        const float tau = fminf(fmaxf(n_theta, a.c_l), a.c_u);
        const float ratio = (n_u == 0.0f) ? 0.0f : tau / n_u;
        a.step_a[r.layer] = a.lr * ratio;
        if (a.norms_out) { a.norms_out[2 * r.layer] = n_theta; a.norms_out[2 * r.layer + 1] = n_u; }
        if (!isfinite(n_theta) || !isfinite(n_u)) atomicOr(a.status, DAT_STATUS_NONFINITE);
        st_release(a.flag_q + r.layer, a.epoch);
    }
    __syncthreads();
    return true;
}

// ---- U: parameter update of one tile -----------------------------------------------------------
__device__ __forceinline__ bool item_update(const FusedArgs &a, const TileRange &r, int *s_flag)
{
    if (!wait_flag(a.flag_q + r.layer, a.epoch, a.status, s_flag)) return false;
    const float na = -__ldcg(a.step_a + r.layer);
#pragma unroll
    for (int it = 0; it < DAT_TILE / 4 / DAT_THREADS; ++it) {
        const int64_t e0 = r.begin + 4 * (int64_t)(it * DAT_THREADS + threadIdx.x);
        if (e0 < r.end) {
            float th[4], m[4];
            dat_load4(a.theta, e0, r.lo, r.hi, th);
            if (e0 >= r.lo && e0 + 4 <= r.hi) {
                const float4 f = __ldcg(reinterpret_cast<const float4 *>(a.mom + e0));
                m[0] = f.x; m[1] = f.y; m[2] = f.z; m[3] = f.w;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) m[j] = (e0 + j >= r.lo && e0 + j < r.hi) ? __ldcg(a.mom + e0 + j) : 0.0f;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) th[j] = __fmaf_rn(na, m[j], th[j]);
            dat_store4(a.theta, e0, r.lo, r.hi, th);
        }
    }
    return true;
}

template <bool IDENTITY>
__global__ void __launch_bounds__(DAT_THREADS)
k_fused_step(const __grid_constant__ FusedArgs a)
{
    __shared__ double s_red[DAT_THREADS / 32][DAT_MAX_WORKERS];
    __shared__ double s_scratch[DAT_THREADS / 32];
    __shared__ int s_flag;
    bool ok = true;
    for (int64_t it = blockIdx.x; ok && it < a.n_items; it += gridDim.x) {
        const uint32_t item = __ldg(a.items + it);
        const uint32_t type = item >> 30;
        const int64_t tile = item & ITEM_TILE_MASK;
        const TileRange r = dat_tile_range(a.off, a.tile_base, a.h, tile);
        if (type == ITEM_N) item_norm(a, r, tile, s_red, &s_flag);
        else if (type == ITEM_Q) ok = item_quant<IDENTITY>(a, r, tile, s_scratch, &s_flag);
        else ok = item_update(a, r, &s_flag);
    }
    // Last CTA out: after a time-out the dependency counters are in an unknown state; clear
    // them so that the next call starts clean.
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const uint32_t old = atomicAdd(a.done, 1u);
        if (old == gridDim.x - 1u) {
            *a.done = 0u;
            if (ld_acquire(a.status) & DAT_STATUS_TIMEOUT)
                for (int l = 0; l < a.h; ++l) { a.cnt_n[l] = 0u; a.cnt_q[l] = 0u; }
        }
    }
}

// ---- host side -------------------------------------------------------------------------------

void dat_fused_destroy(dat_plan_t *plan)
{
    if (!plan->fused) return;
    if (plan->fused->d_items) cudaFree(plan->fused->d_items);
    if (plan->fused->d_sync) cudaFree(plan->fused->d_sync);
    if (plan->fused->d_qpart) cudaFree(plan->fused->d_qpart);
    delete plan->fused;
    plan->fused = nullptr;
}

// Interleave up to three item sequences so that each advances in proportion to its length.
static void merge_proportional(std::vector<uint32_t> &out, uint32_t typeA, int64_t a0, int64_t a1,
                               uint32_t typeB, int64_t b0, int64_t b1, uint32_t typeC, int64_t c0, int64_t c1)
{
    const int64_t len[3] = {a1 - a0, b1 - b0, c1 - c0};
    const int64_t first[3] = {a0, b0, c0};
    const uint32_t type[3] = {typeA, typeB, typeC};
    int64_t pos[3] = {0, 0, 0};
    const int64_t total = len[0] + len[1] + len[2];
    for (int64_t n = 0; n < total; ++n) {
        int best = -1;
        double best_frac = 2.0;
        for (int k = 0; k < 3; ++k) {
            if (pos[k] >= len[k]) continue;
            const double frac = (double)(pos[k] + 0.5) / (double)len[k];
            if (frac < best_frac) { best_frac = frac; best = k; }
        }
        out.push_back((type[best] << 30) | (uint32_t)(first[best] + pos[best]));
        pos[best]++;
    }
}

static int fused_prepare(dat_plan_t *plan)
{
    if (plan->fused) return DAT_OK;
    FusedSchedule *f = new (std::nothrow) FusedSchedule();
    if (!f) return DAT_ERR_NOMEM;
    plan->fused = f;
    const bool identity = (plan->bits == 32);

    // windows of consecutive layers whose gradient tiles (M*4 bytes per element) stay L2-resident
    int l2 = 0;
    cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, plan->device);
    f->window_bytes = l2 > 0 ? (int64_t)l2 / 4 : (int64_t)16 << 20;
    std::vector<int64_t> win;           // layer index where each window starts, plus h
    int64_t acc = 0;
    win.push_back(0);
    for (int64_t l = 0; l < plan->h; ++l) {
        const int64_t bytes = (plan->offsets[l + 1] - plan->offsets[l]) * 4 * plan->M;
        if (acc > 0 && acc + bytes > f->window_bytes) { win.push_back(l); acc = 0; }
        acc += bytes;
    }
    win.push_back(plan->h);
    const int C = (int)win.size() - 1;
    std::vector<uint32_t> items;
    try {
        items.reserve((size_t)plan->n_tiles * 3);
        auto t_begin = [&](int c) { return (c >= 0 && c < C) ? plan->tile_base[win[c]] : 0; };
        auto t_end = [&](int c) { return (c >= 0 && c < C) ? plan->tile_base[win[c + 1]] : 0; };
        if (identity) {
            for (int s = 0; s < C + 1; ++s)
                merge_proportional(items, ITEM_Q, t_begin(s), t_end(s), ITEM_U, t_begin(s - 1), t_end(s - 1),
                                   ITEM_U, 0, 0);
        } else {
            for (int s = 0; s < C + 2; ++s)
                merge_proportional(items, ITEM_N, t_begin(s), t_end(s), ITEM_Q, t_begin(s - 1), t_end(s - 1),
                                   ITEM_U, t_begin(s - 2), t_end(s - 2));
        }
    } catch (...) { return DAT_ERR_NOMEM; }
    f->n_items = (int64_t)items.size();

    cudaError_t e = cudaMalloc((void **)&f->d_items, items.size() * 4);
    if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_sync, ((size_t)plan->h * 4 + 64) * 4);
    if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_qpart, (size_t)plan->n_tiles * 16);
    if (e != cudaSuccess) { plan->last_cuda = (int)e; (void)cudaGetLastError(); return DAT_ERR_NOMEM; }
    DAT_CUDA(plan, cudaMemcpy(f->d_items, items.data(), items.size() * 4, cudaMemcpyHostToDevice));
    DAT_CUDA(plan, cudaMemset(f->d_sync, 0, ((size_t)plan->h * 4 + 64) * 4));

    int per_sm = 0;
    if (identity)
        DAT_CUDA(plan, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_fused_step<true>, DAT_THREADS, 0));
    else
        DAT_CUDA(plan, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_fused_step<false>, DAT_THREADS, 0));
    if (per_sm < 1) return DAT_ERR_CUDA;
    f->ctas_per_sm = per_sm;
    f->grid = per_sm * plan->sm_count;
    return DAT_OK;
}

extern "C" int dat_step(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                        uint64_t seed, uint64_t step, const dat_hparams_t *hp,
                        int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !hp) return DAT_ERR_ARG;
    if (step >> 32) return DAT_ERR_ARG;
    if (!dat_aligned16(theta) || !dat_aligned16(mom) || (code_sum_out && !dat_aligned16(code_sum_out)) ||
        (layer_norms_out && !dat_aligned16(layer_norms_out)) || (scales_out && !dat_aligned16(scales_out)))
        return DAT_ERR_ALIGN;
    FusedArgs a;
    rc = dat_check_grads(plan, grads, &a.gp);
    if (rc != DAT_OK) return rc;
    rc = fused_prepare(plan);
    if (rc != DAT_OK) return rc;
    FusedSchedule *f = plan->fused;
    const bool identity = (plan->bits == 32);

    f->epoch = (f->epoch == 0xFFFFFFFFu) ? 1u : f->epoch + 1u;
    a.keys = dat_make_keys(seed, step);
    a.theta = theta;
    a.mom = mom;
    a.off = plan->d_offsets;
    a.tile_base = plan->d_tile_base;
    a.items = f->d_items;
    a.n_items = f->n_items;
    a.npart = plan->d_partials;
    a.qpart = f->d_qpart;
    const size_t h = (size_t)plan->h;
    a.cnt_n = f->d_sync;
    a.cnt_q = f->d_sync + h;
    a.flag_n = f->d_sync + 2 * h;
    a.flag_q = f->d_sync + 3 * h;
    a.done = f->d_sync + 4 * h;
    a.status = plan->d_status;
    a.worker_norms = plan->d_worker_norms;
    a.scales = plan->d_scales;
    a.qmul = plan->d_qmul;
    a.dq = plan->d_dq;
    a.step_a = plan->d_step_a;
    a.code_sum = identity ? nullptr : code_sum_out;
    a.norms_out = layer_norms_out;
    a.scales_out = identity ? nullptr : scales_out;
    a.h = (int)plan->h;
    a.M = plan->M;
    a.epoch = f->epoch;
    a.S_f = (float)plan->S;
    a.SM_f = (float)((uint64_t)plan->S * (uint64_t)plan->M);
    a.lr = hp->lr;
    a.mu = hp->momentum;
    a.wd = hp->weight_decay;
    a.c_l = hp->c_l;
    a.c_u = hp->c_u;

    void *params[] = {(void *)&a};
    const int64_t want = (f->n_items < (int64_t)f->grid) ? f->n_items : (int64_t)f->grid;
    const dim3 grid((unsigned)(want < 1 ? 1 : want));
    const void *fn = identity ? (const void *)k_fused_step<true> : (const void *)k_fused_step<false>;
    DAT_CUDA(plan, cudaLaunchCooperativeKernel(fn, grid, dim3(DAT_THREADS), params, 0, (cudaStream_t)stream));
    plan->launches++;
    return DAT_OK;
}
