// dat_step_pipelined: Steps 7, 9 and 12 of Algorithm A1 in ONE launch of ordinary (non-persistent)
// CTAs.  Codes, integer sums and g_hat never reach memory; the gradients are read twice (for the norm, then
// for the levels), the second time from L2 only where a layer is small enough to still be there.
//
// The quantizer norm of a layer (Eq. rand_q) must be known before the first level of that layer
// (Eq. xi) can be drawn, and the two layer norms of Eq. 3 before the first parameter moves: three
// phases per layer, each needing the previous one complete for the whole layer.  The flat vector is
// cut into per-layer tiles, and the host lays three streams of tiles side by side in one list of
// work items: item s holds (at most) one tile for each phase,
//     N  sums of squares of the gradients of a tile          (gradients from HBM, L2 evict-first),
//     Q  levels, signed sum, g_hat, m', layer sums of a tile  (the same gradients once more: from L2 for
//                                                             small layers, from HBM for the others),
//     U  theta update of a tile                               (theta and m' kept in L2 with evict-last),
// where the Q stream runs behind the N stream, and the U stream behind the Q stream, by the size of
// the layer plus a fixed number of items.  A CTA takes the next item by an atomic ticket, so items
// start in list order, and does its N part first: the sums a later item waits for are produced by
// CTAs that started earlier and never wait themselves.  The last CTA to finish a layer's N (or Q)
// tiles reduces the layer's partial sums in a fixed order and publishes the layer's factors with the
// call's epoch; a Q (or U) part whose layer is not published yet polls that word, with a limit.
//
// Two-sided quantisation (Algorithm A1 Step 10) adds a fourth stream between Q and U: the Q part then
// stops at g_hat (stored, with the tile's sum of squares), the layer's last Q tile publishes
// nu^_l = ||g_hat_l||_2, and the R part of a later item draws the server's levels of its tile on the
// random stream of index M, forms the receiver's value and goes on with m' and the layer sums.
#include <algorithm>
#include <new>
#include <vector>

#include "dat_internal.cuh"

#ifndef DAT_P_THREADS
#define DAT_P_THREADS 256
#endif
#ifndef DAT_P_GROUPS                              // groups of eight consecutive elements per thread and tile
#define DAT_P_GROUPS 2
#endif
#define DAT_P_TILE (DAT_P_THREADS * 8 * DAT_P_GROUPS)   // elements per tile, tiles start on multiples of 8
#ifndef DAT_P_MINB
#define DAT_P_MINB (1024 / DAT_P_THREADS)         // 64 registers per thread
#endif
#ifndef DAT_P_LAG                                 // items between the last N tile of a layer and its first Q tile
#define DAT_P_LAG 256
#endif
#ifndef DAT_P_LAG_U                               // items between the last Q tile of a layer and its first U tile
#define DAT_P_LAG_U 512
#endif
#ifndef DAT_P_KEEP_T                              // layers of at most this many tiles: the first reads stay in L2 for the second
#define DAT_P_KEEP_T 72
#endif
#ifndef DAT_P_KEEP_TAIL                           // of a larger layer, the first reads of this many last tiles stay in L2 too
#define DAT_P_KEEP_TAIL 64
#endif
#ifndef DAT_P_REVERSE_FROM                        // layers of at least this many tiles: Q walks back from the last tile
#define DAT_P_REVERSE_FROM (DAT_P_KEEP_T + 1)
#endif
#define DAT_P_WAIT_CYCLES (4000000000ll)          // about two seconds

enum { P_MODE_SHARED = 0, P_MODE_PER_WORKER = 1, P_MODE_IDENTITY = 2 };
enum { P_OPT_MOMENTUM = 0, P_OPT_LAMB = 1 };     // the descent direction u of Eq. 3: heavy-ball momentum, or Algorithm A2

struct PipePart {                                 // one tile of one layer; layer < 0: none
    int64_t lo, hi;                               // the layer's element range
    int32_t tb, T;                                // first tile of the layer in the partial-sum tables, tiles of the layer
    int32_t layer, tile;
};
struct PipeItem {
    PipePart n, q, u, r;                          // r: the server's quantizer (two-sided schedules only)
};

struct PipeSchedule {
    char *mem = nullptr;                          // one device allocation, carved up
    size_t mem_bytes = 0;
    PipeItem *d_items = nullptr;                  // the three streams N, Q, U
    int64_t n_items = 0;
    PipeItem *d_items2 = nullptr;                 // the four streams N, Q, R, U of the two-sided step
    int64_t n_items2 = 0;
    double *d_partR = nullptr;                    // n_tiles
    float *d_server = nullptr;                    // 2h: S / nu^_l and nu^_l / S
    int64_t *d_tile_base = nullptr;               // h + 1
    double *d_partN = nullptr;                    // n_tiles * M
    double *d_partQ = nullptr;                    // n_tiles * 2
    uint32_t *d_sync = nullptr;                   // [0] ticket, [1] abort epoch, then cntN[h], cntQ[h], readyN[h], readyQ[h], cntR[h], readyR[h]
    size_t sync_bytes = 0;
    int64_t n_tiles = 0;
    uint32_t epoch = 0;                           // calls made so far
    long long wait_cycles = DAT_P_WAIT_CYCLES;
};

struct PArgs {
    GradPtrs gp;
    PhiloxKeys keys;
    const PipeItem *items;
    const int64_t *off, *tile_base;
    float *theta, *mom, *var;                     // var: second moment (LAMB only)
    LambConst lamb;
    double *partN, *partQ, *partR;
    uint32_t *ticket, *abort_epoch, *cntN, *cntQ, *readyN, *readyQ, *cntR, *readyR, *status;
    float *worker_norms, *scales, *qmul, *dq, *step_a;
    float *ghat, *qmul2, *dq2;                    // two-sided: g_hat / the receiver's value (d), the server's factors (h each)
    float *norms_out, *scales_out, *server_scales_out;
    int32_t *code_sum;
    long long wait_cycles;
    float S_f, SM_f, M_f, mu, wd, lr, c_l, c_u;
    uint32_t epoch, n_items;
    int M, h;
    int64_t d, n_tiles;
};

// ---- memory access helpers ---------------------------------------------------------------------------
// Bulk data goes past L1 (another CTA of the same launch may have written it) with an L2 eviction hint.
__device__ __forceinline__ uint32_t p_ld_acquire(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void p_st_release(uint32_t *p, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}
// theta / m at a layer's ragged ends: element loads from L2 (never from L1, see above)
__device__ __forceinline__ void p_load4_cg(const float *__restrict__ p, int64_t e0, int64_t lo, int64_t hi, float v[4])
{
    if (e0 >= lo && e0 + 4 <= hi) {
        const float4 f = __ldcg(reinterpret_cast<const float4 *>(p + e0));
        v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (e0 + j >= lo && e0 + j < hi) ? __ldcg(p + e0 + j) : 0.0f;
    }
}

// Eight consecutive elements with an L2 eviction hint: two 16-byte accesses where the group lies inside the
// layer, element accesses (no hint) at a layer's ragged ends.
__device__ __forceinline__ void p_ld8(const float *p, int64_t e0, int64_t lo, int64_t hi, float v[8], uint64_t pol)
{
    if (e0 >= lo && e0 + 8 <= hi) {
        const float4 x = dat_ld4_hint(p + e0, pol), y = dat_ld4_hint(p + e0 + 4, pol);
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w; v[4] = y.x; v[5] = y.y; v[6] = y.z; v[7] = y.w;
    } else {
        p_load4_cg(p, e0, lo, hi, v);
        p_load4_cg(p, e0 + 4, lo, hi, v + 4);
    }
}
__device__ __forceinline__ void p_st8(float *p, int64_t e0, int64_t lo, int64_t hi, const float v[8], uint64_t pol)
{
    if (e0 >= lo && e0 + 8 <= hi) {
        dat_st4_hint(p + e0, make_float4(v[0], v[1], v[2], v[3]), pol);
        dat_st4_hint(p + e0 + 4, make_float4(v[4], v[5], v[6], v[7]), pol);
    } else {
        dat_store4(p, e0, lo, hi, v);
        dat_store4(p, e0 + 4, lo, hi, v + 4);
    }
}

// One thread: waits until `word` carries this call's epoch.  Bounded: when the limit runs out the status
// word gets DAT_STATUS_TIMEOUT and the call's abort word is set, which ends every other wait at once.
// Returns false if the part that needs the word must be skipped.
__device__ __forceinline__ bool p_poll(const PArgs &a, const uint32_t *word)
{
    if (p_ld_acquire(word) == a.epoch) return true;
    const long long t0 = clock64();
    for (;;) {
        __nanosleep(128);
        if (p_ld_acquire(word) == a.epoch) return true;
        if (p_ld_acquire(a.abort_epoch) == a.epoch) return false;
        if (clock64() - t0 > a.wait_cycles) {
            atomicOr(a.status, DAT_STATUS_TIMEOUT);
            p_st_release(a.abort_epoch, a.epoch);
            return false;
        }
    }
}

// Self-checking build (-DDAT_SELFCHECK): what an item says about its tiles is checked before it is used;
// a violation sets DAT_STATUS_BOUNDS and the item is skipped, nothing faults.
#ifdef DAT_SELFCHECK
#define P_CHECK(a, cond) ((cond) ? true : (atomicOr((a).status, DAT_STATUS_BOUNDS), false))
#else
#define P_CHECK(a, cond) true
#endif

__device__ __forceinline__ int64_t p_tile_begin(const PipePart &pt)
{
    return (pt.lo & ~(int64_t)7) + (int64_t)pt.tile * DAT_P_TILE;
}
__device__ __forceinline__ bool p_tile_inside(const PipePart &pt)
{
    const int64_t begin = p_tile_begin(pt);
    return begin >= pt.lo && begin + DAT_P_TILE <= pt.hi;
}

// ---- N: sums of squares of one tile, every worker ------------------------------------------------
// A tile is cut into 4M units (worker, quarter tile); warp w of W takes the units [w*4M/W, (w+1)*4M/W),
// lane j the 16-byte pieces j, j+32, ... of a unit, eight pieces in flight.  Units of the same worker
// are summed per lane before the warp reduction; the structure depends on M only, so the sums are the
// same from run to run.  Leaves one sum per run of units in s_unit (zero elsewhere).
__device__ __forceinline__ void p_norm_sums(const PArgs &a, const PipePart &pt, double *s_unit)
{
    constexpr int W = DAT_P_THREADS / 32, QUARTER = DAT_P_TILE / 4, LPU = QUARTER / 128, UPB = 8 / LPU;   // units per batch of 8 loads
    static_assert(LPU >= 1 && LPU <= 8 && UPB * LPU == 8, "quarter tiles of 128 .. 1024 elements");
    const int M = a.M;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int U = 4 * M;
    const int u0 = warp * U / W, u1 = (warp + 1) * U / W;
    const int64_t begin = p_tile_begin(pt);
    double acc = 0.0;
    int run = u0;
    if (p_tile_inside(pt)) {
#ifndef DAT_P_N_POLICY
#define DAT_P_N_POLICY dat_policy_evict_first
#endif
        // A small layer's lines are still in L2 when the Q part of a later item reads them again, and so are those of
        // a larger layer's last tiles, which the Q stream (walking back from the last tile) reads first; the rest of a
        // large layer is gone by then anyway: better it leaves first than push out those lines, theta and m'.
        const uint64_t pol = (pt.T <= DAT_P_KEEP_T || pt.tile >= pt.T - DAT_P_KEEP_TAIL) ? dat_policy_evict_normal() : DAT_P_N_POLICY();
#pragma unroll 1
        for (int ub = u0; ub < u1; ub += UPB) {
            float4 v[8];
#pragma unroll
            for (int k = 0; k < UPB; ++k) {
                const int u = ub + k;
                if (u < u1) {
                    const float *g = a.gp.p[u >> 2] + begin + (u & 3) * QUARTER + 4 * lane;
#pragma unroll
                    for (int b = 0; b < LPU; ++b) v[k * LPU + b] = dat_ld4_hint(g + 128 * b, pol);
                }
            }
#pragma unroll
            for (int k = 0; k < UPB; ++k) {
                const int u = ub + k;
                if (u < u1) {
                    if ((u >> 2) != (run >> 2)) {
                        acc = dat_warp_sum(acc);
                        if (lane == 0) s_unit[run] = acc;
                        acc = 0.0;
                        run = u;
                    }
#pragma unroll
                    for (int b = 0; b < LPU; ++b) {
                        const float4 x = v[k * LPU + b];
                        acc = fma((double)x.x, (double)x.x, acc);
                        acc = fma((double)x.y, (double)x.y, acc);
                        acc = fma((double)x.z, (double)x.z, acc);
                        acc = fma((double)x.w, (double)x.w, acc);
                    }
                }
            }
        }
    } else {
#pragma unroll 1
        for (int u = u0; u < u1; ++u) {
            if ((u >> 2) != (run >> 2)) {
                acc = dat_warp_sum(acc);
                if (lane == 0) s_unit[run] = acc;
                acc = 0.0;
                run = u;
            }
            const float *__restrict__ g = a.gp.p[u >> 2];
            const int64_t e = begin + (u & 3) * QUARTER + 4 * lane;
#pragma unroll
            for (int b = 0; b < LPU; ++b) {
                float t[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                if (e + 128 * b < pt.hi) dat_load4(g, e + 128 * b, pt.lo, pt.hi, t);
#pragma unroll
                for (int k = 0; k < 4; ++k) acc = fma((double)t[k], (double)t[k], acc);
            }
        }
    }
    if (u1 > u0) {
        acc = dat_warp_sum(acc);
        if (lane == 0) s_unit[run] = acc;
    }
}

// Warp 0, after the barrier that follows the N sums: writes the tile's M partial sums and counts the tile
// in.  Returns (in lane 0) whether this was the layer's last tile.
__device__ __forceinline__ bool p_norm_publish(const PArgs &a, const PipePart &pt, const double *s_unit)
{
    const int M = a.M, lane = threadIdx.x & 31;
    for (int i = lane; i < M; i += 32) {
        const double *s = s_unit + 4 * i;
        a.partN[((int64_t)pt.tb + pt.tile) * M + i] = ((s[0] + s[1]) + s[2]) + s[3];
    }
    __threadfence();
    __syncwarp();
    bool last = false;
    if (lane == 0) {
        __threadfence();
        last = (atomicAdd(a.cntN + pt.layer, 1u) == (uint32_t)pt.T - 1u);
    }
    return last;
}

// The CTA that counted in the layer's last N tile (every thread): nu_{i,l} = sqrt(sum over the tiles),
// nu_l = max_i, and the layer's two factors, published with the call's epoch.
template <int MODE>
__device__ __forceinline__ void p_norm_finish(const PArgs &a, const PipePart &pt, float *s_norm)
{
    const int M = a.M, layer = pt.layer;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t tb = pt.tb;
    const uint32_t T = (uint32_t)pt.T;
    __threadfence();
    for (int i = warp; i < M; i += DAT_P_THREADS / 32) {
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
        uint32_t t = lane;
        for (; t + 96 < T; t += 128) {            // four loads in flight per lane
            const double x0 = __ldcg(a.partN + (tb + t) * M + i), x1 = __ldcg(a.partN + (tb + t + 32) * M + i);
            const double x2 = __ldcg(a.partN + (tb + t + 64) * M + i), x3 = __ldcg(a.partN + (tb + t + 96) * M + i);
            s0 += x0; s1 += x1; s2 += x2; s3 += x3;
        }
        for (; t < T; t += 32) s0 += __ldcg(a.partN + (tb + t) * M + i);
        const double s = dat_warp_sum((s0 + s1) + (s2 + s3));
        if (lane == 0) {
            const float nrm = (float)sqrt(s);
            s_norm[i] = nrm;
            a.worker_norms[(int64_t)i * a.h + layer] = nrm;
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
        if (MODE == P_MODE_PER_WORKER) {
            // every worker keeps its own norm (Eq. rand_q as written): index i*h + l; nu_{i,l} itself is in worker_norms
            for (int i = 0; i < M; ++i) {
                a.qmul[(int64_t)i * a.h + layer] = (s_norm[i] == 0.0f) ? 0.0f : a.S_f / s_norm[i];
                if (a.scales_out) a.scales_out[(int64_t)i * a.h + layer] = s_norm[i];
            }
        } else {
            a.scales[layer] = nu;
            a.qmul[layer] = (nu == 0.0f) ? 0.0f : a.S_f / nu;
            a.dq[layer] = (nu == 0.0f) ? 0.0f : nu / a.SM_f;
            if (a.scales_out) a.scales_out[layer] = nu;
        }
        if (bad) atomicOr(a.status, DAT_STATUS_NONFINITE);
        a.cntN[layer] = 0u;
        __threadfence();
        p_st_release(a.readyN + layer, a.epoch);
    }
}

// ---- the layer's step length from the partial sums of theta^2 and m'^2 (Eq. 3), by the CTA that counted
// in the layer's last Q tile (every thread) ----------------------------------------------------------
__device__ __forceinline__ void p_quant_finish(const PArgs &a, const PipePart &pt, double *scratch)
{
    const int layer = pt.layer;
    const int64_t tb = pt.tb;
    const uint32_t T = (uint32_t)pt.T;
    __threadfence();
    double x = 0.0, y = 0.0;
    for (uint32_t t = threadIdx.x; t < T; t += DAT_P_THREADS) {
        x += __ldcg(a.partQ + 2 * (tb + t));
        y += __ldcg(a.partQ + 2 * (tb + t) + 1);
    }
    x = dat_warp_sum(x);
    y = dat_warp_sum(y);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { scratch[2 * (threadIdx.x >> 5)] = x; scratch[2 * (threadIdx.x >> 5) + 1] = y; }
    __syncthreads();
    if (threadIdx.x == 0) {
        x = 0.0; y = 0.0;
#pragma unroll
        for (int w = 0; w < DAT_P_THREADS / 32; ++w) { x += scratch[2 * w]; y += scratch[2 * w + 1]; }
        const float n_theta = (float)sqrt(x), n_u = (float)sqrt(y);
        const float tau = fminf(fmaxf(n_theta, a.c_l), a.c_u);
        const float ratio = (n_u == 0.0f) ? 0.0f : tau / n_u;
        a.step_a[layer] = a.lr * ratio;
        if (a.norms_out) { a.norms_out[2 * layer] = n_theta; a.norms_out[2 * layer + 1] = n_u; }
        if (!isfinite(n_theta) || !isfinite(n_u)) atomicOr(a.status, DAT_STATUS_NONFINITE);
        a.cntQ[layer] = 0u;
        __threadfence();
        p_st_release(a.readyQ + layer, a.epoch);
    }
}

// Eq. grad_agg as written, every worker on its own grid: acc = sum_i nu_{i,l} * (signed level_i), in fp32
// with one fused multiply-add per worker, ascending; the caller divides by S*M.  Levels by the plain form
// of Eq. xi with the worker's own S/nu_{i,l}.
template <bool RNG16>
__device__ __forceinline__ void p_rows_per_worker(const PArgs &a, int layer, int64_t e0, int64_t lo, int64_t hi, float acc[8])
{
    const bool full = (e0 >= lo && e0 + 8 <= hi);
    const uint64_t pol = dat_policy_evict_first();
    const float two_b = a.S_f + 1.0f;
#pragma unroll 1
    for (int i = 0; i < a.M; ++i) {
        float v[8];
        if (full) {
            const float4 a0 = dat_ld4_hint(a.gp.p[i] + e0, pol), a1 = dat_ld4_hint(a.gp.p[i] + e0 + 4, pol);
            v[0] = a0.x; v[1] = a0.y; v[2] = a0.z; v[3] = a0.w; v[4] = a1.x; v[5] = a1.y; v[6] = a1.z; v[7] = a1.w;
        } else {
            dat_load4(a.gp.p[i], e0, lo, hi, v);
            dat_load4(a.gp.p[i], e0 + 4, lo, hi, v + 4);
        }
        const float t = __ldcg(a.qmul + (int64_t)i * a.h + layer), nu = __ldcg(a.worker_norms + (int64_t)i * a.h + layer);
        uint32_t w[8];
        if (RNG16) {
            dat_random_words((uint64_t)e0 >> 3, (uint32_t)i, a.keys, w);
        } else {
            dat_random_words((uint64_t)e0 >> 2, (uint32_t)i, a.keys, w);
            dat_random_words(((uint64_t)e0 >> 2) + 1, (uint32_t)i, a.keys, w + 4);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float u1 = RNG16 ? dat_u1_from_half((j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xFFFFu)) : dat_u1_from_word(w[j]);
            const float lf = (float)dat_level_u1(v[j], t, two_b, u1);
            acc[j] = __fmaf_rn(nu, (v[j] < 0.0f) ? -lf : lf, acc[j]);
        }
    }
}

// ---- m' (or m', v') and the layer sums of Eq. 3, pass 1, for one thread's group of eight elements whose
// g_hat is in registers: theta and m are loaded only now (registers limit the resident warps here).
template <int OPT>
__device__ __forceinline__ void p_direction(const PArgs &a, int64_t e0, int64_t lo, int64_t hi, const float ghat[8],
                                            double &ss_theta, double &ss_u)
{
    // what the U part reads again (theta, m', v') is kept in L2 (evict-last); the old m is dead (evict-first)
    const uint64_t keep = dat_policy_evict_last();
    float th[8], m[8];
    p_ld8(a.theta, e0, lo, hi, th, keep);
    p_ld8(a.mom, e0, lo, hi, m, dat_policy_evict_first());
    if (OPT == P_OPT_LAMB) {
        // Algorithm A2: both moments are stored, the direction is formed on the fly for the layer sums
        float v[8];
        p_ld8(a.var, e0, lo, hi, v, keep);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            m[j] = __fmaf_rn(a.lamb.beta1, m[j], __fmul_rn(a.lamb.om1, ghat[j]));
            v[j] = __fmaf_rn(a.lamb.beta2, v[j], __fmul_rn(a.lamb.om2, __fmul_rn(ghat[j], ghat[j])));
            const bool inside = (e0 + j >= lo && e0 + j < hi);
            const float u = inside ? dat_lamb_direction(a.lamb, m[j], v[j], th[j]) : 0.0f;
            ss_theta = fma((double)th[j], (double)th[j], ss_theta);
            ss_u = fma((double)u, (double)u, ss_u);
        }
        p_st8(a.var, e0, lo, hi, v, keep);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            m[j] = __fmaf_rn(a.mu, m[j], __fmaf_rn(a.wd, th[j], ghat[j]));
            ss_theta = fma((double)th[j], (double)th[j], ss_theta);
            ss_u = fma((double)m[j], (double)m[j], ss_u);
        }
    }
    p_st8(a.mom, e0, lo, hi, m, keep);
}

// ---- Q: levels (Eq. xi), signed sum over the workers and g_hat (Eq. grad_agg), m' and the layer sums
// (Eq. 3, pass 1) of one tile; codes, sums and g_hat stay in registers.  Leaves the tile's two sums per
// warp in scratch[2w], scratch[2w + 1].  TWO (Algorithm A1 Step 10 follows): stops at g_hat, which is
// stored, and leaves the tile's sum of g_hat^2 per warp in scratch[2w]. ----------------------------
template <bool RNG16, int MODE, int OPT, bool TWO>
__device__ __forceinline__ void p_part_quant(const PArgs &a, const PipePart &pt, double *scratch)
{
    const int M = a.M, layer = pt.layer;
    const int64_t lo = pt.lo, hi = pt.hi;
    float t = 0.0f, f = 0.0f;
    if (MODE == P_MODE_SHARED) { t = __ldcg(a.qmul + layer); f = __ldcg(a.dq + layer); }
    const float two_b = a.S_f + 1.0f, inv_two_b = 1.0f / two_b;
    // scaled form of Eq. xi: valid while t 2^-b is a normal number
    const bool plain = (t != 0.0f) && !(t >= 1.17549435e-38f * two_b && t <= 3.402823466e38f);
    const QuConst qc = {t, t * inv_two_b, two_b, inv_two_b * (1.0f / 65536.0f), -127.0f * inv_two_b, __float_as_uint(inv_two_b)};
    double ss_theta = 0.0, ss_u = 0.0;
    const int64_t begin = p_tile_begin(pt);
#pragma unroll 1
    for (int k = 0; k < DAT_P_GROUPS; ++k) {
        const int64_t e0 = begin + 8 * (int64_t)(k * DAT_P_THREADS + threadIdx.x);
        if (e0 >= hi) continue;
        const bool full = (e0 >= lo && e0 + 8 <= hi);
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
        if (MODE == P_MODE_IDENTITY) {
#pragma unroll 2
            for (int i = 0; i < M; ++i) {           // Q is the identity: the ordered fp32 sum of the workers' gradients
                float v[8];
                dat_load4(a.gp.p[i], e0, lo, hi, v);
                dat_load4(a.gp.p[i], e0 + 4, lo, hi, v + 4);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] += v[j];
            }
        } else if (MODE == P_MODE_PER_WORKER) p_rows_per_worker<RNG16>(a, layer, e0, lo, hi, acc);
        else if (full && !plain) qu_rows<RNG16, true, false>(a.gp, a.keys, qc, M, e0, lo, hi, acc);       // nearly always
        else if (full) qu_rows<RNG16, true, true>(a.gp, a.keys, qc, M, e0, lo, hi, acc);
        else if (!plain) qu_rows<RNG16, false, false>(a.gp, a.keys, qc, M, e0, lo, hi, acc);
        else qu_rows<RNG16, false, true>(a.gp, a.keys, qc, M, e0, lo, hi, acc);
        if (TWO) {
            if (MODE == P_MODE_SHARED && a.code_sum) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (e0 + j >= lo && e0 + j < hi) a.code_sum[e0 + j] = (int)acc[j];
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
                acc[j] = (MODE == P_MODE_IDENTITY) ? acc[j] / a.M_f : (MODE == P_MODE_PER_WORKER) ? acc[j] / a.SM_f : acc[j] * f;
            p_st8(a.ghat, e0, lo, hi, acc, dat_policy_evict_last());   // the R part of a later item reads it again
#pragma unroll
            for (int j = 0; j < 8; ++j) ss_theta = fma((double)acc[j], (double)acc[j], ss_theta);
            continue;
        }
        // theta and m only now: registers are what limits the number of resident warps here.  (The same
        // arithmetic as p_direction, spelled out so that the loads are issued before g_hat is scaled: the step
        // is 3 % slower with the call.)
        float th[8], m[8];
        if (full) {                                 // theta is read again by the U part (evict-last), m is dead (evict-first)
            const uint64_t pf = dat_policy_evict_first(), pth = dat_policy_evict_last();
            const float4 t0 = dat_ld4_hint(a.theta + e0, pth), t1 = dat_ld4_hint(a.theta + e0 + 4, pth);
            const float4 m0 = dat_ld4_hint(a.mom + e0, pf), m1 = dat_ld4_hint(a.mom + e0 + 4, pf);
            th[0] = t0.x; th[1] = t0.y; th[2] = t0.z; th[3] = t0.w; th[4] = t1.x; th[5] = t1.y; th[6] = t1.z; th[7] = t1.w;
            m[0] = m0.x; m[1] = m0.y; m[2] = m0.z; m[3] = m0.w; m[4] = m1.x; m[5] = m1.y; m[6] = m1.z; m[7] = m1.w;
        } else {
            p_load4_cg(a.theta, e0, lo, hi, th);
            p_load4_cg(a.theta, e0 + 4, lo, hi, th + 4);
            p_load4_cg(a.mom, e0, lo, hi, m);
            p_load4_cg(a.mom, e0 + 4, lo, hi, m + 4);
        }
        if (MODE == P_MODE_SHARED && a.code_sum) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (e0 + j >= lo && e0 + j < hi) a.code_sum[e0 + j] = (int)acc[j];
        }
        if (OPT == P_OPT_LAMB) {
            // Algorithm A2: both moments are stored, the direction is formed on the fly for the layer sums
            float v[8];
            p_ld8(a.var, e0, lo, hi, v, dat_policy_evict_last());
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float ghat = (MODE == P_MODE_IDENTITY) ? acc[j] / a.M_f : (MODE == P_MODE_PER_WORKER) ? acc[j] / a.SM_f : acc[j] * f;
                m[j] = __fmaf_rn(a.lamb.beta1, m[j], __fmul_rn(a.lamb.om1, ghat));
                v[j] = __fmaf_rn(a.lamb.beta2, v[j], __fmul_rn(a.lamb.om2, __fmul_rn(ghat, ghat)));
                const bool inside = (e0 + j >= lo && e0 + j < hi);
                const float u = inside ? dat_lamb_direction(a.lamb, m[j], v[j], th[j]) : 0.0f;
                ss_theta = fma((double)th[j], (double)th[j], ss_theta);
                ss_u = fma((double)u, (double)u, ss_u);
            }
            p_st8(a.var, e0, lo, hi, v, dat_policy_evict_last());
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float ghat = (MODE == P_MODE_IDENTITY) ? acc[j] / a.M_f : (MODE == P_MODE_PER_WORKER) ? acc[j] / a.SM_f : acc[j] * f;
                m[j] = __fmaf_rn(a.mu, m[j], __fmaf_rn(a.wd, th[j], ghat));
                ss_theta = fma((double)th[j], (double)th[j], ss_theta);
                ss_u = fma((double)m[j], (double)m[j], ss_u);
            }
        }
        if (full) {
            const uint64_t pf = dat_policy_evict_last();   // the U part of a later item reads m' again
            dat_st4_hint(a.mom + e0, make_float4(m[0], m[1], m[2], m[3]), pf);
            dat_st4_hint(a.mom + e0 + 4, make_float4(m[4], m[5], m[6], m[7]), pf);
        } else {
            dat_store4(a.mom, e0, lo, hi, m);
            dat_store4(a.mom, e0 + 4, lo, hi, m + 4);
        }
    }
    __threadfence();                               // m' (and v'), or g_hat, are read by a later part of another CTA
    ss_theta = dat_warp_sum(ss_theta);
    ss_u = dat_warp_sum(ss_u);
    if ((threadIdx.x & 31) == 0) {
        scratch[2 * (threadIdx.x >> 5)] = ss_theta;
        scratch[2 * (threadIdx.x >> 5) + 1] = ss_u;
    }
}

// ---- R: Algorithm A1 Step 10 on one tile.  g_hat <- nu^_l * sign * level / S with the level of Eq. xi
// drawn on the random stream of index M (the first one no worker uses), then m' and the layer sums as in
// the Q part of the one-sided step. ------------------------------------------------------------------
template <bool RNG16, int OPT>
__device__ __forceinline__ void p_part_requant(const PArgs &a, const PipePart &pt, double *scratch)
{
    const int64_t lo = pt.lo, hi = pt.hi;
    const float t = __ldcg(a.qmul2 + pt.layer), f = __ldcg(a.dq2 + pt.layer);
    const float two_b = a.S_f + 1.0f;
    double ss_theta = 0.0, ss_u = 0.0;
    const int64_t begin = p_tile_begin(pt);
#pragma unroll 1
    for (int k = 0; k < DAT_P_GROUPS; ++k) {
        const int64_t e0 = begin + 8 * (int64_t)(k * DAT_P_THREADS + threadIdx.x);
        if (e0 >= hi) continue;
        float v[8];
        p_ld8(a.ghat, e0, lo, hi, v, dat_policy_evict_first());
        uint32_t w[8];
        if (RNG16) {
            dat_random_words((uint64_t)e0 >> 3, (uint32_t)a.M, a.keys, w);
        } else {
            dat_random_words((uint64_t)e0 >> 2, (uint32_t)a.M, a.keys, w);
            dat_random_words(((uint64_t)e0 >> 2) + 1, (uint32_t)a.M, a.keys, w + 4);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float u1 = RNG16 ? dat_u1_from_half((j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xFFFFu)) : dat_u1_from_word(w[j]);
            const int lev = (int)dat_level_u1(v[j], t, two_b, u1);
            v[j] = (float)((v[j] < 0.0f) ? -lev : lev) * f;
        }
        p_st8(a.ghat, e0, lo, hi, v, dat_policy_evict_first());   // the receiver's value
        p_direction<OPT>(a, e0, lo, hi, v, ss_theta, ss_u);
    }
    __threadfence();
    ss_theta = dat_warp_sum(ss_theta);
    ss_u = dat_warp_sum(ss_u);
    if ((threadIdx.x & 31) == 0) {
        scratch[2 * (threadIdx.x >> 5)] = ss_theta;
        scratch[2 * (threadIdx.x >> 5) + 1] = ss_u;
    }
}

// Two-sided step, one thread after the barrier that follows the Q part: the tile's sum of g_hat^2 (warps in
// index order), counted in.  Returns whether this was the layer's last tile.
__device__ __forceinline__ bool p_server_publish(const PArgs &a, const PipePart &pt, const double *scratch)
{
    double x = 0.0;
#pragma unroll
    for (int w = 0; w < DAT_P_THREADS / 32; ++w) x += scratch[2 * w];
    a.partR[(int64_t)pt.tb + pt.tile] = x;
    __threadfence();
    return atomicAdd(a.cntR + pt.layer, 1u) == (uint32_t)pt.T - 1u;
}

// The CTA that counted in the layer's last Q tile of a two-sided step (every thread): the server's norm
// nu^_l = ||g_hat_l||_2 from the tiles' sums in index order, and its two factors, published with the epoch.
__device__ __forceinline__ void p_server_finish(const PArgs &a, const PipePart &pt, double *scratch)
{
    const int layer = pt.layer;
    const int64_t tb = pt.tb;
    const uint32_t T = (uint32_t)pt.T;
    __threadfence();
    double x = 0.0;
    for (uint32_t t = threadIdx.x; t < T; t += DAT_P_THREADS) x += __ldcg(a.partR + tb + t);
    x = dat_warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        x = 0.0;
#pragma unroll
        for (int w = 0; w < DAT_P_THREADS / 32; ++w) x += scratch[w];
        const float nu = (float)sqrt(x);
        a.qmul2[layer] = (nu == 0.0f) ? 0.0f : a.S_f / nu;
        a.dq2[layer] = (nu == 0.0f) ? 0.0f : nu / a.S_f;
        if (a.server_scales_out) a.server_scales_out[layer] = nu;
        if (!isfinite(nu)) atomicOr(a.status, DAT_STATUS_NONFINITE);
        a.cntR[layer] = 0u;
        __threadfence();
        p_st_release(a.readyR + layer, a.epoch);
    }
}

// One thread, after the barrier that follows the Q part: the tile's two sums (warps in index order),
// counted in.  Returns whether this was the layer's last tile.
__device__ __forceinline__ bool p_quant_publish(const PArgs &a, const PipePart &pt, const double *scratch)
{
    double x = 0.0, y = 0.0;
#pragma unroll
    for (int w = 0; w < DAT_P_THREADS / 32; ++w) { x += scratch[2 * w]; y += scratch[2 * w + 1]; }
    a.partQ[2 * ((int64_t)pt.tb + pt.tile)] = x;
    a.partQ[2 * ((int64_t)pt.tb + pt.tile) + 1] = y;
    __threadfence();
    return atomicAdd(a.cntQ + pt.layer, 1u) == (uint32_t)pt.T - 1u;
}

// ---- U: theta' = theta - a_l m' (Eq. 3, pass 2) of one tile ---------------------------------------
template <int OPT>
__device__ __forceinline__ void p_part_update(const PArgs &a, const PipePart &pt)
{
    const int64_t lo = pt.lo, hi = pt.hi;
    const float na = -__ldcg(a.step_a + pt.layer);
    const uint64_t pol_first = dat_policy_evict_first();
    const int64_t begin = p_tile_begin(pt);
#pragma unroll
    for (int k = 0; k < DAT_P_GROUPS; ++k) {
        const int64_t e0 = begin + 8 * (int64_t)(k * DAT_P_THREADS + threadIdx.x);
        if (e0 >= hi) continue;
        if (OPT == P_OPT_LAMB) {
            // the direction once more from the stored moments: the same fp32 operations give the same bits
            float th[8], m[8], v[8];
            p_ld8(a.theta, e0, lo, hi, th, pol_first);
            p_ld8(a.mom, e0, lo, hi, m, pol_first);
            p_ld8(a.var, e0, lo, hi, v, pol_first);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool inside = (e0 + j >= lo && e0 + j < hi);
                const float u = inside ? dat_lamb_direction(a.lamb, m[j], v[j], th[j]) : 0.0f;
                th[j] = __fmaf_rn(na, u, th[j]);
            }
            p_st8(a.theta, e0, lo, hi, th, pol_first);
        } else if (e0 >= lo && e0 + 8 <= hi) {
            float4 t0 = dat_ld4_hint(a.theta + e0, pol_first), t1 = dat_ld4_hint(a.theta + e0 + 4, pol_first);
            const float4 m0 = dat_ld4_hint(a.mom + e0, pol_first), m1 = dat_ld4_hint(a.mom + e0 + 4, pol_first);
            t0.x = __fmaf_rn(na, m0.x, t0.x); t0.y = __fmaf_rn(na, m0.y, t0.y); t0.z = __fmaf_rn(na, m0.z, t0.z); t0.w = __fmaf_rn(na, m0.w, t0.w);
            t1.x = __fmaf_rn(na, m1.x, t1.x); t1.y = __fmaf_rn(na, m1.y, t1.y); t1.z = __fmaf_rn(na, m1.z, t1.z); t1.w = __fmaf_rn(na, m1.w, t1.w);
            dat_st4_hint(a.theta + e0, t0, pol_first);
            dat_st4_hint(a.theta + e0 + 4, t1, pol_first);
        } else {
            float th[8], m[8];
            p_load4_cg(a.theta, e0, lo, hi, th);
            p_load4_cg(a.theta, e0 + 4, lo, hi, th + 4);
            p_load4_cg(a.mom, e0, lo, hi, m);
            p_load4_cg(a.mom, e0 + 4, lo, hi, m + 4);
#pragma unroll
            for (int j = 0; j < 8; ++j) th[j] = __fmaf_rn(na, m[j], th[j]);
            dat_store4(a.theta, e0, lo, hi, th);
            dat_store4(a.theta, e0 + 4, lo, hi, th + 4);
        }
    }
}

template <bool RNG16, int MODE, int OPT, bool TWO>
__global__ void __launch_bounds__(DAT_P_THREADS, DAT_P_MINB)
k_step_pipelined(const __grid_constant__ PArgs a)
{
    __shared__ double s_unit[4 * DAT_MAX_WORKERS];
    __shared__ float s_norm[DAT_MAX_WORKERS];
    __shared__ __align__(16) PipeItem s_item;
    __shared__ int s_ctl[4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // items are taken in the order in which CTAs start, whatever order the hardware starts them in
    if (warp == 0) {
        uint32_t tk = 0;
        if (lane == 0) {
            tk = atomicAdd(a.ticket, 1u);
            if (tk == a.n_items - 1u) *a.ticket = 0u;  // every ticket of this call is out: ready for the next call
        }
        tk = __shfl_sync(0xFFFFFFFFu, tk, 0);
        if (!P_CHECK(a, tk < a.n_items)) tk = 0;
        if (lane < (int)((TWO ? sizeof(PipeItem) : 3 * sizeof(PipePart)) / 16))
            reinterpret_cast<uint4 *>(&s_item)[lane] = __ldg(reinterpret_cast<const uint4 *>(a.items + tk) + lane);
    }
    for (int u = threadIdx.x; u < 4 * a.M; u += DAT_P_THREADS) s_unit[u] = 0.0;
    __syncthreads();
    const PipePart pn = s_item.n, pq = s_item.q, pu = s_item.u;
    PipePart pm = pq;                               // the part that leaves m' and the tile's two sums of Eq. 3
#ifdef DAT_SELFCHECK
    {
        bool ok = pn.layer < a.h && pq.layer < a.h && pu.layer < a.h;
        const PipePart pr = TWO ? s_item.r : pq;
        ok = ok && pr.layer < a.h;
        const PipePart *pp[4] = {&pn, &pq, &pu, &pr};
        for (int k = 0; k < 4 && ok; ++k)
            if (pp[k]->layer >= 0)
                ok = pp[k]->tile >= 0 && pp[k]->tile < pp[k]->T && (int64_t)pp[k]->tb + pp[k]->tile < a.n_tiles &&
                     pp[k]->lo >= 0 && pp[k]->lo < pp[k]->hi && pp[k]->hi <= a.d;
        if (!P_CHECK(a, ok)) return;
    }
#endif
    // The CTA meets at five barriers: item read; N sums in shared memory; (A) tile counted in and the Q part's
    // layer known to be published; Q sums in shared memory; (B) tile counted in and the U part's layer
    // published.  Between them warp 0 does the publishing and the polling.
    if (pn.layer >= 0) p_norm_sums(a, pn, s_unit);
    __syncthreads();
    if (warp == 0) {
        bool n_last = false, q_go = true;
        if (pn.layer >= 0) n_last = p_norm_publish(a, pn, s_unit);
        if (lane == 0) {
            if (pq.layer >= 0 && MODE != P_MODE_IDENTITY) q_go = p_poll(a, a.readyN + pq.layer);
            s_ctl[0] = n_last;
            s_ctl[1] = q_go;
        }
    }
    __syncthreads();                               // (A)
    if (s_ctl[0]) p_norm_finish<MODE>(a, pn, s_norm);
    bool alive = (s_ctl[1] != 0);
    if (alive && pq.layer >= 0) p_part_quant<RNG16, MODE, OPT, TWO>(a, pq, s_unit);
    __syncthreads();
    if (TWO) {
        // Step 10: the tile's sum of g_hat^2 counted in; the layer's last tile publishes the server's norm;
        // then the R part of this item (a tile of an earlier layer) once that layer's norm is published
        pm = s_item.r;
        if (threadIdx.x == 0) s_ctl[2] = (alive && pq.layer >= 0) ? (int)p_server_publish(a, pq, s_unit) : 0;
        __syncthreads();
        if (s_ctl[2]) p_server_finish(a, pq, s_unit);
        if (threadIdx.x == 0) s_ctl[1] = (alive && pm.layer >= 0) ? (int)p_poll(a, a.readyR + pm.layer) : (int)alive;
        __syncthreads();
        alive = (s_ctl[1] != 0);
        if (alive && pm.layer >= 0) p_part_requant<RNG16, OPT>(a, pm, s_unit);
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        bool q_last = false, u_go = alive;
        if (alive && pm.layer >= 0) q_last = p_quant_publish(a, pm, s_unit);
        if (alive && pu.layer >= 0) u_go = p_poll(a, a.readyQ + pu.layer);
        s_ctl[2] = q_last;
        s_ctl[3] = u_go;
    }
    __syncthreads();                               // (B)
    if (s_ctl[2]) p_quant_finish(a, pm, s_unit);
    if (s_ctl[3] && pu.layer >= 0) p_part_update<OPT>(a, pu);
}

// ---- host: the item list -----------------------------------------------------------------------------
void dat_pipe_destroy(dat_plan_t *plan)
{
    if (!plan->pipe) return;
    if (plan->pipe->mem) cudaFree(plan->pipe->mem);
    delete plan->pipe;
    plan->pipe = nullptr;
}

static size_t p_align(size_t x) { return (x + 255) / 256 * 256; }

// Called by dat_plan_create (device current).  Allocates the schedule's tables (synchronous).
int dat_pipe_build(dat_plan_t *plan)
{
    PipeSchedule *g = new (std::nothrow) PipeSchedule();
    if (!g) return DAT_ERR_NOMEM;
    plan->pipe = g;
    const int h = (int)plan->h, M = plan->M;
    const bool identity = (plan->bits == 32);
    try {
        std::vector<int64_t> tb((size_t)h + 1);
        int64_t nt = 0;
        for (int l = 0; l < h; ++l) {
            tb[l] = nt;
            nt += (plan->offsets[l + 1] - (plan->offsets[l] & ~(int64_t)7) + DAT_P_TILE - 1) / DAT_P_TILE;
        }
        tb[h] = nt;
        g->n_tiles = nt;
        if (nt > ((int64_t)1 << 30)) return DAT_ERR_UNSUPPORTED;
        // layers smallest first (ties in index order): the distance between the N and the Q stream is the
        // size of the layer being worked on, so it grows slowly and the streams stay paired to the end
        std::vector<int> order((size_t)h);
        for (int l = 0; l < h; ++l) order[l] = l;
        std::stable_sort(order.begin(), order.end(), [&](int x, int y) {
            return plan->offsets[x + 1] - plan->offsets[x] < plan->offsets[y + 1] - plan->offsets[y];
        });
        // slot of every tile in each of the three streams (four with the server's quantizer between Q and U)
        const PipePart nopart = {0, 1, 0, 1, -1, 0};
        const PipeItem none = {nopart, nopart, nopart, nopart};
        auto part = [&](int l, int64_t t) {
            PipePart pp = {plan->offsets[l], plan->offsets[l + 1], (int32_t)tb[l], (int32_t)(tb[l + 1] - tb[l]), l, (int32_t)t};
            return pp;
        };
        auto build = [&](bool two) {
            std::vector<PipeItem> items;
            auto at = [&](int64_t slot) -> PipeItem & {
                if ((int64_t)items.size() <= slot) items.resize((size_t)slot + 1, none);
                return items[(size_t)slot];
            };
            std::vector<int64_t> done_n((size_t)h, -1 - (int64_t)DAT_P_LAG), done_q((size_t)h, 0), done_r((size_t)h, 0);
            int64_t slot = 0;
            if (!identity)
                for (int k = 0; k < h; ++k) {
                    const int l = order[k];
                    for (int64_t t = 0; t < tb[l + 1] - tb[l]; ++t) { at(slot).n = part(l, t); done_n[l] = slot++; }
                }
            slot = 0;
            for (int k = 0; k < h; ++k) {
                const int l = order[k];
                const int64_t T = tb[l + 1] - tb[l];
                slot = std::max(slot, done_n[l] + DAT_P_LAG + 1);
                // a layer that L2 cannot hold next to what streams in meanwhile is walked back from its last
                // tile (what N read last, and marked to stay, is read first); the others in N's order
                const bool reverse = T >= DAT_P_REVERSE_FROM;
                for (int64_t t = 0; t < T; ++t) { at(slot).q = part(l, reverse ? T - 1 - t : t); done_q[l] = slot++; }
            }
            if (two) {
                slot = 0;
                for (int k = 0; k < h; ++k) {
                    const int l = order[k];
                    slot = std::max(slot, done_q[l] + DAT_P_LAG_U + 1);
                    for (int64_t t = 0; t < tb[l + 1] - tb[l]; ++t) { at(slot).r = part(l, t); done_r[l] = slot++; }
                }
            }
            slot = 0;
            for (int k = 0; k < h; ++k) {
                const int l = order[k];
                slot = std::max(slot, (two ? done_r[l] : done_q[l]) + DAT_P_LAG_U + 1);
                for (int64_t t = 0; t < tb[l + 1] - tb[l]; ++t) { at(slot).u = part(l, t); ++slot; }
            }
            return items;
        };
        const std::vector<PipeItem> items = build(false);
        const std::vector<PipeItem> items2 = identity ? std::vector<PipeItem>() : build(true);
        g->n_items2 = (int64_t)items2.size();
        g->n_items = (int64_t)items.size();

        size_t off = 0;
        auto take = [&](size_t bytes) { size_t o = off; off = p_align(off + bytes); return o; };
        const size_t o_items = take(items.size() * sizeof(PipeItem)), o_items2 = take(items2.size() * sizeof(PipeItem));
        const size_t o_tb = take(((size_t)h + 1) * 8);
        const size_t o_pn = take((size_t)nt * (size_t)M * 8), o_pq = take((size_t)nt * 16), o_pr = take((size_t)nt * 8);
        const size_t o_server = take(2 * (size_t)h * 4);
        g->sync_bytes = (2 + 6 * (size_t)h) * 4;
        const size_t o_sync = take(g->sync_bytes);
        g->mem_bytes = off;
        cudaError_t e;
        e = cudaMalloc((void **)&g->mem, off);
        if (e != cudaSuccess) { g->mem = nullptr; plan->last_cuda = (int)e; (void)cudaGetLastError(); return DAT_ERR_NOMEM; }
        g->d_items = (PipeItem *)(g->mem + o_items);
        g->d_items2 = (PipeItem *)(g->mem + o_items2);
        g->d_partR = (double *)(g->mem + o_pr);
        g->d_server = (float *)(g->mem + o_server);
        g->d_tile_base = (int64_t *)(g->mem + o_tb);
        g->d_partN = (double *)(g->mem + o_pn);
        g->d_partQ = (double *)(g->mem + o_pq);
        g->d_sync = (uint32_t *)(g->mem + o_sync);
        e = cudaMemset(g->mem, 0, off);
        if (e == cudaSuccess) e = cudaMemcpy(g->d_items, items.data(), items.size() * sizeof(PipeItem), cudaMemcpyHostToDevice);
        if (e == cudaSuccess && !items2.empty())
            e = cudaMemcpy(g->d_items2, items2.data(), items2.size() * sizeof(PipeItem), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(g->d_tile_base, tb.data(), ((size_t)h + 1) * 8, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) return dat_cuda_fail(plan, e);
    } catch (...) {
        return DAT_ERR_NOMEM;
    }
    return DAT_OK;
}

// After a call that timed out the arrival counters and the ticket are left mid-way: clear them
// (enqueued on `s`; called by dat_get_status when it finds DAT_STATUS_TIMEOUT).
cudaError_t dat_pipe_reset(dat_plan_t *plan, cudaStream_t s)
{
    PipeSchedule *g = plan->pipe;
    if (!g || !g->mem) return cudaSuccess;
    return cudaMemsetAsync(g->d_sync, 0, g->sync_bytes, s);
}

// One launch of the step.  lamb == nullptr: the momentum direction with hp; else Algorithm A2 with *lamb.
// g_hat != nullptr: the two-sided step (Algorithm A1 Step 10 between the aggregation and the update).
static int p_launch(dat_plan_t *plan, float *theta, float *mom, float *var, const float *const *grads,
                    uint64_t seed, uint64_t step, const dat_hparams_t *hp, const LambConst *lamb, float lr, float c_l, float c_u,
                    int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream,
                    float *g_hat = nullptr, float *server_scales_out = nullptr)
{
    if (step >> 32) return DAT_ERR_ARG;
    if (plan->elem_base || plan->worker_base) return DAT_ERR_UNSUPPORTED;     // a slice of a larger problem: separate calls only
    if (!dat_aligned16(theta) || !dat_aligned16(mom) || (var && !dat_aligned16(var)) || (code_sum_out && !dat_aligned16(code_sum_out)) ||
        (layer_norms_out && !dat_aligned16(layer_norms_out)) || (scales_out && !dat_aligned16(scales_out)) ||
        (g_hat && !dat_aligned16(g_hat)) || (server_scales_out && !dat_aligned16(server_scales_out)))
        return DAT_ERR_ALIGN;
    const bool two = (g_hat != nullptr);
    {   // the call's epoch and the Philox key are launch parameters: a captured graph would replay them unchanged
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing((cudaStream_t)stream, &cap) != cudaSuccess) { (void)cudaGetLastError(); return DAT_ERR_CUDA; }
        if (cap != cudaStreamCaptureStatusNone) return DAT_ERR_UNSUPPORTED;
    }
    if (two && plan->bits == 32) return DAT_ERR_BITS;      // nothing to quantize with
    PArgs a;
    int rc = dat_check_grads(plan, grads, &a.gp);
    if (rc != DAT_OK) return rc;
    PipeSchedule *g = plan->pipe;
    if (!g || !g->mem) return DAT_ERR_ARG;
    const bool identity = (plan->bits == 32);
    const bool per_worker = !identity && plan->scale_mode == DAT_SCALE_PER_WORKER;
    const size_t h = (size_t)plan->h;
    a.keys = dat_make_keys(seed, step);
    a.items = two ? g->d_items2 : g->d_items;
    a.off = plan->d_offsets;
    a.tile_base = g->d_tile_base;
    a.theta = theta;
    a.mom = mom;
    a.var = var;
    if (lamb) a.lamb = *lamb;
    else a.lamb = LambConst{0.0f, 0.0f, 0.0f, 0.0f, 1.0f, 1.0f, 1.0f, 0.0f};
    a.partN = g->d_partN;
    a.partQ = g->d_partQ;
    a.partR = g->d_partR;
    a.ticket = g->d_sync;
    a.abort_epoch = g->d_sync + 1;
    a.cntN = g->d_sync + 2;
    a.cntQ = a.cntN + h;
    a.readyN = a.cntQ + h;
    a.readyQ = a.readyN + h;
    a.cntR = a.readyQ + h;
    a.readyR = a.cntR + h;
    a.ghat = g_hat;
    a.qmul2 = g->d_server;
    a.dq2 = g->d_server + h;
    a.server_scales_out = server_scales_out;
    a.status = plan->d_status;
    a.worker_norms = plan->d_worker_norms;
    a.scales = plan->d_scales;
    a.qmul = plan->d_qmul;
    a.dq = plan->d_dq;
    a.step_a = plan->d_step_a;
    a.norms_out = layer_norms_out;
    a.scales_out = identity ? nullptr : scales_out;
    a.code_sum = (identity || per_worker) ? nullptr : code_sum_out;
    a.wait_cycles = g->wait_cycles;
    a.S_f = (float)plan->S;
    a.SM_f = (float)((uint64_t)plan->S * (uint64_t)plan->M);
    a.M_f = (float)plan->M;
    a.mu = hp ? hp->momentum : 0.0f;
    a.wd = hp ? hp->weight_decay : 0.0f;
    a.lr = lr;
    a.c_l = c_l;
    a.c_u = c_u;
    if (++g->epoch == 0u) ++g->epoch;              // 0 is what the words hold before the first call
    a.epoch = g->epoch;
    a.n_items = (uint32_t)(two ? g->n_items2 : g->n_items);
    a.M = plan->M;
    a.h = (int)plan->h;
    a.d = plan->d;
    a.n_tiles = g->n_tiles;
    cudaStream_t s = (cudaStream_t)stream;
    const unsigned grid = a.n_items;
    const bool rng16 = (plan->rng_bits == 16);
#define P_GO(R, MODE, OPT, TWO) k_step_pipelined<R, MODE, OPT, TWO><<<grid, DAT_P_THREADS, 0, s>>>(a)
#define P_GO_OPT(R, MODE)                                                                                           \
    do {                                                                                                            \
        if (two) { if (lamb) P_GO(R, MODE, P_OPT_LAMB, true); else P_GO(R, MODE, P_OPT_MOMENTUM, true); }           \
        else if (lamb) P_GO(R, MODE, P_OPT_LAMB, false);                                                            \
        else P_GO(R, MODE, P_OPT_MOMENTUM, false);                                                                  \
    } while (0)
    if (identity) { if (lamb) P_GO(true, P_MODE_IDENTITY, P_OPT_LAMB, false); else P_GO(true, P_MODE_IDENTITY, P_OPT_MOMENTUM, false); }
    else if (per_worker && rng16) P_GO_OPT(true, P_MODE_PER_WORKER);
    else if (per_worker) P_GO_OPT(false, P_MODE_PER_WORKER);
    else if (rng16) P_GO_OPT(true, P_MODE_SHARED);
    else P_GO_OPT(false, P_MODE_SHARED);
#undef P_GO_OPT
#undef P_GO
    DAT_LAUNCHED(plan);
    return DAT_OK;
}

extern "C" int dat_step_pipelined(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                                  uint64_t seed, uint64_t step, const dat_hparams_t *hp,
                                  int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !hp) return DAT_ERR_ARG;
    return p_launch(plan, theta, mom, nullptr, grads, seed, step, hp, nullptr, hp->lr, hp->c_l, hp->c_u, code_sum_out,
                    layer_norms_out, scales_out, stream);
}

extern "C" int dat_step_lamb(dat_plan_t *plan, float *theta, float *mom, float *var, const float *const *grads,
                             uint64_t seed, uint64_t step, const dat_lamb_hparams_t *hp, int64_t t,
                             int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !var || !hp || t < 1) return DAT_ERR_ARG;
    if (!(hp->beta1 > 0.0f && hp->beta1 < 1.0f && hp->beta2 > 0.0f && hp->beta2 < 1.0f)) return DAT_ERR_ARG;
    const LambConst c = dat_lamb_const(hp, t);
    return p_launch(plan, theta, mom, var, grads, seed, step, nullptr, &c, hp->lr, hp->c_l, hp->c_u, code_sum_out,
                    layer_norms_out, scales_out, stream);
}

extern "C" int dat_step_two_sided(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                                  uint64_t seed, uint64_t step, const dat_hparams_t *hp, float *g_hat,
                                  int32_t *code_sum_out, float *layer_norms_out, float *scales_out,
                                  float *server_scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !hp || !g_hat) return DAT_ERR_ARG;
    return p_launch(plan, theta, mom, nullptr, grads, seed, step, hp, nullptr, hp->lr, hp->c_l, hp->c_u, code_sum_out,
                    layer_norms_out, scales_out, stream, g_hat, server_scales_out);
}

extern "C" int dat_step_lamb_two_sided(dat_plan_t *plan, float *theta, float *mom, float *var, const float *const *grads,
                                       uint64_t seed, uint64_t step, const dat_lamb_hparams_t *hp, int64_t t, float *g_hat,
                                       int32_t *code_sum_out, float *layer_norms_out, float *scales_out,
                                       float *server_scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !var || !hp || !g_hat || t < 1) return DAT_ERR_ARG;
    if (!(hp->beta1 > 0.0f && hp->beta1 < 1.0f && hp->beta2 > 0.0f && hp->beta2 < 1.0f)) return DAT_ERR_ARG;
    const LambConst c = dat_lamb_const(hp, t);
    return p_launch(plan, theta, mom, var, grads, seed, step, nullptr, &c, hp->lr, hp->c_l, hp->c_u, code_sum_out,
                    layer_norms_out, scales_out, stream, g_hat, server_scales_out);
}

// Test hook (see dat.h): a short wait limit, and a layer whose norm never completes in the next call.
extern "C" int dat_plan_test_stall(dat_plan_t *plan, int64_t wait_cycles, int64_t layer, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    PipeSchedule *g = plan->pipe;
    if (!g || !g->mem || wait_cycles < 0 || layer >= plan->h) return DAT_ERR_ARG;
    g->wait_cycles = wait_cycles ? (long long)wait_cycles : DAT_P_WAIT_CYCLES;
    if (layer >= 0) {
        // a count that the layer's tiles cannot bring to T - 1: nobody becomes the layer's last tile
        static const uint32_t far = 0x40000000u;
        DAT_CUDA(plan, cudaMemcpyAsync(g->d_sync + 2 + layer, &far, sizeof far, cudaMemcpyHostToDevice, (cudaStream_t)stream));
        DAT_CUDA(plan, cudaStreamSynchronize((cudaStream_t)stream));
    }
    return DAT_OK;
}
