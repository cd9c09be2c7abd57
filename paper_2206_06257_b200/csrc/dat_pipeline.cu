// dat_step_pipelined: Steps 7, 9 and 12 of Algorithm A1 in ONE launch of ordinary (non-persistent)
// CTAs that reads every gradient from HBM once.
//
// The quantizer norm of a layer (Eq. rand_q) must be known before the first level of that layer
// (Eq. xi) can be drawn, and the two layer norms of Eq. 3 before the first parameter moves: three
// phases per layer, each needing the previous one complete for the whole layer.  The flat vector is
// cut into per-layer tiles, and the host lays three streams of tiles side by side in one list of
// work items: item s holds (at most) one tile for each phase,
//     N  sums of squares of the gradients of a tile          (gradients come from HBM),
//     Q  levels, signed sum, g_hat, m', layer sums of a tile  (the same gradients, now from L2),
//     U  theta update of a tile                               (theta and m' still in L2),
// where the Q stream runs behind the N stream, and the U stream behind the Q stream, by the size of
// the layer plus a fixed number of items.  A CTA takes the next item by an atomic ticket, so items
// start in list order, and does its N part first: the sums a later item waits for are produced by
// CTAs that started earlier and never wait themselves.  The last CTA to finish a layer's N (or Q)
// tiles reduces the layer's partial sums in a fixed order and publishes the layer's factors with the
// call's epoch; a Q (or U) part whose layer is not published yet polls that word, with a limit.
#include <algorithm>
#include <new>
#include <vector>

#include "dat_internal.cuh"

#define DAT_P_THREADS 256
#define DAT_P_TILE 2048                           // elements per tile (eight per thread), tiles start on multiples of 8
#ifndef DAT_P_MINB
#define DAT_P_MINB 4
#endif
#ifndef DAT_P_LAG                                 // items between the last N tile of a layer and its first Q tile
#define DAT_P_LAG 384
#endif
#ifndef DAT_P_REVERSE_FROM                        // layers of at least this many tiles: Q walks back from the last tile
#define DAT_P_REVERSE_FROM 640
#endif
#ifndef DAT_P_N_POLICY                            // L2 priority of the gradients when they are first read
#define DAT_P_N_POLICY dat_policy_evict_last
#endif
#define DAT_P_WAIT_CYCLES (4000000000ll)          // about two seconds

enum { P_MODE_SHARED = 0, P_MODE_IDENTITY = 2 };

struct PipePart {                                 // one tile of one layer; layer < 0: none
    int64_t lo, hi;                               // the layer's element range
    int32_t tb, T;                                // first tile of the layer in the partial-sum tables, tiles of the layer
    int32_t layer, tile;
};
struct PipeItem {
    PipePart n, q, u;
};

struct PipeSchedule {
    char *mem = nullptr;                          // one device allocation, carved up
    size_t mem_bytes = 0;
    PipeItem *d_items = nullptr;
    int64_t n_items = 0;
    int64_t *d_tile_base = nullptr;               // h + 1
    double *d_partN = nullptr;                    // n_tiles * M
    double *d_partQ = nullptr;                    // n_tiles * 2
    uint32_t *d_sync = nullptr;                   // [0] ticket, [1] abort epoch, then cntN[h], cntQ[h], readyN[h], readyQ[h]
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
    float *theta, *mom;
    double *partN, *partQ;
    uint32_t *ticket, *abort_epoch, *cntN, *cntQ, *readyN, *readyQ, *status;
    float *worker_norms, *scales, *qmul, *dq, *step_a;
    float *norms_out, *scales_out;
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

// Arrival of one tile of a layer: true (in every thread) in the CTA that arrives last.  Every
// thread has fenced what it wrote for the layer.
__device__ __forceinline__ bool p_arrive(uint32_t *cnt, uint32_t total, int *s_flag)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        *s_flag = (atomicAdd(cnt, 1u) == total - 1u);
    }
    __syncthreads();
    const bool last = (*s_flag != 0);
    __syncthreads();
    if (last) __threadfence();
    return last;
}

// Waits until `word` carries this call's epoch.  Bounded: when the limit runs out the status word
// gets DAT_STATUS_TIMEOUT and the call's abort word is set, which ends every other wait at once.
// Returns false (in every thread) if the part must be skipped.
__device__ __forceinline__ bool p_wait(const PArgs &a, const uint32_t *word, int *s_flag)
{
    if (threadIdx.x == 0) {
        bool ok = (p_ld_acquire(word) == a.epoch);
        if (!ok) {
            const long long t0 = clock64();
            for (;;) {
                __nanosleep(128);
                if (p_ld_acquire(word) == a.epoch) { ok = true; break; }
                if (p_ld_acquire(a.abort_epoch) == a.epoch) break;
                if (clock64() - t0 > a.wait_cycles) {
                    atomicOr(a.status, DAT_STATUS_TIMEOUT);
                    p_st_release(a.abort_epoch, a.epoch);
                    break;
                }
            }
        }
        *s_flag = ok ? 1 : 0;
    }
    __syncthreads();
    const bool ok = (*s_flag != 0);
    __syncthreads();
    return ok;
}

// ---- staging through shared memory ---------------------------------------------------------------
// Every thread streams its own sequence of 32-byte entries (two 16-byte slots) through a private
// ring in shared memory: the parts of the N tile it sums, then for its eight elements of the Q tile
// one entry per worker, theta and m, then theta and m' of its eight elements of the U tile.  Entry j
// sits in ring position j mod DAT_P_DEPTH; it is fetched by two asynchronous 16-byte copies DEPTH
// entries ahead of its use, across the borders of the three parts, and read back by the thread that
// fetched it -- so the copies need no barrier, only the thread's own wait for its copy groups, and
// what is in flight costs no registers.  Slot k of thread t is p_stage[k * 256 + t].
extern __shared__ float4 p_stage[];
#ifndef DAT_P_DEPTH
#define DAT_P_DEPTH 6
#endif
#define DAT_P_STAGE_BYTES (2 * DAT_P_DEPTH * DAT_P_THREADS * 16)

// Self-checking build (-DDAT_SELFCHECK): every address formed from an item is checked before it is used;
// a violation sets DAT_STATUS_BOUNDS and the access is skipped, nothing faults.
#ifdef DAT_SELFCHECK
#define P_CHECK(a, cond) ((cond) ? true : (atomicOr((a).status, DAT_STATUS_BOUNDS), false))
#else
#define P_CHECK(a, cond) true
#endif

__device__ __forceinline__ void p_cp16(const PArgs &a, float4 *dst, const float *base, int64_t e, uint64_t pol)
{
    const float *src = base + e;
#ifdef DAT_SELFCHECK
    const int64_t slot_off = (const char *)dst - (const char *)p_stage;
    if (!P_CHECK(a, e >= 0 && e + 4 <= a.d && ((uintptr_t)src & 15u) == 0 && slot_off >= 0 &&
                    slot_off + 16 <= DAT_P_STAGE_BYTES && (slot_off & 15) == 0)) return;
#endif
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" :: "r"(d), "l"(src), "l"(pol) : "memory");
}
__device__ __forceinline__ void p_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void p_cp_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

// What a thread needs to know to fetch entry j of its sequence.
struct Seq {
    int nN, nQ, nU;                                // entries of the three parts (0: that part reads global memory itself)
    int u0;                                        // N: first unit of this warp
    int64_t eN, eQ, eU;                            // N: tile begin + 4 lane; Q, U: the thread's first element
    uint64_t pol_last, pol_first, pol_normal;
};

__device__ __forceinline__ void p_issue(const PArgs &a, const Seq &q, int j)
{
    float4 *dst = p_stage + (2 * (j % DAT_P_DEPTH)) * DAT_P_THREADS + threadIdx.x;
    if (j < q.nN) {
        // unit u = u0 + j/2 (worker u/4, quarter u%4), its copies 2(j%2) and 2(j%2)+1 of four
        const int u = q.u0 + (j >> 1);
        const int64_t e = q.eN + (u & 3) * (DAT_P_TILE / 4) + 256 * (j & 1);
        p_cp16(a, dst, a.gp.p[u >> 2], e, q.pol_last);
        p_cp16(a, dst + DAT_P_THREADS, a.gp.p[u >> 2], e + 128, q.pol_last);
    } else if (j < q.nN + q.nQ) {
        const int i = j - q.nN;
        const float *base = (i < a.M) ? a.gp.p[i] : (i == a.M ? a.theta : a.mom);
        const uint64_t pol = (i < a.M) ? q.pol_first : q.pol_normal;     // a gradient is dead once its level is drawn
        p_cp16(a, dst, base, q.eQ, pol);
        p_cp16(a, dst + DAT_P_THREADS, base, q.eQ + 4, pol);
    } else if (j < q.nN + q.nQ + q.nU) {
        const float *base = (j == q.nN + q.nQ) ? a.theta : a.mom;
        p_cp16(a, dst, base, q.eU, q.pol_first);
        p_cp16(a, dst + DAT_P_THREADS, base, q.eU + 4, q.pol_first);
    }
    p_cp_commit();                                 // one group per entry, also past the end: the count stays uniform
}

// Entry j has arrived (every entry up to j + DEPTH - 1 has been issued): its eight floats.
__device__ __forceinline__ void p_take(int j, float v[8])
{
    p_cp_wait<DAT_P_DEPTH - 1>();
    const float4 *src = p_stage + (2 * (j % DAT_P_DEPTH)) * DAT_P_THREADS + threadIdx.x;
    const float4 a0 = src[0], a1 = src[DAT_P_THREADS];
    v[0] = a0.x; v[1] = a0.y; v[2] = a0.z; v[3] = a0.w; v[4] = a1.x; v[5] = a1.y; v[6] = a1.z; v[7] = a1.w;
}

// ---- N: sums of squares of one tile, every worker ------------------------------------------------
// A tile is cut into 4M units (worker, quarter tile of 512 elements); warp w takes the units
// [w*4M/8, (w+1)*4M/8), a unit being two entries per lane.  Units of the same worker are summed per
// lane before the warp reduction; the structure depends on M only, so the sums are the same from
// run to run.
__device__ __forceinline__ void p_norm_sums(const PArgs &a, const PipePart &pt, const Seq &q, double *s_unit)
{
    const int M = a.M;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int U = 4 * M;
    const int u0 = warp * U / 8, u1 = (warp + 1) * U / 8;
    double acc = 0.0;
    int run = u0;
    if (q.nN > 0) {
#pragma unroll 1
        for (int j = 0; j < q.nN; ++j) {
            const int u = u0 + (j >> 1);
            if ((u >> 2) != (run >> 2)) {
                acc = dat_warp_sum(acc);
                if (lane == 0) s_unit[run] = acc;
                acc = 0.0;
                run = u;
            }
            float v[8];
            p_take(j, v);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc = fma((double)v[k], (double)v[k], acc);
            p_issue(a, q, j + DAT_P_DEPTH);        // into the slots just read
        }
    } else {
        const int64_t begin = (pt.lo & ~(int64_t)7) + (int64_t)pt.tile * DAT_P_TILE;
#pragma unroll 1
        for (int u = u0; u < u1; ++u) {
            if ((u >> 2) != (run >> 2)) {
                acc = dat_warp_sum(acc);
                if (lane == 0) s_unit[run] = acc;
                acc = 0.0;
                run = u;
            }
            const float *__restrict__ g = a.gp.p[u >> 2];
            const int64_t e = begin + (u & 3) * (DAT_P_TILE / 4) + 4 * lane;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
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

// Writes the tile's M partial sums, counts the tile in, and in the CTA that holds the layer's last
// tile: nu_{i,l} = sqrt(sum over the tiles), nu_l = max_i, and the layer's two factors.
__device__ __forceinline__ void p_norm_publish(const PArgs &a, const PipePart &pt, double *s_unit, float *s_norm, int *s_flag)
{
    const int M = a.M, layer = pt.layer;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t tb = pt.tb;
    const uint32_t T = (uint32_t)pt.T;
    __syncthreads();                               // every warp's unit sums are in s_unit
    if (threadIdx.x < M) {
        const double *s = s_unit + 4 * threadIdx.x;
        a.partN[(tb + pt.tile) * M + threadIdx.x] = ((s[0] + s[1]) + s[2]) + s[3];
        __threadfence();
    }
    if (!p_arrive(a.cntN + layer, T, s_flag)) return;
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
        a.scales[layer] = nu;
        a.qmul[layer] = (nu == 0.0f) ? 0.0f : a.S_f / nu;
        a.dq[layer] = (nu == 0.0f) ? 0.0f : nu / a.SM_f;
        if (a.scales_out) a.scales_out[layer] = nu;
        if (bad) atomicOr(a.status, DAT_STATUS_NONFINITE);
        a.cntN[layer] = 0u;
        __threadfence();
        p_st_release(a.readyN + layer, a.epoch);
    }
}

// ---- the layer's step length from the partial sums of theta^2 and m'^2 (Eq. 3), by the last Q tile --
__device__ __forceinline__ void p_finish_update_sums(const PArgs &a, int layer, int64_t tb, uint32_t T, double *scratch)
{
    double x = 0.0, y = 0.0;
    for (uint32_t t = threadIdx.x; t < T; t += DAT_P_THREADS) {
        x += __ldcg(a.partQ + 2 * (tb + t));
        y += __ldcg(a.partQ + 2 * (tb + t) + 1);
    }
    x = dat_block_sum(x, scratch);
    y = dat_block_sum(y, scratch);
    if (threadIdx.x == 0) {
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

// One worker's eight elements: levels by the scaled form of Eq. xi, signed float sum (exact).
template <bool RNG16>
__device__ __forceinline__ void p_levels8(const float v[8], const uint32_t w[8], const QuConst &qc, float acc[8])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float u1s;
        if (RNG16) u1s = __fmaf_rn(__uint_as_float(__byte_perm(w[j >> 1], 0x4B000000u, (j & 1) ? 0x7632 : 0x7610)), qc.c0, qc.c1);
        else u1s = __uint_as_float(qc.ubits | (w[j] & 0x007FFFFFu));
        const float ys = __saturatef(__fmaf_rn(fabsf(v[j]), qc.ts, u1s));
        const float lf = __fmaf_rz(ys, qc.two_b, 8388607.0f) - 8388608.0f;
        const float sg = __uint_as_float((__float_as_uint(v[j]) & 0x80000000u) | 0x3F800000u);
        acc[j] = __fmaf_rn(lf, sg, acc[j]);
    }
}

template <bool RNG16>
__device__ __forceinline__ void p_words8(const PArgs &a, int64_t e0, uint32_t worker, uint32_t w[8])
{
    if (RNG16) {
        dat_random_words((uint64_t)e0 >> 3, worker, a.keys, w);
    } else {
        dat_random_words((uint64_t)e0 >> 2, worker, a.keys, w);
        dat_random_words(((uint64_t)e0 >> 2) + 1, worker, a.keys, w + 4);
    }
}

// ---- Q: levels (Eq. xi), signed sum over the workers and g_hat (Eq. grad_agg), m' and the layer sums
// (Eq. 3, pass 1) of one tile; codes, sums and g_hat stay in registers ----------------------------
template <bool RNG16, int MODE>
__device__ __forceinline__ void p_part_quant(const PArgs &a, const PipePart &pt, const Seq &q, double *scratch, int *s_flag)
{
    const int M = a.M, layer = pt.layer;
    const int64_t lo = pt.lo, hi = pt.hi;
    float t = 0.0f, f = 0.0f;
    if (MODE != P_MODE_IDENTITY) { t = __ldcg(a.qmul + layer); f = __ldcg(a.dq + layer); }
    const float two_b = a.S_f + 1.0f, inv_two_b = 1.0f / two_b;
    // scaled form of Eq. xi: valid while t 2^-b is a normal number
    const bool plain = (t != 0.0f) && !(t >= 1.17549435e-38f * two_b && t <= 3.402823466e38f);
    const QuConst qc = {t, t * inv_two_b, two_b, inv_two_b * (1.0f / 65536.0f), -127.0f * inv_two_b, __float_as_uint(inv_two_b)};
    double ss_theta = 0.0, ss_u = 0.0;
    const int64_t e0 = q.eQ;
    const bool staged = q.nQ > 0;                  // the whole tile lies inside the layer and its rows were fetched ahead
    if (e0 < hi) {
        const bool full = (e0 >= lo && e0 + 8 <= hi);
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
        if (staged) {
#pragma unroll 1
            for (int i = 0; i < M; ++i) {
                float v[8];
                p_take(q.nN + i, v);
                if (!plain) {                       // nearly always
                    uint32_t w[8];
                    p_words8<RNG16>(a, e0, (uint32_t)i, w);
                    p_levels8<RNG16>(v, w, qc, acc);
                }
                p_issue(a, q, q.nN + i + DAT_P_DEPTH);
            }
        }
        if (MODE == P_MODE_IDENTITY) {
#pragma unroll 2
            for (int i = 0; i < M; ++i) {           // Q is the identity: the ordered fp32 sum of the workers' gradients
                float v[8];
                dat_load4(a.gp.p[i], e0, lo, hi, v);
                dat_load4(a.gp.p[i], e0 + 4, lo, hi, v + 4);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] += v[j];
            }
        } else if (staged && !plain) { }
        else if (full && !plain) qu_rows<RNG16, true, false>(a.gp, a.keys, qc, M, e0, lo, hi, acc);
        else if (full) qu_rows<RNG16, true, true>(a.gp, a.keys, qc, M, e0, lo, hi, acc);
        else if (!plain) qu_rows<RNG16, false, false>(a.gp, a.keys, qc, M, e0, lo, hi, acc);
        else qu_rows<RNG16, false, true>(a.gp, a.keys, qc, M, e0, lo, hi, acc);
        float th[8], m[8];
        if (staged) {
            p_take(q.nN + M, th);
            p_issue(a, q, q.nN + M + DAT_P_DEPTH);
            p_take(q.nN + M + 1, m);
            p_issue(a, q, q.nN + M + 1 + DAT_P_DEPTH);
        } else {
            p_load4_cg(a.theta, e0, lo, hi, th);
            p_load4_cg(a.theta, e0 + 4, lo, hi, th + 4);
            p_load4_cg(a.mom, e0, lo, hi, m);
            p_load4_cg(a.mom, e0 + 4, lo, hi, m + 4);
        }
        if (MODE != P_MODE_IDENTITY && a.code_sum) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (e0 + j >= lo && e0 + j < hi) a.code_sum[e0 + j] = (int)acc[j];
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float ghat = (MODE == P_MODE_IDENTITY) ? acc[j] / a.M_f : acc[j] * f;
            m[j] = __fmaf_rn(a.mu, m[j], __fmaf_rn(a.wd, th[j], ghat));
            ss_theta = fma((double)th[j], (double)th[j], ss_theta);
            ss_u = fma((double)m[j], (double)m[j], ss_u);
        }
        dat_store4(a.mom, e0, lo, hi, m);
        dat_store4(a.mom, e0 + 4, lo, hi, m + 4);
    }
    __threadfence();                               // m' is read by the U part of another CTA
    const double x = dat_block_sum(ss_theta, scratch);
    const double y = dat_block_sum(ss_u, scratch);
    if (threadIdx.x == 0) {
        a.partQ[2 * (pt.tb + pt.tile)] = x;
        a.partQ[2 * (pt.tb + pt.tile) + 1] = y;
        __threadfence();
    }
    if (p_arrive(a.cntQ + layer, (uint32_t)pt.T, s_flag)) p_finish_update_sums(a, layer, pt.tb, (uint32_t)pt.T, scratch);
}

// ---- U: theta' = theta - a_l m' (Eq. 3, pass 2) of one tile ---------------------------------------
__device__ __forceinline__ void p_part_update(const PArgs &a, const PipePart &pt, const Seq &q)
{
    const int64_t lo = pt.lo, hi = pt.hi;
    const float na = -__ldcg(a.step_a + pt.layer);
    const int64_t e0 = q.eU;
    if (e0 >= hi) return;
    float th[8], m[8];
    if (q.nU > 0) {
        p_take(q.nN + q.nQ, th);
        p_issue(a, q, q.nN + q.nQ + DAT_P_DEPTH);
        p_take(q.nN + q.nQ + 1, m);
        p_issue(a, q, q.nN + q.nQ + 1 + DAT_P_DEPTH);
    } else {
        p_load4_cg(a.theta, e0, lo, hi, th);
        p_load4_cg(a.theta, e0 + 4, lo, hi, th + 4);
        p_load4_cg(a.mom, e0, lo, hi, m);
        p_load4_cg(a.mom, e0 + 4, lo, hi, m + 4);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) th[j] = __fmaf_rn(na, m[j], th[j]);
    if (e0 >= lo && e0 + 8 <= hi) {
        const uint64_t pol_first = q.pol_first;
        dat_st4_hint(a.theta + e0, make_float4(th[0], th[1], th[2], th[3]), pol_first);
        dat_st4_hint(a.theta + e0 + 4, make_float4(th[4], th[5], th[6], th[7]), pol_first);
    } else {
        dat_store4(a.theta, e0, lo, hi, th);
        dat_store4(a.theta, e0 + 4, lo, hi, th + 4);
    }
}

__device__ __forceinline__ bool p_tile_inside(const PipePart &pt)
{
    const int64_t begin = (pt.lo & ~(int64_t)7) + (int64_t)pt.tile * DAT_P_TILE;
    return begin >= pt.lo && begin + DAT_P_TILE <= pt.hi;
}

template <bool RNG16, int MODE>
__global__ void __launch_bounds__(DAT_P_THREADS, DAT_P_MINB)
k_step_pipelined(const __grid_constant__ PArgs a)
{
    __shared__ double s_unit[4 * DAT_MAX_WORKERS];
    __shared__ float s_norm[DAT_MAX_WORKERS];
    __shared__ __align__(16) PipeItem s_item;
    __shared__ int s_flag;
    __shared__ int s_seen[2];                      // the layers this item waits for were already published when it started
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
        if (lane < (int)(sizeof(PipeItem) / 16))
            reinterpret_cast<uint4 *>(&s_item)[lane] = __ldg(reinterpret_cast<const uint4 *>(a.items + tk) + lane);
    }
    for (int u = threadIdx.x; u < 4 * a.M; u += DAT_P_THREADS) s_unit[u] = 0.0;
    __syncthreads();
    const PipePart pn = s_item.n, pq = s_item.q, pu = s_item.u;
#ifdef DAT_SELFCHECK
    {
        bool ok = pn.layer < a.h && pq.layer < a.h && pu.layer < a.h;
        const PipePart *pp[3] = {&pn, &pq, &pu};
        for (int k = 0; k < 3 && ok; ++k)
            if (pp[k]->layer >= 0)
                ok = pp[k]->tile >= 0 && pp[k]->tile < pp[k]->T && (int64_t)pp[k]->tb + pp[k]->tile < a.n_tiles &&
                     pp[k]->lo >= 0 && pp[k]->lo < pp[k]->hi && pp[k]->hi <= a.d;
        if (!P_CHECK(a, ok)) return;
    }
#endif
    // what the other two parts wait for: look now, so that the answer is there when it is needed
    if (threadIdx.x < 2) {
        const bool want = (threadIdx.x == 0) ? (pq.layer >= 0 && MODE != P_MODE_IDENTITY) : (pu.layer >= 0);
        const uint32_t *word = (threadIdx.x == 0) ? a.readyN + pq.layer : a.readyQ + pu.layer;
        s_seen[threadIdx.x] = want ? (p_ld_acquire(word) == a.epoch) : 1;
    }
    // the thread's sequence of entries
    Seq q;
    q.pol_last = DAT_P_N_POLICY();
    q.pol_first = dat_policy_evict_first();
    q.pol_normal = dat_policy_evict_normal();
    q.u0 = warp * (4 * a.M) / 8;
    q.nN = (pn.layer >= 0 && p_tile_inside(pn)) ? 2 * ((warp + 1) * (4 * a.M) / 8 - q.u0) : 0;
    q.nQ = (pq.layer >= 0 && MODE != P_MODE_IDENTITY && p_tile_inside(pq)) ? a.M + 2 : 0;
    q.nU = 0;                                      // known once s_seen[1] is
    q.eN = (pn.lo & ~(int64_t)7) + (int64_t)pn.tile * DAT_P_TILE + 4 * lane;
    q.eQ = (pq.lo & ~(int64_t)7) + (int64_t)pq.tile * DAT_P_TILE + 8 * (int64_t)threadIdx.x;
    q.eU = (pu.lo & ~(int64_t)7) + (int64_t)pu.tile * DAT_P_TILE + 8 * (int64_t)threadIdx.x;
    // DEPTH entries ahead; the first DEPTH entries never reach the U part unless N and Q are both absent or short,
    // in which case U is fetched the plain way
#pragma unroll
    for (int j = 0; j < DAT_P_DEPTH; ++j) p_issue(a, q, j);

    if (pn.layer >= 0) p_norm_sums(a, pn, q, s_unit);
    __syncthreads();                               // s_seen is there (and every warp's unit sums)
    // m' of the U tile may be fetched ahead only if its layer was seen published (then it is visible)
    if (pu.layer >= 0 && s_seen[1] && p_tile_inside(pu) && q.nQ >= DAT_P_DEPTH) q.nU = 2;    // (its entries have not been passed yet)
    if (pn.layer >= 0) p_norm_publish(a, pn, s_unit, s_norm, &s_flag);
    bool alive = true;
    if (pq.layer >= 0) {
        alive = (MODE == P_MODE_IDENTITY) || s_seen[0] || p_wait(a, a.readyN + pq.layer, &s_flag);
        if (alive) p_part_quant<RNG16, MODE>(a, pq, q, s_unit, &s_flag);
    }
    if (alive && pu.layer >= 0) {
        alive = s_seen[1] || p_wait(a, a.readyQ + pu.layer, &s_flag);
        if (alive) p_part_update(a, pu, q);
    }
    p_cp_wait<0>();
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
        // slot of every tile in each of the three streams
        std::vector<PipeItem> items;
        const PipePart nopart = {0, 1, 0, 1, -1, 0};
        const PipeItem none = {nopart, nopart, nopart};
        auto part = [&](int l, int64_t t) {
            PipePart pp = {plan->offsets[l], plan->offsets[l + 1], (int32_t)tb[l], (int32_t)(tb[l + 1] - tb[l]), l, (int32_t)t};
            return pp;
        };
        auto at = [&](int64_t slot) -> PipeItem & {
            if ((int64_t)items.size() <= slot) items.resize((size_t)slot + 1, none);
            return items[(size_t)slot];
        };
        std::vector<int64_t> done_n((size_t)h, -1 - (int64_t)DAT_P_LAG), done_q((size_t)h, 0);
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
            // tile (what N read last is read first); the others in N's order, every tile at the same distance
            const bool reverse = T >= DAT_P_REVERSE_FROM;
            for (int64_t t = 0; t < T; ++t) { at(slot).q = part(l, reverse ? T - 1 - t : t); done_q[l] = slot++; }
        }
        slot = 0;
        for (int k = 0; k < h; ++k) {
            const int l = order[k];
            slot = std::max(slot, done_q[l] + DAT_P_LAG + 1);
            for (int64_t t = 0; t < tb[l + 1] - tb[l]; ++t) { at(slot).u = part(l, t); ++slot; }
        }
        g->n_items = (int64_t)items.size();

        size_t off = 0;
        auto take = [&](size_t bytes) { size_t o = off; off = p_align(off + bytes); return o; };
        const size_t o_items = take(items.size() * sizeof(PipeItem)), o_tb = take(((size_t)h + 1) * 8);
        const size_t o_pn = take((size_t)nt * (size_t)M * 8), o_pq = take((size_t)nt * 16);
        g->sync_bytes = (2 + 4 * (size_t)h) * 4;
        const size_t o_sync = take(g->sync_bytes);
        g->mem_bytes = off;
        cudaError_t e = cudaFuncSetAttribute(k_step_pipelined<true, P_MODE_IDENTITY>, cudaFuncAttributeMaxDynamicSharedMemorySize, DAT_P_STAGE_BYTES);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_step_pipelined<true, P_MODE_SHARED>, cudaFuncAttributeMaxDynamicSharedMemorySize, DAT_P_STAGE_BYTES);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_step_pipelined<false, P_MODE_SHARED>, cudaFuncAttributeMaxDynamicSharedMemorySize, DAT_P_STAGE_BYTES);
        if (e != cudaSuccess) return dat_cuda_fail(plan, e);
        e = cudaMalloc((void **)&g->mem, off);
        if (e != cudaSuccess) { g->mem = nullptr; plan->last_cuda = (int)e; (void)cudaGetLastError(); return DAT_ERR_NOMEM; }
        g->d_items = (PipeItem *)(g->mem + o_items);
        g->d_tile_base = (int64_t *)(g->mem + o_tb);
        g->d_partN = (double *)(g->mem + o_pn);
        g->d_partQ = (double *)(g->mem + o_pq);
        g->d_sync = (uint32_t *)(g->mem + o_sync);
        e = cudaMemset(g->mem, 0, off);
        if (e == cudaSuccess) e = cudaMemcpy(g->d_items, items.data(), items.size() * sizeof(PipeItem), cudaMemcpyHostToDevice);
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

extern "C" int dat_step_pipelined(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                                  uint64_t seed, uint64_t step, const dat_hparams_t *hp,
                                  int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !hp) return DAT_ERR_ARG;
    if (plan->bits != 32 && plan->scale_mode != DAT_SCALE_SHARED_MAX) return DAT_ERR_UNSUPPORTED;
    if (step >> 32) return DAT_ERR_ARG;
    if (!dat_aligned16(theta) || !dat_aligned16(mom) || (code_sum_out && !dat_aligned16(code_sum_out)) ||
        (layer_norms_out && !dat_aligned16(layer_norms_out)) || (scales_out && !dat_aligned16(scales_out)))
        return DAT_ERR_ALIGN;
    PArgs a;
    rc = dat_check_grads(plan, grads, &a.gp);
    if (rc != DAT_OK) return rc;
    PipeSchedule *g = plan->pipe;
    if (!g || !g->mem) return DAT_ERR_ARG;
    const bool identity = (plan->bits == 32);
    const size_t h = (size_t)plan->h;
    a.keys = dat_make_keys(seed, step);
    a.items = g->d_items;
    a.off = plan->d_offsets;
    a.tile_base = g->d_tile_base;
    a.theta = theta;
    a.mom = mom;
    a.partN = g->d_partN;
    a.partQ = g->d_partQ;
    a.ticket = g->d_sync;
    a.abort_epoch = g->d_sync + 1;
    a.cntN = g->d_sync + 2;
    a.cntQ = a.cntN + h;
    a.readyN = a.cntQ + h;
    a.readyQ = a.readyN + h;
    a.status = plan->d_status;
    a.worker_norms = plan->d_worker_norms;
    a.scales = plan->d_scales;
    a.qmul = plan->d_qmul;
    a.dq = plan->d_dq;
    a.step_a = plan->d_step_a;
    a.norms_out = layer_norms_out;
    a.scales_out = identity ? nullptr : scales_out;
    a.code_sum = identity ? nullptr : code_sum_out;
    a.wait_cycles = g->wait_cycles;
    a.S_f = (float)plan->S;
    a.SM_f = (float)((uint64_t)plan->S * (uint64_t)plan->M);
    a.M_f = (float)plan->M;
    a.mu = hp->momentum;
    a.wd = hp->weight_decay;
    a.lr = hp->lr;
    a.c_l = hp->c_l;
    a.c_u = hp->c_u;
    if (++g->epoch == 0u) ++g->epoch;              // 0 is what the words hold before the first call
    a.epoch = g->epoch;
    a.n_items = (uint32_t)g->n_items;
    a.M = plan->M;
    a.h = (int)plan->h;
    a.d = plan->d;
    a.n_tiles = g->n_tiles;
    cudaStream_t s = (cudaStream_t)stream;
    const unsigned grid = (unsigned)g->n_items;
    if (identity) k_step_pipelined<true, P_MODE_IDENTITY><<<grid, DAT_P_THREADS, DAT_P_STAGE_BYTES, s>>>(a);
    else if (plan->rng_bits == 16) k_step_pipelined<true, P_MODE_SHARED><<<grid, DAT_P_THREADS, DAT_P_STAGE_BYTES, s>>>(a);
    else k_step_pipelined<false, P_MODE_SHARED><<<grid, DAT_P_THREADS, DAT_P_STAGE_BYTES, s>>>(a);
    DAT_LAUNCHED(plan);
    return DAT_OK;
}
