// dat_step: Steps 7, 9 and 12 of Algorithm A1 in ONE persistent, warp-specialised kernel.
//
// The flat vector is cut into per-layer tiles of FT elements.  Every tile passes through three
// stages of work, each a work item:
//   N  read the M gradient tiles, fp64 sums of squares per worker.  When a layer's last
//      contribution has arrived, nu_l, S/nu_l and nu_l/(S*M) are published  [||g||_2 of Eq. rand_q]
//   Q  (needs nu_l) re-read the gradient tiles -- by construction still in L2 for layers that
//      fit -- draw the stochastic levels (Eq. xi), sum the signed codes over the workers and
//      scale (Eq. grad_agg), form m' = mu*m + g_hat + wd*theta, store m', fp64 sums of theta^2
//      and m'^2.  When a layer is complete, a_l = lr*tau(||theta_l||)/||u_l|| is published [Eq. 3]
//   U  (needs a_l) theta -= a_l * m'                                                    [Eq. 3]
//
// The host lays the items out as a software pipeline: the N items of one window of layers are
// interleaved with the Q items of the previous window and the U items of the one before, so
// that HBM streaming (N) overlaps the L2- and ALU-bound work (Q, U) and a layer's dependency
// is normally met long before its consumers are reached.  CTA c (one per SM) executes items
// c, c+G, c+2G, ... in order.  Inside a CTA one producer warp walks the list ahead of the
// consumers and moves every tile into a ring of shared-memory stages with bulk asynchronous
// copies (cp.async.bulk, completion counted on an mbarrier; no multicast); eight consumer
// warps take the stages in order.  Tiles that touch a layer boundary or are not full are read
// with ordinary masked loads instead.
//
// An item depends only on items earlier in the list and all CTAs are co-resident (cooperative
// launch), so the list cannot deadlock.  Every wait -- on an mbarrier, on a layer flag -- is
// bounded all the same: when one runs out the thread sets DAT_STATUS_TIMEOUT and the CTA's abort
// flag, every other waiter sees it and leaves, the producer waits (bounded) for its copies in
// flight, and the kernel returns; the last CTA out clears the dependency counters.
#include <algorithm>
#include <new>

#include "dat_internal.cuh"

#define FT 1024                                  // elements per fused tile
#define F_CW 8                                   // consumer warps
#define F_CT (F_CW * 32)                         // consumer threads; thread t owns elements 4t..4t+3
#define F_THREADS (F_CT + 64)                    // + one producer warp + one reducer warp
#define F_ROWS 4                                 // worker rows per stage
#define F_STAGES 4
#define F_RED 2                                  // reduction hand-off buffers
#define F_CTAS_PER_SM 2
#define F_STAGE_FLOATS ((F_ROWS + 2) * FT)       // gradient rows + theta row + momentum row
#define F_STAGE_BYTES (F_STAGE_FLOATS * 4)
#define F_WAIT_CYCLES (1ll << 31)                // bound of every device-side wait (about a second)

enum { ITEM_N = 0u, ITEM_Q = 1u, ITEM_U = 2u, ITEM_END = 3u };
#define ITEM_FLUSH 0x20000000u                   // the CTA's last item of this kind in the layer
#define ITEM_TILE_MASK 0x1FFFFFFFu

struct FusedSchedule {
    uint32_t *d_items = nullptr;
    int64_t n_items = 0;
    int64_t *d_tile_base = nullptr;   // h+1, tiles of FT elements
    int64_t *d_slot_base = nullptr;   // h+1, partial-sum slots per layer
    uint32_t *d_expect = nullptr;     // 2h: contributions expected per layer (N, Q)
    uint32_t *d_sync = nullptr;       // cnt_n[h] cnt_q[h] flag_n[h] flag_q[h] done[1]
    double *d_npart = nullptr;        // slots * M
    double *d_qpart = nullptr;        // slots * 2
    size_t sync_words = 0;
    uint32_t epoch = 0;
    int grid = 0;
    int64_t window_bytes = 0;
    size_t smem_bytes = 0;
};

struct FusedArgs {
    GradPtrs gp;
    PhiloxKeys keys;
    float *theta, *mom;
    const int64_t *off, *tile_base, *slot_base;
    const uint32_t *items, *expect;
    int64_t n_items;
    double *npart, *qpart;
    uint32_t *cnt_n, *cnt_q, *flag_n, *flag_q, *done, *status;
    float *worker_norms, *scales, *qmul, *dq, *step_a;
    int32_t *code_sum;
    float *norms_out, *scales_out;
    int h, M;
    uint32_t epoch;
    float S_f, SM_f, lr, mu, wd, c_l, c_u;
#ifdef DAT_PROF
    unsigned long long *prof;                    // development builds only
#endif
};

// What a stage holds: written by the producer (four 16-byte stores), read by every consumer thread.
struct __align__(16) StageHdr {
    uint32_t kind;                               // ITEM_*
    uint32_t flags;                              // HDR_*
    int layer;
    int chunk;                                   // which group of F_ROWS workers
    long long begin, lo;                         // first element of the tile; the layer's bounds [lo, hi)
    long long hi, slot;                          // slot: where the CTA's running sums go on a flush
    float f0, f1;                                // Q: S/nu_l and nu_l/(S*M);  U: -a_l
    int pad[2];
};
enum { HDR_FAST = 1u, HDR_FLUSH = 2u, HDR_LAST_CHUNK = 4u };

// What the consumers hand to the reducer warp with a buffer of per-warp partial sums.
struct RedDesc {
    uint32_t kind;                               // ITEM_N, ITEM_Q or ITEM_END
    uint32_t flush;
    int layer;
    long long slot;
};

#ifdef DAT_PROF
#define PROF_T0() const long long prof_t0 = clock64()
#define PROF_ADD(k) do { if (a.prof && (threadIdx.x & 31) == 0 && (threadIdx.x == 0 || threadIdx.x >= F_CT)) a.prof[blockIdx.x * 16 + (k)] += (unsigned long long)(clock64() - prof_t0); } while (0)
#define PROF_TRACE(role, idx, col, val) do { if (a.prof && blockIdx.x == 0 && (threadIdx.x & 31) == 0 && (idx) < 4096) a.prof[296 * 16 + ((role) * 4096 + (idx)) * 8 + (col)] = (unsigned long long)(val); } while (0)
#else
#define PROF_TRACE(role, idx, col, val) do {} while (0)
#define PROF_T0() do {} while (0)
#define PROF_ADD(k) do {} while (0)
#endif

struct Shared {
    unsigned long long full[F_STAGES], empty[F_STAGES];
    unsigned long long red_full[F_RED], red_empty[F_RED];
    StageHdr hdr[F_STAGES];
    RedDesc rdesc[F_RED];
    double red[F_RED][F_CW][DAT_MAX_WORKERS];    // per-warp partial sums handed to the reducer
    double acc_n[DAT_MAX_WORKERS];               // the CTA's running sums for its current layer (reducer)
    double acc_q[2];
    int abort_flag;
};

// ---- PTX wrappers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, uint32_t bytes)
{
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// global -> shared bulk copy; completion (in bytes) is counted on `bar`.  16-byte aligned
// addresses, size a multiple of 16.  The destination is this CTA's own shared memory.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, unsigned long long *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
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

// ---- bounded waits ------------------------------------------------------------------------------
__device__ __forceinline__ void raise_timeout(Shared &sh, uint32_t *status)
{
    atomicOr(status, DAT_STATUS_TIMEOUT);
    atomicExch(&sh.abort_flag, 1);
}

__device__ __forceinline__ bool wait_mbar(Shared &sh, unsigned long long *bar, uint32_t parity, uint32_t *status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spins & 63u) == 0u) {
            if (*(volatile int *)&sh.abort_flag) return false;
            if (clock64() - t0 > F_WAIT_CYCLES) break;
        }
    }
    raise_timeout(sh, status);
    return false;
}

__device__ __forceinline__ bool wait_flag(Shared &sh, const uint32_t *flag, uint32_t epoch, uint32_t *status)
{
    if (ld_acquire(flag) == epoch) return true;
    const long long t0 = clock64();
    for (uint32_t spins = 1;; ++spins) {
        __nanosleep(32);
        if (ld_acquire(flag) == epoch) return true;
        if ((spins & 15u) == 0u) {
            if (*(volatile int *)&sh.abort_flag || (ld_acquire(status) & DAT_STATUS_TIMEOUT)) {
                atomicExch(&sh.abort_flag, 1);
                return false;
            }
            if (clock64() - t0 > F_WAIT_CYCLES) break;
        }
    }
    raise_timeout(sh, status);
    return false;
}

// ---- producer warp -------------------------------------------------------------------------------
// The layer a kind of item is working in (items of one kind come in layer order), with what
// the producer has already learnt about it.
struct LayerCursor {
    int layer = -1;
    long long t0 = 0, t1 = 0, lo = 0, hi = 0;
    long long first_tile = -1;                   // the CTA's first tile of its running sums in this layer
    bool flag_seen = false;
    float f0 = 0.0f, f1 = 0.0f;
};

__device__ __forceinline__ void cursor_seek(const FusedArgs &a, LayerCursor &c, long long tile)
{
    if (c.layer >= 0 && tile >= c.t0 && tile < c.t1) return;
    c.layer = dat_find(a.tile_base, a.h, tile);
    c.t0 = __ldg(a.tile_base + c.layer);
    c.t1 = __ldg(a.tile_base + c.layer + 1);
    c.lo = __ldg(a.off + c.layer);
    c.hi = __ldg(a.off + c.layer + 1);
    c.flag_seen = false;
}

// All 32 lanes walk the CTA's item list together (warp-uniform control flow).  Per stage: wait
// until the slot is free, announce the bytes, start the copies (lane r moves row r), write the
// stage header, arrive.  Layer flags are waited for here, ahead of the consumers; a flag already
// seen is not read again.  Returns the number of stages issued.
template <bool IDENTITY>
__device__ __forceinline__ uint32_t producer(const FusedArgs &a, Shared &sh, float *stages)
{
    const int lane = threadIdx.x & 31;
    LayerCursor cn, cq, cu;
    uint32_t issued = 0;
    const int nchunks = (a.M + F_ROWS - 1) / F_ROWS;
    const long long G = gridDim.x;
    uint32_t next_item = (blockIdx.x < a.n_items) ? __ldg(a.items + blockIdx.x) : 0u;
    for (long long it = blockIdx.x; it < a.n_items; it += G) {
        const uint32_t item = next_item;
        if (it + G < a.n_items) next_item = __ldg(a.items + it + G);
        const uint32_t type = item >> 30;
        const long long tile = item & ITEM_TILE_MASK;
        LayerCursor cur = (type == ITEM_N) ? cn : (type == ITEM_Q) ? cq : cu;     // by value: stays in registers
        cursor_seek(a, cur, tile);
        const long long begin = (cur.lo & ~3ll) + (tile - cur.t0) * FT;
        const bool fast = (begin >= cur.lo) && (begin + FT <= cur.hi);
        long long slot_idx = 0;
        if (type != ITEM_U) {
            if (cur.first_tile < 0) cur.first_tile = tile;
            const long long nt = cur.t1 - cur.t0;
            slot_idx = __ldg(a.slot_base + cur.layer) + ((nt <= G) ? (cur.first_tile - cur.t0) : (long long)blockIdx.x);
            if (item & ITEM_FLUSH) cur.first_tile = -1;
        }
        if (type == ITEM_U && !cur.flag_seen) {
            // m' of this tile was written by the tile's Q item: the layer's flag orders it
            { PROF_T0();
            if (!wait_flag(sh, a.flag_q + cur.layer, a.epoch, a.status)) return issued;
            PROF_ADD(7); }
            cur.f0 = -__ldcg(a.step_a + cur.layer);
            cur.flag_seen = true;
            asm volatile("fence.proxy.async;" ::: "memory");
        }
        const int nst = (type == ITEM_U) ? 1 : nchunks;
        for (int c = 0; c < nst; ++c) {
            const uint32_t slot = issued % F_STAGES, use = issued / F_STAGES;
            PROF_TRACE(1, issued, 0, clock64());
            { PROF_T0();
            if (!wait_mbar(sh, &sh.empty[slot], (use & 1u) ^ 1u, a.status)) return issued;
            PROF_ADD(6); }
            PROF_TRACE(1, issued, 1, clock64());
            PROF_TRACE(1, issued, 2, type | ((unsigned long long)cur.layer << 16));
            PROF_T0();
            float *st = stages + (size_t)slot * F_STAGE_FLOATS;
            if (fast) {
                const bool params = (type == ITEM_U) || (type == ITEM_Q && c == nst - 1);   // theta and m rows
                const int rows = (type == ITEM_U) ? 0 : min(F_ROWS, a.M - c * F_ROWS);
                if (lane == 0) mbar_expect_tx(&sh.full[slot], (uint32_t)(rows + (params ? 2 : 0)) * (FT * 4));
                __syncwarp();
                PROF_TRACE(1, issued, 4, clock64());
                if (lane < rows) bulk_g2s(st + lane * FT, a.gp.p[c * F_ROWS + lane] + begin, FT * 4, &sh.full[slot]);
                if (params && lane == F_ROWS) bulk_g2s(st + F_ROWS * FT, a.theta + begin, FT * 4, &sh.full[slot]);
                if (params && lane == F_ROWS + 1) bulk_g2s(st + (F_ROWS + 1) * FT, a.mom + begin, FT * 4, &sh.full[slot]);
            }
            PROF_TRACE(1, issued, 5, clock64());
            issued++;
            if (type == ITEM_Q && !IDENTITY && !cur.flag_seen) {
                // every copy announced above has been started, so the stage completes even if
                // this wait gives up
                PROF_T0();
                if (!wait_flag(sh, a.flag_n + cur.layer, a.epoch, a.status)) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.full[slot]);
                    return issued;
                }
                PROF_ADD(7);
                cur.f0 = __ldcg(a.qmul + cur.layer);
                cur.f1 = __ldcg(a.dq + cur.layer);
                cur.flag_seen = true;
            }
            if (lane == 0) {
                uint4 *H = reinterpret_cast<uint4 *>(&sh.hdr[slot]);
                const uint32_t flags = (fast ? HDR_FAST : 0u) | ((item & ITEM_FLUSH) ? HDR_FLUSH : 0u) |
                                       ((c == nst - 1) ? HDR_LAST_CHUNK : 0u);
                H[0] = make_uint4(type, flags, (uint32_t)cur.layer, (uint32_t)c);
                H[1] = make_uint4((uint32_t)begin, (uint32_t)(begin >> 32), (uint32_t)cur.lo, (uint32_t)(cur.lo >> 32));
                H[2] = make_uint4((uint32_t)cur.hi, (uint32_t)(cur.hi >> 32), (uint32_t)slot_idx, (uint32_t)(slot_idx >> 32));
                H[3] = make_uint4(__float_as_uint(cur.f0), __float_as_uint(cur.f1), 0u, 0u);
            }
            PROF_TRACE(1, issued - 1, 6, clock64());
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.full[slot]);      // release: the header is visible once the stage completes
            PROF_ADD(8);
            PROF_TRACE(1, issued - 1, 3, clock64());
        }
        if (type == ITEM_N) cn = cur; else if (type == ITEM_Q) cq = cur; else cu = cur;
    }
    {   // end marker
        const uint32_t slot = issued % F_STAGES, use = issued / F_STAGES;
        if (!wait_mbar(sh, &sh.empty[slot], (use & 1u) ^ 1u, a.status)) return issued;
        if (lane == 0) sh.hdr[slot].kind = ITEM_END;
        issued++;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.full[slot]);
    }
    return issued;
}

// ---- reducer warp ----------------------------------------------------------------------------------
// Takes the consumers' per-warp sums of an item, folds them into the CTA's running sums of the
// layer and, on a flush item, publishes those to global memory.  The CTA whose contribution
// completes a layer reduces all contributions in a fixed order and publishes the layer's scale
// (N) or step length (Q) behind a release flag.  All of this costs several global round trips;
// keeping it in a warp of its own keeps them off the consumers' path.
__device__ __forceinline__ void finish_norm(const FusedArgs &a, Shared &sh, int layer, long long slot, int buf,
                                            bool flush, int lane)
{
    for (int i = lane; i < a.M; i += 32) {
        double s = sh.acc_n[i];
#pragma unroll
        for (int w = 0; w < F_CW; ++w) s += sh.red[buf][w][i];
        sh.acc_n[i] = s;
    }
    __syncwarp();
    if (!flush) return;
    for (int i = lane; i < a.M; i += 32) { a.npart[slot * a.M + i] = sh.acc_n[i]; sh.acc_n[i] = 0.0; }
    __threadfence();
    __syncwarp();
    uint32_t last = 0;
    if (lane == 0) {
        const uint32_t old = atomicAdd(a.cnt_n + layer, 1u);
        last = (old == __ldg(a.expect + layer) - 1u);
        if (last) { a.cnt_n[layer] = 0u; __threadfence(); }
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    const long long s0 = __ldg(a.slot_base + layer);
    const int ns = (int)(__ldg(a.slot_base + layer + 1) - s0);
    float nu = 0.0f;
    bool bad = false;
    for (int i = 0; i < a.M; ++i) {
        double acc = 0.0;
        for (int s = lane; s < ns; s += 32) acc += __ldcg(a.npart + (s0 + s) * a.M + i);
        acc = dat_warp_sum(acc);
        const float nrm = (float)sqrt(acc);
        if (lane == 0) a.worker_norms[(long long)i * a.h + layer] = nrm;
        bad |= !isfinite(nrm);
        nu = (i == 0 || nrm > nu) ? nrm : nu;
    }
    if (lane == 0) {
        a.scales[layer] = nu;
        a.qmul[layer] = (nu == 0.0f) ? 0.0f : a.S_f / nu;
        a.dq[layer] = (nu == 0.0f) ? 0.0f : nu / a.SM_f;
        if (a.scales_out) a.scales_out[layer] = nu;
        if (bad) atomicOr(a.status, DAT_STATUS_NONFINITE);
        st_release(a.flag_n + layer, a.epoch);
    }
}

__device__ __forceinline__ void finish_quant(const FusedArgs &a, Shared &sh, int layer, long long slot, int buf,
                                             bool flush, int lane)
{
    if (lane < 2) {
        double s = sh.acc_q[lane];
#pragma unroll
        for (int w = 0; w < F_CW; ++w) s += sh.red[buf][w][lane];
        sh.acc_q[lane] = s;
    }
    __syncwarp();
    if (!flush) return;
    if (lane < 2) { a.qpart[slot * 2 + lane] = sh.acc_q[lane]; sh.acc_q[lane] = 0.0; }
    __threadfence();
    __syncwarp();
    uint32_t last = 0;
    if (lane == 0) {
        const uint32_t old = atomicAdd(a.cnt_q + layer, 1u);
        last = (old == __ldg(a.expect + a.h + layer) - 1u);
        if (last) { a.cnt_q[layer] = 0u; __threadfence(); }
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    const long long s0 = __ldg(a.slot_base + layer);
    const int ns = (int)(__ldg(a.slot_base + layer + 1) - s0);
    double x = 0.0, y = 0.0;
    for (int s = lane; s < ns; s += 32) { x += __ldcg(a.qpart + (s0 + s) * 2); y += __ldcg(a.qpart + (s0 + s) * 2 + 1); }
    x = dat_warp_sum(x);
    y = dat_warp_sum(y);
    if (lane == 0) {
        const float n_theta = (float)sqrt(x), n_u = (float)sqrt(y);
        const float tau = fminf(fmaxf(n_theta, a.c_l), a.c_u);
        const float ratio = (n_u == 0.0f) ? 0.0f : tau / n_u;
        a.step_a[layer] = a.lr * ratio;
        if (a.norms_out) { a.norms_out[2 * layer] = n_theta; a.norms_out[2 * layer + 1] = n_u; }
        if (!isfinite(n_theta) || !isfinite(n_u)) atomicOr(a.status, DAT_STATUS_NONFINITE);
        st_release(a.flag_q + layer, a.epoch);
    }
}

__device__ __forceinline__ void reducer(const FusedArgs &a, Shared &sh)
{
    const int lane = threadIdx.x & 31;
    for (uint32_t k = 0;; ++k) {
        const uint32_t b = k % F_RED, use = k / F_RED;
        if (!wait_mbar(sh, &sh.red_full[b], use & 1u, a.status)) return;
        const uint32_t kind = sh.rdesc[b].kind;
        if (kind == ITEM_END) return;
        PROF_T0();
        const bool flush = sh.rdesc[b].flush != 0;
        const int layer = sh.rdesc[b].layer;
        const long long slot = sh.rdesc[b].slot;
        if (kind == ITEM_N) finish_norm(a, sh, layer, slot, (int)b, flush, lane);
        else finish_quant(a, sh, layer, slot, (int)b, flush, lane);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.red_empty[b]);
        PROF_ADD(5);
    }
}

// ---- consumer warps -----------------------------------------------------------------------------------
// Cross-lane sum of F_ROWS (= 4) per-lane values: after the call, lanes with (lane & 7) == 0 hold
// the warp total of value number (lane >> 3).  Fixed order: 2 exchange-and-halve steps, 3 plain.
__device__ __forceinline__ double warp_sum_rows(double v[F_ROWS], int lane)
{
    static_assert(F_ROWS == 4, "warp_sum_rows is written for four rows");
    {
        const bool up = lane & 16;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const double send = up ? v[k] : v[k + 2], keep = up ? v[k + 2] : v[k];
            v[k] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 16);
        }
    }
    {
        const bool up = lane & 8;
        const double send = up ? v[0] : v[1], keep = up ? v[1] : v[0];
        v[0] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
    }
    v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 4);
    v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 2);
    v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 1);
    return v[0];
}

// The four elements of consumer thread `ct` in one row of a tile: from the stage (bulk-copied
// tiles) or, masked, from global memory (tiles at a layer boundary).
template <bool FAST>
__device__ __forceinline__ void load_group(const float *stage_row, const float *global_row, long long e0,
                                           long long lo, long long hi, int ct, float v[4])
{
    if (FAST) {
        const float4 f = *reinterpret_cast<const float4 *>(stage_row + 4 * ct);
        v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
    } else {
        dat_load4(global_row, e0, lo, hi, v);
    }
}

template <bool FAST, bool FULL>
__device__ __forceinline__ void rows_sumsq(const FusedArgs &a, const float *st, int chunk, int rows, long long e0,
                                           long long lo, long long hi, int ct, double acc[F_ROWS])
{
#pragma unroll
    for (int r = 0; r < F_ROWS; ++r) {
        acc[r] = 0.0;
        if (FULL || r < rows) {
            float v[4];
            load_group<FAST>(st + r * FT, a.gp.p[chunk * F_ROWS + r], e0, lo, hi, ct, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[r] = fma((double)v[j], (double)v[j], acc[r]);
        }
    }
}

template <bool IDENTITY, bool FAST, bool FULL>
__device__ __forceinline__ void rows_quant(const FusedArgs &a, const float *st, int chunk, int rows, long long e0,
                                           long long lo, long long hi, int ct, float qmul, int sum[4], float facc[4])
{
    const float S1_f = a.S_f + 1.0f;
#pragma unroll
    for (int r = 0; r < F_ROWS; ++r) {
        if (FULL || r < rows) {
            float v[4];
            load_group<FAST>(st + r * FT, a.gp.p[chunk * F_ROWS + r], e0, lo, hi, ct, v);
            if (IDENTITY) {
#pragma unroll
                for (int j = 0; j < 4; ++j) facc[j] += v[j];
            } else {
                uint32_t w[4];
                dat_random_words((uint64_t)e0 >> 2, (uint32_t)(chunk * F_ROWS + r), a.keys, w);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    sum[j] = dat_add_signed_level(sum[j], v[j], dat_level_bits(v[j], qmul, S1_f, w[j]));
            }
        }
    }
}

// Eight warps; consumer thread ct owns elements 4ct..4ct+3 of every tile.  Everything a stage
// needs to know comes from its header, so the consumers touch global memory only for the
// results (and for the masked loads of boundary tiles).  Per-warp partial sums go to the
// reducer warp through a small ring of buffers; the consumers never wait for global memory.
template <bool IDENTITY>
__device__ __forceinline__ void consumer(const FusedArgs &a, Shared &sh, const float *stages)
{
    const int ct = threadIdx.x, lane = ct & 31, warp = ct >> 5;
    uint32_t taken = 0, nred = 0;
    int sum[4] = {0, 0, 0, 0};
    float facc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    const float Mf = (float)a.M;
    for (;;) {
        const uint32_t slot = taken % F_STAGES, use = taken / F_STAGES;
        if (threadIdx.x == 0) PROF_TRACE(0, taken, 0, clock64());
        { PROF_T0();
        if (!wait_mbar(sh, &sh.full[slot], use & 1u, a.status)) return;
        PROF_ADD(0); }
        PROF_T0();
        const StageHdr &H = sh.hdr[slot];
        const uint32_t kind = H.kind;
        if (threadIdx.x == 0) { PROF_TRACE(0, taken, 1, clock64()); PROF_TRACE(0, taken, 2, kind | (H.flags << 4) | ((unsigned long long)H.layer << 16)); }
        taken++;
        const uint32_t rb = nred % F_RED, ruse = nred / F_RED;
        if (kind == ITEM_END) {
            if (!wait_mbar(sh, &sh.red_empty[rb], (ruse & 1u) ^ 1u, a.status)) return;
            if (ct == 0) sh.rdesc[rb].kind = ITEM_END;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.red_full[rb]);
            return;
        }
        const uint32_t flags = H.flags;
        const bool fast = flags & HDR_FAST, last_chunk = flags & HDR_LAST_CHUNK;
        const int chunk = H.chunk;
        const long long lo = H.lo, hi = H.hi, e0 = H.begin + 4 * (long long)ct;
        const float f0 = H.f0, f1 = H.f1;
        const float *st = stages + (size_t)slot * F_STAGE_FLOATS;
        const int rows = min(F_ROWS, a.M - chunk * F_ROWS);

        if (kind == ITEM_N) {
            double acc[F_ROWS];
            if (fast && rows == F_ROWS) rows_sumsq<true, true>(a, st, chunk, rows, e0, lo, hi, ct, acc);
            else if (fast) rows_sumsq<true, false>(a, st, chunk, rows, e0, lo, hi, ct, acc);
            else rows_sumsq<false, false>(a, st, chunk, rows, e0, lo, hi, ct, acc);
            // the item's first chunk claims a hand-off buffer
            if (chunk == 0 && !wait_mbar(sh, &sh.red_empty[rb], (ruse & 1u) ^ 1u, a.status)) return;
            if (ct == 0 && last_chunk) {
                sh.rdesc[rb].kind = ITEM_N; sh.rdesc[rb].flush = flags & HDR_FLUSH;
                sh.rdesc[rb].layer = H.layer; sh.rdesc[rb].slot = H.slot;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.empty[slot]);
            const double s = warp_sum_rows(acc, lane);
            if ((lane & 7) == 0 && (lane >> 3) < rows) sh.red[rb][warp][chunk * F_ROWS + (lane >> 3)] = s;
            if (last_chunk) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.red_full[rb]);
                nred++;
            }
            PROF_ADD(1);
        } else if (kind == ITEM_Q) {
            if (chunk == 0) {
#pragma unroll
                for (int j = 0; j < 4; ++j) { sum[j] = 0; facc[j] = 0.0f; }
            }
            if (fast && rows == F_ROWS) rows_quant<IDENTITY, true, true>(a, st, chunk, rows, e0, lo, hi, ct, f0, sum, facc);
            else if (fast) rows_quant<IDENTITY, true, false>(a, st, chunk, rows, e0, lo, hi, ct, f0, sum, facc);
            else rows_quant<IDENTITY, false, false>(a, st, chunk, rows, e0, lo, hi, ct, f0, sum, facc);
            if (!last_chunk) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.empty[slot]);
                PROF_ADD(2);
                continue;
            }
            float th[4], m[4], ghat[4];
            if (fast) {
                load_group<true>(st + F_ROWS * FT, a.theta, e0, lo, hi, ct, th);
                load_group<true>(st + (F_ROWS + 1) * FT, a.mom, e0, lo, hi, ct, m);
            } else {
                load_group<false>(st, a.theta, e0, lo, hi, ct, th);
                load_group<false>(st, a.mom, e0, lo, hi, ct, m);
            }
            if (ct == 0) {
                sh.rdesc[rb].kind = ITEM_Q; sh.rdesc[rb].flush = flags & HDR_FLUSH;
                sh.rdesc[rb].layer = H.layer; sh.rdesc[rb].slot = H.slot;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.empty[slot]);
            if (IDENTITY) {
#pragma unroll
                for (int j = 0; j < 4; ++j) ghat[j] = facc[j] / Mf;
            } else {
                if (a.code_sum) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (e0 + j >= lo && e0 + j < hi) a.code_sum[e0 + j] = sum[j];
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) ghat[j] = (float)sum[j] * f1;
            }
            double ss0 = 0.0, ss1 = 0.0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                m[j] = __fmaf_rn(a.mu, m[j], __fmaf_rn(a.wd, th[j], ghat[j]));
                ss0 = fma((double)th[j], (double)th[j], ss0);
                ss1 = fma((double)m[j], (double)m[j], ss1);
            }
            if (e0 < hi) dat_store4(a.mom, e0, lo, hi, m);
            ss0 = dat_warp_sum(ss0);
            ss1 = dat_warp_sum(ss1);
            if (!wait_mbar(sh, &sh.red_empty[rb], (ruse & 1u) ^ 1u, a.status)) return;
            if (lane == 0) { sh.red[rb][warp][0] = ss0; sh.red[rb][warp][1] = ss1; }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.red_full[rb]);
            nred++;
            PROF_ADD(2);
        } else {
            float th[4], m[4];
            if (fast) {
                load_group<true>(st + F_ROWS * FT, a.theta, e0, lo, hi, ct, th);
                load_group<true>(st + (F_ROWS + 1) * FT, a.mom, e0, lo, hi, ct, m);
            } else {
                dat_load4(a.theta, e0, lo, hi, th);
#pragma unroll
                for (int j = 0; j < 4; ++j) m[j] = (e0 + j >= lo && e0 + j < hi) ? __ldcg(a.mom + e0 + j) : 0.0f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.empty[slot]);
#pragma unroll
            for (int j = 0; j < 4; ++j) th[j] = __fmaf_rn(f0, m[j], th[j]);
            if (e0 < hi) dat_store4(a.theta, e0, lo, hi, th);
            PROF_ADD(3);
        }
    }
}

template <bool IDENTITY>
__global__ void __launch_bounds__(F_THREADS, F_CTAS_PER_SM)
k_fused_step(const __grid_constant__ FusedArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *stages = reinterpret_cast<float *>(smem_raw);
    Shared &sh = *reinterpret_cast<Shared *>(smem_raw + (size_t)F_STAGES * F_STAGE_BYTES);

    if (threadIdx.x == 0) {
        for (int s = 0; s < F_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], F_CW); }
        for (int b = 0; b < F_RED; ++b) { mbar_init(&sh.red_full[b], F_CW); mbar_init(&sh.red_empty[b], 1); }
        sh.abort_flag = 0;
        sh.acc_q[0] = sh.acc_q[1] = 0.0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < DAT_MAX_WORKERS) sh.acc_n[threadIdx.x] = 0.0;
    __syncthreads();

    PROF_T0();
    uint32_t issued = 0;
    const int warp = threadIdx.x >> 5;
    if (warp < F_CW) consumer<IDENTITY>(a, sh, stages);
    else if (warp == F_CW) issued = producer<IDENTITY>(a, sh, stages);
    else reducer(a, sh);
    __syncthreads();
    PROF_ADD(threadIdx.x == 0 ? 9 : 10);

    if (threadIdx.x == F_CT) {
        // After an abort copies may still be in flight: wait (bounded) for the last use of every
        // stage before the shared memory is given back.
        if (*(volatile int *)&sh.abort_flag) {
            const uint32_t first = issued > F_STAGES ? issued - F_STAGES : 0;
            for (uint32_t s = first; s < issued; ++s) {
                unsigned long long *bar = &sh.full[s % F_STAGES];
                const uint32_t parity = (s / F_STAGES) & 1u;
                const long long t0 = clock64();
                while (!mbar_try_wait(bar, parity) && clock64() - t0 < F_WAIT_CYCLES) {}
            }
        }
        // Last CTA out: after a time-out the dependency counters are in an unknown state; clear
        // them so that the next call starts clean.
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
#ifdef DAT_PROF
static unsigned long long *g_dat_prof = nullptr;
extern "C" void dat_prof_set_buffer(unsigned long long *device_buffer) { g_dat_prof = device_buffer; }
#endif

void dat_fused_destroy(dat_plan_t *plan)
{
    FusedSchedule *f = plan->fused;
    if (!f) return;
    void *ptrs[] = {f->d_items, f->d_tile_base, f->d_slot_base, f->d_expect, f->d_sync, f->d_npart, f->d_qpart};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    delete f;
    plan->fused = nullptr;
}

// The item list: three pointers walk the tiles in layer order.  N runs ahead; a Q tile may be
// emitted once every N tile of its layer was emitted at least `slack` N-items ago (time for the
// stragglers, the reduction and the flag to land), and N may not run more than `max_lag` tiles
// ahead of Q (what L2 can keep) unless Q itself is waiting; U follows Q in the same way.
// Eligible kinds are emitted in turn, so that HBM streaming (N) and the L2/ALU-bound work (Q, U)
// interleave one to one.
static void build_items(std::vector<uint32_t> &items, const std::vector<int64_t> &tile_base, int64_t h,
                        bool identity, int64_t slack, int64_t max_lag)
{
    const int64_t nt = tile_base[h];
    int64_t n = identity ? nt : 0, q = 0, u = 0;
    int64_t lq = 0, lu = 0;                         // layers of the next Q and U tiles
    while (u < nt) {
        while (lq < h && q >= tile_base[lq + 1]) ++lq;
        while (lu < h && u >= tile_base[lu + 1]) ++lu;
        const bool q_ok = q < nt && (n == nt || n >= tile_base[lq + 1] + slack);
        const bool u_ok = (q == nt || q >= tile_base[lu + 1] + slack);
        const bool n_ok = n < nt && (!q_ok || n - q < max_lag);
        if (n_ok) items.push_back(((uint32_t)ITEM_N << 30) | (uint32_t)n++);
        if (q_ok) items.push_back(((uint32_t)ITEM_Q << 30) | (uint32_t)q++);
        if (u_ok) items.push_back(((uint32_t)ITEM_U << 30) | (uint32_t)u++);
    }
}

template <typename T>
static cudaError_t upload(T **dst, const std::vector<T> &src)
{
    cudaError_t e = cudaMalloc((void **)dst, src.size() * sizeof(T));
    if (e != cudaSuccess) return e;
    return cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
}

static int fused_prepare(dat_plan_t *plan)
{
    if (plan->fused) return DAT_OK;
    FusedSchedule *f = new (std::nothrow) FusedSchedule();
    if (!f) return DAT_ERR_NOMEM;
    plan->fused = f;
    const bool identity = (plan->bits == 32);
    const int64_t h = plan->h;
    const int G = plan->sm_count * F_CTAS_PER_SM;
    f->grid = G;
    f->smem_bytes = (size_t)F_STAGES * F_STAGE_BYTES + sizeof(Shared);

    int l2 = 0;
    cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, plan->device);
    f->window_bytes = l2 > 0 ? (int64_t)l2 / 10 * 7 : (int64_t)32 << 20;

    std::vector<uint32_t> items;
    std::vector<int64_t> tile_base(h + 1), slot_base(h + 1);
    std::vector<uint32_t> expect(2 * h, 0);
    try {
        int64_t nt = 0, ns = 0;
        for (int64_t l = 0; l < h; ++l) {
            tile_base[l] = nt;
            slot_base[l] = ns;
            const int64_t a = plan->offsets[l] & ~(int64_t)3;
            const int64_t n = (plan->offsets[l + 1] - a + FT - 1) / FT;
            nt += n;
            ns += std::min<int64_t>(n, G);
        }
        tile_base[h] = nt;
        slot_base[h] = ns;
        if (nt > (int64_t)ITEM_TILE_MASK) return DAT_ERR_UNSUPPORTED;

        // how far N may run ahead of Q: the gradient tiles in between must stay in L2
        const int64_t tile_bytes = (int64_t)FT * 4 * plan->M;
        const int64_t max_lag = std::max<int64_t>(f->window_bytes / tile_bytes, 2 * (int64_t)G);
        items.reserve((size_t)nt * 3);
        build_items(items, tile_base, h, identity, /*slack=*/2 * (int64_t)G, max_lag);
        // flush marks: for every CTA the last N and the last Q item of each layer; count them
        std::vector<int64_t> last_n((size_t)G, -1), last_q((size_t)G, -1);      // item index of the CTA's latest N/Q
        std::vector<int> lay_n((size_t)G, -1), lay_q((size_t)G, -1);
        auto layer_of = [&](int64_t tile) {
            return (int64_t)(std::upper_bound(tile_base.begin(), tile_base.end(), tile) - tile_base.begin()) - 1;
        };
        for (int64_t i = 0; i < (int64_t)items.size(); ++i) {
            const uint32_t type = items[i] >> 30;
            if (type == ITEM_U) continue;
            const int cta = (int)(i % G);
            const int l = (int)layer_of(items[i] & ITEM_TILE_MASK);
            std::vector<int64_t> &last = (type == ITEM_N) ? last_n : last_q;
            std::vector<int> &lay = (type == ITEM_N) ? lay_n : lay_q;
            const int64_t ntl = tile_base[l + 1] - tile_base[l];
            if (last[cta] >= 0 && (lay[cta] != l)) {           // the CTA moved on to another layer
                items[last[cta]] |= ITEM_FLUSH;
                expect[(type == ITEM_N ? 0 : h) + lay[cta]]++;
            }
            last[cta] = i;
            lay[cta] = l;
            if (ntl <= G) {                                     // small layers: one slot per tile, flush at once
                items[i] |= ITEM_FLUSH;
                expect[(type == ITEM_N ? 0 : h) + l]++;
                last[cta] = -1;
            }
        }
        for (int c = 0; c < G; ++c) {
            if (last_n[c] >= 0) { items[last_n[c]] |= ITEM_FLUSH; expect[lay_n[c]]++; }
            if (last_q[c] >= 0) { items[last_q[c]] |= ITEM_FLUSH; expect[h + lay_q[c]]++; }
        }
        f->n_items = (int64_t)items.size();
        f->sync_words = (size_t)h * 4 + 64;
        cudaError_t e = upload(&f->d_items, items);
        if (e == cudaSuccess) e = upload(&f->d_tile_base, tile_base);
        if (e == cudaSuccess) e = upload(&f->d_slot_base, slot_base);
        if (e == cudaSuccess) e = upload(&f->d_expect, expect);
        if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_sync, f->sync_words * 4);
        if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_npart, (size_t)ns * plan->M * 8);
        if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_qpart, (size_t)ns * 16);
        if (e == cudaSuccess) e = cudaMemset(f->d_sync, 0, f->sync_words * 4);
        if (e == cudaSuccess) e = cudaMemset(f->d_npart, 0, (size_t)ns * plan->M * 8);
        if (e == cudaSuccess) e = cudaMemset(f->d_qpart, 0, (size_t)ns * 16);
        if (e != cudaSuccess) { plan->last_cuda = (int)e; (void)cudaGetLastError(); return DAT_ERR_NOMEM; }
    } catch (...) { return DAT_ERR_NOMEM; }

    const void *fn = identity ? (const void *)k_fused_step<true> : (const void *)k_fused_step<false>;
    DAT_CUDA(plan, cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)f->smem_bytes));
    int per_sm = 0;
    DAT_CUDA(plan, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, F_THREADS, f->smem_bytes));
    if (per_sm < F_CTAS_PER_SM) return DAT_ERR_UNSUPPORTED;      // the list needs all CTAs resident
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
    if (rc != DAT_OK) { dat_fused_destroy(plan); return rc; }
    FusedSchedule *f = plan->fused;
    const bool identity = (plan->bits == 32);

    f->epoch = (f->epoch == 0xFFFFFFFFu) ? 1u : f->epoch + 1u;
    a.keys = dat_make_keys(seed, step);
    a.theta = theta;
    a.mom = mom;
    a.off = plan->d_offsets;
    a.tile_base = f->d_tile_base;
    a.slot_base = f->d_slot_base;
    a.items = f->d_items;
    a.expect = f->d_expect;
    a.n_items = f->n_items;
    a.npart = f->d_npart;
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

#ifdef DAT_PROF
    a.prof = g_dat_prof;
#endif
    void *params[] = {(void *)&a};
    const void *fn = identity ? (const void *)k_fused_step<true> : (const void *)k_fused_step<false>;
    DAT_CUDA(plan, cudaLaunchCooperativeKernel(fn, dim3((unsigned)f->grid), dim3(F_THREADS), params, f->smem_bytes,
                                               (cudaStream_t)stream));
    plan->launches++;
    return DAT_OK;
}
