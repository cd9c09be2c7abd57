// dat_step: Steps 7, 9 and 12 of Algorithm A1 in ONE persistent, warp-specialised kernel.
//
// The flat vector is cut into per-layer tiles of FT elements.  Every tile passes through three
// work items:
//   N  read the M gradient tiles, fp64 sums of squares per worker.  When a layer's last
//      contribution has arrived, nu_l, S/nu_l and nu_l/(S*M) are published  [||g||_2 of Eq. rand_q]
//   Q  (needs nu_l) re-read the gradient tiles -- by construction still in L2 for layers that
//      fit -- draw the stochastic levels (Eq. xi), sum the signed codes over the workers and
//      scale (Eq. grad_agg), form m' = mu*m + g_hat + wd*theta, store m', fp64 sums of theta^2
//      and m'^2.  When a layer is complete, a_l = lr*tau(||theta_l||)/||u_l|| is published [Eq. 3]
//   U  (needs a_l) theta -= a_l * m'                                                    [Eq. 3]
//
// The host lays the items out as one list in which N runs ahead of Q and Q ahead of U by just
// enough for the dependencies (and no more than L2 can hold); CTA c (two per SM) owns items
// c, c+G, c+2G, ...  Inside a CTA the work is split by role:
//   - two NORM warps stream the CTA's N items straight from HBM with wide loads (HBM-bound,
//     fp64/conversion pipes);
//   - a PRODUCER warp walks the Q and U items ahead of the consumers, waits for the layer flags
//     and moves every tile (M gradient rows, theta, m) into a ring of shared-memory stages with
//     bulk asynchronous copies (cp.async.bulk, completion counted on an mbarrier; no multicast);
//   - eight CONSUMER warps take the stages in order (integer/fp32 pipes: Philox, levels, sums);
//   - a REDUCER warp takes the per-warp partial sums of both groups, keeps the CTA's running
//     sums per layer, publishes them, and -- for the contribution that completes a layer --
//     reduces all contributions in a fixed order and releases the layer's flag.  This keeps the
//     global-memory round trips of the reductions off the streaming and computing warps.
// Tiles that touch a layer boundary or are not full are read with ordinary masked loads.
//
// An item depends only on items earlier in the list and all CTAs are co-resident (cooperative
// launch), so the list cannot deadlock.  Every wait -- on an mbarrier, on a layer flag, on the
// norm warps' throttle -- is bounded all the same: when one runs out the thread sets
// DAT_STATUS_TIMEOUT and the CTA's abort flag, every other waiter sees it and leaves, the
// producer waits (bounded) for its copies in flight, and the kernel returns; the last CTA out
// clears the dependency counters.
#include <algorithm>
#include <cstdlib>
#include <new>

#include "dat_internal.cuh"

#define FT 1024                                  // elements per fused tile
#define F_CW 8                                   // consumer warps (Q and U items)
#define F_CT (F_CW * 32)                         // consumer threads; thread t owns elements 4t..4t+3
#define F_NW 1                                   // norm issuer warp (walks the N items, starts their copies)
#define F_NT (F_NW * 32)
#define F_THREADS (F_CT + F_NT + 64)             // + one producer warp + one reducer warp
#define F_ROWS 4                                 // worker rows per stage
#define F_STAGES 2
#define F_NBUF 3                                 // norm warps' own tile buffers (F_ROWS rows each)
#define F_RED 2                                  // hand-off buffers, consumers -> reducer, Q items
#define F_REDN 1                                 // the same for N items (M values per warp: kept single to fit two CTAs per SM)
#define F_NLEAD 12                               // default: list items the norm warps may run ahead of the producer
#define F_CTAS_PER_SM 2
#define F_STAGE_FLOATS ((F_ROWS + 2) * FT)       // gradient rows + theta row + momentum row
#define F_STAGE_BYTES (F_STAGE_FLOATS * 4)
#define F_NBUF_FLOATS (F_ROWS * FT)
#define F_WAIT_CYCLES (1ll << 31)                // bound of every device-side wait (about a second)

enum { ITEM_N = 0u, ITEM_Q = 1u, ITEM_U = 2u, ITEM_END = 3u };
#define ITEM_FLUSH 0x20000000u                   // the CTA's last item of this kind in the layer
#define ITEM_TILE_MASK 0x1FFFFFFFu

struct FusedSchedule {
    uint4 *d_recs = nullptr;          // the item records, grouped by CTA
    int64_t *d_cta_first = nullptr;   // G+1: first record of each CTA
    int64_t n_items = 0;
    int64_t *d_slot_base = nullptr;   // h+1, partial-sum slots per layer
    uint32_t *d_expect = nullptr;     // 2h: contributions expected per layer (N, Q)
    uint32_t *d_sync = nullptr;       // cnt_n[h] cnt_q[h] done[1]
    unsigned long long *d_flags = nullptr;   // per layer: (epoch, S/nu) (epoch, nu/(S*M)) (epoch, -a_l)
    double *d_npart = nullptr;        // slots * M
    double *d_qpart = nullptr;        // slots * 2
    size_t sync_words = 0;
    int64_t n_slots = 0;
    uint32_t epoch = 0;
    int grid = 0;
    int nlead = F_NLEAD;
    int64_t slack = 0;
    int64_t window_bytes = 0;
    size_t smem_bytes = 0;
};

struct FusedArgs {
    GradPtrs gp;
    PhiloxKeys keys;
    float *theta, *mom;
    const int64_t *off, *slot_base, *cta_first;
    const uint4 *recs;
    const uint32_t *expect;
    double *npart, *qpart;
    uint32_t *cnt_n, *cnt_q, *done, *status;
    unsigned long long *flags;                   // 3 words per layer, each (epoch << 32) | float bits
    float *worker_norms, *scales;
    int32_t *code_sum;
    float *norms_out, *scales_out;
    int h, M, nlead;
    uint32_t epoch;
    float S_f, SM_f, lr, mu, wd, c_l, c_u;
#ifdef DAT_PROF
    unsigned long long *prof;                    // development builds only
#endif
#ifdef DAT_SELFCHECK
    long long d, n_slots;                        // self-checking builds: bounds of the flat vector and of the slots
    long long *check_log;                        // [0] = number of violations, then (site, value) pairs
#endif
};

// What a stage holds: written by the producer (four 16-byte stores), read by every consumer thread.
struct __align__(16) StageHdr {
    uint32_t kind;                               // ITEM_Q, ITEM_U or ITEM_END
    uint32_t flags;                              // HDR_*
    int layer;
    int chunk;                                   // which group of F_ROWS workers
    long long begin, lo;                         // first element of the tile; the layer's bounds [lo, hi)
    long long hi, slot;                          // slot: where the CTA's running sums go on a flush
    float f0, f1;                                // Q: S/nu_l and nu_l/(S*M);  U: -a_l
    int pad[2];
};
enum { HDR_FAST = 1u, HDR_FLUSH = 2u, HDR_LAST_CHUNK = 4u };

// What a group hands to the reducer warp with a buffer of per-warp partial sums.
struct RedDesc {
    uint32_t kind;                               // ITEM_N, ITEM_Q or ITEM_END
    uint32_t flush;
    int layer;
    long long slot;
};

#ifdef DAT_PROF
// counters: 0 c.wait_full 1 n.wait 2 c.Q 3 c.U 4 n.work 5 r.work 6 p.wait_empty 7 p.wait_flag 8 p.issue 9 total
#define PROF_T0() const long long prof_t0 = clock64()
#define PROF_ADD(k) do { if (a.prof && (threadIdx.x & 31) == 0 && (threadIdx.x == 0 || threadIdx.x == F_CT || threadIdx.x >= F_CT + F_NT)) sh.prof[(k)] += (unsigned long long)(clock64() - prof_t0); } while (0)
#define PROF_LAYER(layer, col) do { if (a.prof) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); a.prof[296 * 16 + 2 * 4096 * 8 + (layer) * 4 + (col)] = t_; } } while (0)
#define PROF_TRACE(role, idx, col, val) do { if (a.prof && blockIdx.x == 0 && (threadIdx.x & 31) == 0 && (idx) < 4096) a.prof[296 * 16 + ((role) * 4096 + (idx)) * 8 + (col)] = (unsigned long long)(val); } while (0)
#else
#define PROF_TRACE(role, idx, col, val) do {} while (0)
#define PROF_LAYER(layer, col) do {} while (0)
#define PROF_T0() do {} while (0)
#define PROF_ADD(k) do {} while (0)
#endif

// What a norm buffer holds: written by the issuing norm warp, read by both.
struct __align__(16) NormHdr {
    uint32_t kind;                               // ITEM_N or ITEM_END
    uint32_t flags;                              // HDR_FAST | HDR_FLUSH | HDR_LAST_CHUNK
    int layer;
    int row0;                                    // first worker row of this pass
    long long begin, lo;
    long long hi, slot;
};

#ifdef DAT_SELFCHECK
// Self-checking build: a failed check records (site, value), sets DAT_STATUS_BOUNDS and the
// guarded access is skipped.
#define DAT_CHECK(cond, site, value) ((cond) ? true : (dat_check_fail(a, (site), (long long)(value)), false))
__device__ __noinline__ void dat_check_fail(const FusedArgs &a, int site, long long value)
{
    atomicOr(a.status, DAT_STATUS_BOUNDS);
    if (a.check_log) {
        const unsigned long long k = atomicAdd((unsigned long long *)a.check_log, 1ull);
        if (k < 64) { a.check_log[1 + 2 * k] = ((long long)blockIdx.x << 32) | (threadIdx.x << 8) | site; a.check_log[2 + 2 * k] = value; }
    }
}
#else
#define DAT_CHECK(cond, site, value) (true)
#endif

struct Shared {
    unsigned long long full[F_STAGES], empty[F_STAGES];
    unsigned long long nfull[F_NBUF], nempty[F_NBUF];         // norm warps' buffers
    unsigned long long nred_full[F_REDN], nred_empty[F_REDN]; // consumers -> reducer, N items
    unsigned long long qred_full[F_RED], qred_empty[F_RED];   // consumer warps -> reducer
    StageHdr hdr[F_STAGES];
    NormHdr nhdr[F_NBUF];
    RedDesc ndesc[F_REDN], qdesc[F_RED];
    double red_n[F_REDN][F_CW][DAT_MAX_WORKERS];  // per-warp sums of squares of one N item
    double red_q[F_RED][F_CW][2];                // per-warp sums of theta^2 and m'^2 of one Q item
    double acc_n[DAT_MAX_WORKERS];               // the CTA's running sums for its current layer (reducer)
    double acc_q[2];
#ifdef DAT_PROF
    unsigned long long prof[16];
#endif
    int q_pos;                                   // list position of the producer (throttles the norm warps)
    int n_issued;                                // passes the norm warps have started
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
__device__ __forceinline__ bool mbar_test_wait(unsigned long long *bar, uint32_t parity)      // never blocks
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
__device__ __forceinline__ void red_add(uint32_t *p)
{
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
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

// ---- the item list -----------------------------------------------------------------------------
// One 16-byte record per item, written by the host, grouped by CTA in execution order:
//   x = kind | flush << 2 | fast << 3 | layer << 8     y = partial-sum slot (N, Q)
//   z, w = first element of the tile (a multiple of 4)
// "fast" = a full tile inside its layer (moved by bulk copies); other tiles are masked with the
// layer's bounds.  A warp fetches 32 records with one coalesced load.
#define REC_FLUSH 4u
#define REC_FAST 8u

struct Item {
    uint32_t kind, flags;
    int layer;
    long long slot, begin;
};

__device__ __forceinline__ Item item_from(uint4 r)
{
    Item it;
    it.kind = r.x & 3u;
    it.flags = r.x & (REC_FLUSH | REC_FAST);
    it.layer = (int)(r.x >> 8);
    it.slot = r.y;
    it.begin = (long long)(((unsigned long long)r.w << 32) | r.z);
    return it;
}

__device__ __forceinline__ uint4 shfl_rec(uint4 r, int src)
{
    return make_uint4(__shfl_sync(0xFFFFFFFFu, r.x, src), __shfl_sync(0xFFFFFFFFu, r.y, src),
                      __shfl_sync(0xFFFFFFFFu, r.z, src), __shfl_sync(0xFFFFFFFFu, r.w, src));
}

// The layer's bounds as the consumers need them: exact for masked tiles, the tile itself otherwise.
__device__ __forceinline__ void item_bounds(const FusedArgs &a, const Item &it, long long &lo, long long &hi)
{
    if (it.flags & REC_FAST) { lo = it.begin; hi = it.begin + FT; }
    else { lo = __ldg(a.off + it.layer); hi = __ldg(a.off + it.layer + 1); }
}

// Per-layer result words: (epoch << 32) | float bits.  Valid once the epoch matches.
__device__ __forceinline__ unsigned long long ld_acquire64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Waits (bounded) until the `nwords` result words at p carry this call's epoch; returns their
// float payloads.  One round trip when they are already there.
__device__ __forceinline__ bool wait_words(Shared &sh, const unsigned long long *p, int nwords, uint32_t epoch,
                                           uint32_t *status, float out[2])
{
    const long long t0 = clock64();
    for (uint32_t spins = 0;; ++spins) {
        const unsigned long long w0 = ld_acquire64(p);
        const unsigned long long w1 = (nwords > 1) ? ld_acquire64(p + 1) : w0;
        if ((uint32_t)(w0 >> 32) == epoch && (uint32_t)(w1 >> 32) == epoch) {
            out[0] = __uint_as_float((uint32_t)w0);
            out[1] = __uint_as_float((uint32_t)w1);
            return true;
        }
        __nanosleep(32);
        if ((spins & 15u) == 15u) {
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

// Cross-lane sum of four per-lane values: after the call, lanes with (lane & 7) == 0 hold the
// warp total of value number (lane >> 3).  Fixed order: 2 exchange-and-halve steps, 3 plain.
__device__ __forceinline__ double warp_sum4(double v[4], int lane)
{
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

// ---- norm warps ------------------------------------------------------------------------------------
// Each pass over F_ROWS worker rows of a tile goes through one of the norm warps' own
// shared-memory buffers.  The first norm warp walks the CTA's N items and starts the bulk copies
// up to F_NBUF passes ahead (lane r moves row r); both warps then add the exact fp64 squares of
// their halves of every pass, in order, and hand the per-warp sums of each item to the reducer.
struct NormWalk {
    long long first, n;                          // this CTA's records
    int pos = 0;                                 // list position of the next record to look at
    uint4 batch;                                 // lane j holds record (pos rounded down to 32) + j
    int batch_base = -1;
    bool have_item = false;                      // an N item has been found and waits for the throttle
    Item item;
    int item_pos = 0;
    int row0 = -1;                               // next worker row of the item being cut into passes
    long long lo = 0, hi = 0;
};

enum { NORM_ISSUED = 0, NORM_END = 1, NORM_LATER = 2, NORM_FAIL = 3 };

// Tries to start pass number `seq` (buffer seq % F_NBUF): the next F_ROWS rows of the current
// item, or of the next N item of the list -- unless that item is still too far ahead of the
// producer (NORM_LATER: the caller goes on with what is already in flight; what is streamed here
// must still be in L2 when the consumers re-read it).  Writes the buffer's header; ITEM_END when
// the list is exhausted.  Called by the whole first norm warp.
__device__ __forceinline__ int norm_issue(const FusedArgs &a, Shared &sh, float *nbuf, NormWalk &w, uint32_t seq, int lane)
{
    const uint32_t b = seq % F_NBUF, use = seq / F_NBUF;
    PROF_T0();
    if (w.row0 < 0) {                            // next N item
        while (!w.have_item && w.pos < w.n) {
            if ((w.pos & ~31) != w.batch_base) {
                w.batch_base = w.pos & ~31;
                w.batch = (w.batch_base + lane < w.n) ? __ldg(a.recs + w.first + w.batch_base + lane) : make_uint4(ITEM_U, 0, 0, 0);
            }
            const uint4 r = shfl_rec(w.batch, w.pos & 31);
            if ((r.x & 3u) == ITEM_N) { w.have_item = true; w.item = item_from(r); w.item_pos = w.pos; }
            w.pos++;
        }
        if (!w.have_item) {
            if (!wait_mbar(sh, &sh.nempty[b], (use & 1u) ^ 1u, a.status)) return NORM_FAIL;
            if (lane == 0) { sh.nhdr[b].kind = ITEM_END; sh.n_issued = (int)seq + 1; }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.nfull[b]);
            return NORM_END;
        }
        if (w.item_pos > *(volatile int *)&sh.q_pos + a.nlead) return NORM_LATER;
        item_bounds(a, w.item, w.lo, w.hi);
        w.row0 = 0;
        w.have_item = false;
    }
    PROF_ADD(10);
    const int rows = min(F_ROWS, a.M - w.row0);
    const bool last = (w.row0 + F_ROWS >= a.M);
    const bool fast = (w.item.flags & REC_FAST) != 0;
    { PROF_T0();
    if (!wait_mbar(sh, &sh.nempty[b], (use & 1u) ^ 1u, a.status)) return NORM_FAIL;
    PROF_ADD(12); }
    {
    PROF_T0();
    if (fast) {
        if (lane == 0) mbar_expect_tx(&sh.nfull[b], (uint32_t)rows * (FT * 4));
        __syncwarp();
        if (lane < rows) {
            if (DAT_CHECK(w.item.begin >= 0 && w.item.begin + FT <= a.d && w.row0 + lane < a.M && (w.item.begin & 3) == 0, 1, w.item.begin))
                bulk_g2s(nbuf + (size_t)b * F_NBUF_FLOATS + lane * FT, a.gp.p[w.row0 + lane] + w.item.begin, FT * 4, &sh.nfull[b]);
        }
    }
    if (lane == 0) {
        uint4 *H = reinterpret_cast<uint4 *>(&sh.nhdr[b]);
        const uint32_t flags = (fast ? HDR_FAST : 0u) | ((w.item.flags & REC_FLUSH) ? HDR_FLUSH : 0u) | (last ? HDR_LAST_CHUNK : 0u);
        H[0] = make_uint4(ITEM_N, flags, (uint32_t)w.item.layer, (uint32_t)w.row0);
        H[1] = make_uint4((uint32_t)w.item.begin, (uint32_t)(w.item.begin >> 32), (uint32_t)w.lo, (uint32_t)(w.lo >> 32));
        H[2] = make_uint4((uint32_t)w.hi, (uint32_t)(w.hi >> 32), (uint32_t)w.item.slot, (uint32_t)(w.item.slot >> 32));
        sh.n_issued = (int)seq + 1;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.nfull[b]);
    w.row0 = last ? -1 : w.row0 + F_ROWS;
    PROF_ADD(11);
    }
    return NORM_ISSUED;
}

// F_ROWS rows of a full tile from a norm buffer: consumer thread ct owns the 16-byte group ct.
template <bool FULL>
__device__ __forceinline__ void norm_rows(const float *buf, int rows, int ct, double acc[F_ROWS])
{
#pragma unroll
    for (int r = 0; r < F_ROWS; ++r) {
        acc[r] = 0.0;
        if (FULL || r < rows) {
            const float4 v = *(reinterpret_cast<const float4 *>(buf + r * FT) + ct);
            const double x = (double)v.x, y = (double)v.y, z = (double)v.z, w = (double)v.w;
            acc[r] = fma(w, w, fma(z, z, fma(y, y, x * x)));
        }
    }
}

// The same for a tile at a layer boundary: masked global loads.
__device__ __noinline__ void norm_rows_masked(const FusedArgs &a, int row0, int rows, long long begin, long long lo,
                                               long long hi, int ct, double acc[F_ROWS])
{
#pragma unroll 1
    for (int r = 0; r < F_ROWS; ++r) {
        double s = 0.0;
        if (r < rows) {
            float v[4];
            dat_load4(a.gp.p[row0 + r], begin + 4 * (long long)ct, lo, hi, v);
            s = fma((double)v[3], (double)v[3], fma((double)v[2], (double)v[2], fma((double)v[1], (double)v[1], (double)v[0] * (double)v[0])));
        }
        acc[r] = s;
    }
}

// One pass of the norm ring, taken by every consumer warp.  Returns 1 = pass done, 0 = end
// marker, -1 = a wait gave up.  The caller has seen nfull[seq % F_NBUF] complete.
__device__ __forceinline__ int norm_consume(const FusedArgs &a, Shared &sh, const float *nbuf, uint32_t seq,
                                            uint32_t &nred, int ct, double nacc[2 * F_ROWS])
{
    static_assert(F_ROWS == 4, "the cross-lane sum is written for four rows");
    const int lane = ct & 31, warp = ct >> 5;
    const uint32_t b = seq % F_NBUF;
    PROF_T0();
    const NormHdr &H = sh.nhdr[b];
    const uint32_t rb = nred % F_REDN, ruse = nred / F_REDN;
    if (H.kind != ITEM_N) {
        if (!wait_mbar(sh, &sh.nred_empty[rb], (ruse & 1u) ^ 1u, a.status)) return -1;
        if (ct == 0) sh.ndesc[rb].kind = ITEM_END;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.nred_full[rb]);
        return 0;
    }
    const uint32_t flags = H.flags;
    const int row0 = H.row0, rows = min(F_ROWS, a.M - row0);
    double acc[F_ROWS];
    if ((flags & HDR_FAST) && rows == F_ROWS) norm_rows<true>(nbuf + (size_t)b * F_NBUF_FLOATS, rows, ct, acc);
    else if (flags & HDR_FAST) norm_rows<false>(nbuf + (size_t)b * F_NBUF_FLOATS, rows, ct, acc);
    else norm_rows_masked(a, row0, rows, H.begin, H.lo, H.hi, ct, acc);
    const int layer = H.layer;
    const long long slot = H.slot;
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.nempty[b]);
    const bool last = (flags & HDR_LAST_CHUNK) != 0;
    if (a.M <= 2 * F_ROWS) {
        // Few workers: every thread keeps its own running sums over the CTA's tiles of the layer
        // and they are reduced across lanes only when the CTA's contribution is due.
        if (row0 == 0) {
#pragma unroll
            for (int r = 0; r < F_ROWS; ++r) nacc[r] += acc[r];
        } else {
#pragma unroll
            for (int r = 0; r < F_ROWS; ++r) nacc[F_ROWS + r] += acc[r];
        }
        if (last && (flags & HDR_FLUSH)) {
            if (!wait_mbar(sh, &sh.nred_empty[rb], (ruse & 1u) ^ 1u, a.status)) return -1;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const double s = warp_sum4(nacc + half * F_ROWS, lane);
                if ((lane & 7) == 0 && half * F_ROWS + (lane >> 3) < a.M) sh.red_n[rb][warp][half * F_ROWS + (lane >> 3)] = s;
            }
#pragma unroll
            for (int r = 0; r < 2 * F_ROWS; ++r) nacc[r] = 0.0;
            if (ct == 0) { sh.ndesc[rb].kind = ITEM_N; sh.ndesc[rb].flush = 1u; sh.ndesc[rb].layer = layer; sh.ndesc[rb].slot = slot; }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.nred_full[rb]);
            nred++;
        }
    } else {
        // the item's first pass claims a hand-off buffer
        if (row0 == 0 && !wait_mbar(sh, &sh.nred_empty[rb], (ruse & 1u) ^ 1u, a.status)) return -1;
        const double s = warp_sum4(acc, lane);
        if ((lane & 7) == 0 && (lane >> 3) < rows) sh.red_n[rb][warp][row0 + (lane >> 3)] = s;
        if (last) {
            if (ct == 0) {
                sh.ndesc[rb].kind = ITEM_N; sh.ndesc[rb].flush = flags & HDR_FLUSH;
                sh.ndesc[rb].layer = layer; sh.ndesc[rb].slot = slot;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.nred_full[rb]);
            nred++;
        }
    }
    PROF_ADD(1);
    return 1;
}

// The norm issuer warp: walks the CTA's N items and keeps the norm buffers filled, staying
// within `nlead` list items of the producer.
__device__ __forceinline__ void norm_issuer(const FusedArgs &a, Shared &sh, float *nbuf)
{
    const int lane = threadIdx.x & 31;
    NormWalk w;
    w.first = __ldg(a.cta_first + blockIdx.x);
    w.n = __ldg(a.cta_first + blockIdx.x + 1) - w.first;
    long long t_idle = 0;
    for (uint32_t seq = 0;;) {
        const int r = norm_issue(a, sh, nbuf, w, seq, lane);
        if (r == NORM_FAIL || r == NORM_END) return;
        if (r == NORM_ISSUED) { ++seq; t_idle = 0; continue; }
        // the next item is still too far ahead of the producer
        PROF_T0();
        if (t_idle == 0) t_idle = clock64();
        __nanosleep(64);
        if (*(volatile int *)&sh.abort_flag) return;
        if (clock64() - t_idle > F_WAIT_CYCLES) { raise_timeout(sh, a.status); return; }
        PROF_ADD(4);
    }
}

// ---- producer warp -------------------------------------------------------------------------------
// All 32 lanes walk the CTA's item list together (warp-uniform control flow), skipping the N
// items.  Per stage: wait until the slot is free, announce the bytes, start the copies (lane r
// moves row r), write the stage header, arrive.  Layer flags are waited for here, ahead of the
// consumers; a flag already seen is not read again.  Returns the number of stages issued.
template <bool IDENTITY>
__device__ __forceinline__ uint32_t producer(const FusedArgs &a, Shared &sh, float *stages)
{
    const int lane = threadIdx.x & 31;
    uint32_t issued = 0;
    const int nchunks = (a.M + F_ROWS - 1) / F_ROWS;
    const long long first = __ldg(a.cta_first + blockIdx.x);
    const int n = (int)(__ldg(a.cta_first + blockIdx.x + 1) - first);
    int q_layer = -1, u_layer = -1;              // layers whose result words this warp has seen
    float q_f[2] = {0.0f, 0.0f}, u_f[2] = {0.0f, 0.0f};
    uint4 batch = make_uint4(0, 0, 0, 0);
    for (int pos = 0; pos < n; ++pos) {
        if ((pos & 31) == 0) batch = (pos + lane < n) ? __ldg(a.recs + first + pos + lane) : make_uint4(0, 0, 0, 0);
        const uint4 rec = shfl_rec(batch, pos & 31);
        if (lane == 0) *(volatile int *)&sh.q_pos = pos;
        if ((rec.x & 3u) == ITEM_N) continue;
        const Item item = item_from(rec);
        const uint32_t type = item.kind;
        const bool fast = (item.flags & REC_FAST) != 0;
        long long lo, hi;
        item_bounds(a, item, lo, hi);
        if (type == ITEM_U && u_layer != item.layer) {
            // m' of this tile was written by the tile's Q item: the layer's result word orders it
            if (blockIdx.x == 0 && lane == 0) PROF_LAYER(item.layer, 3);
            { PROF_T0();
            if (!wait_words(sh, a.flags + 3 * (long long)item.layer + 2, 1, a.epoch, a.status, u_f)) return issued;
            PROF_ADD(7); }
            u_layer = item.layer;
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
            PROF_TRACE(1, issued, 2, type | ((unsigned long long)item.layer << 16));
            PROF_T0();
            float *st = stages + (size_t)slot * F_STAGE_FLOATS;
            if (fast) {
                const long long begin = item.begin;
                const bool params = (type == ITEM_U) || (c == nst - 1);                     // theta and m rows
                const int rows = (type == ITEM_U) ? 0 : min(F_ROWS, a.M - c * F_ROWS);
                if (lane == 0) mbar_expect_tx(&sh.full[slot], (uint32_t)(rows + (params ? 2 : 0)) * (FT * 4));
                __syncwarp();
                const bool in_range = DAT_CHECK(begin >= 0 && begin + FT <= a.d && (begin & 3) == 0 && c * F_ROWS + rows <= a.M, 2, begin);
                if (in_range && lane < rows) bulk_g2s(st + lane * FT, a.gp.p[c * F_ROWS + lane] + begin, FT * 4, &sh.full[slot]);
                if (in_range && params && lane == F_ROWS) bulk_g2s(st + F_ROWS * FT, a.theta + begin, FT * 4, &sh.full[slot]);
                if (in_range && params && lane == F_ROWS + 1) bulk_g2s(st + (F_ROWS + 1) * FT, a.mom + begin, FT * 4, &sh.full[slot]);
            }
            issued++;
            if (type == ITEM_Q && !IDENTITY && q_layer != item.layer) {
                // every copy announced above has been started, so the stage completes even if
                // this wait gives up
                if (blockIdx.x == 0 && lane == 0) PROF_LAYER(item.layer, 2);
                PROF_T0();
                if (!wait_words(sh, a.flags + 3 * (long long)item.layer, 2, a.epoch, a.status, q_f)) {
                    if (lane == 0) sh.hdr[slot].kind = ITEM_END;      // nothing valid to consume in this stage
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.full[slot]);
                    return issued;
                }
                PROF_ADD(7);
                q_layer = item.layer;
            }
            if (lane == 0) {
                uint4 *H = reinterpret_cast<uint4 *>(&sh.hdr[slot]);
                const uint32_t flags = (fast ? HDR_FAST : 0u) | ((item.flags & REC_FLUSH) ? HDR_FLUSH : 0u) |
                                       ((c == nst - 1) ? HDR_LAST_CHUNK : 0u);
                H[0] = make_uint4(type, flags, (uint32_t)item.layer, (uint32_t)c);
                H[1] = make_uint4((uint32_t)item.begin, (uint32_t)(item.begin >> 32), (uint32_t)lo, (uint32_t)(lo >> 32));
                H[2] = make_uint4((uint32_t)hi, (uint32_t)(hi >> 32), (uint32_t)item.slot, (uint32_t)(item.slot >> 32));
                H[3] = make_uint4(__float_as_uint(type == ITEM_U ? u_f[0] : q_f[0]), __float_as_uint(q_f[1]), 0u, 0u);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.full[slot]);      // release: the header is visible once the stage completes
            PROF_ADD(8);
            PROF_TRACE(1, issued - 1, 3, clock64());
        }
    }
    if (lane == 0) *(volatile int *)&sh.q_pos = 0x3FFFFFFF;          // nothing left to stay close to
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
// N: fold the norm warps' sums into the CTA's running sums of the layer; on a flush item publish
// them and, if that completed the layer, reduce all contributions and publish the scale.
__device__ __forceinline__ void finish_norm(const FusedArgs &a, Shared &sh, int layer, long long slot, int buf,
                                            bool flush, int lane)
{
    for (int i = lane; i < a.M; i += 32) {
        double s = sh.acc_n[i];
#pragma unroll
        for (int w = 0; w < F_CW; ++w) s += sh.red_n[buf][w][i];
        sh.acc_n[i] = s;
    }
    __syncwarp();
    if (!flush) return;
    if (!DAT_CHECK(slot >= 0 && slot < a.n_slots && layer >= 0 && layer < a.h, 8, slot)) return;
    for (int i = lane; i < a.M; i += 32) { a.npart[slot * a.M + i] = sh.acc_n[i]; sh.acc_n[i] = 0.0; }
    __threadfence();
    __syncwarp();
    if (lane == 0) red_add(a.cnt_n + layer);      // no answer needed: the layer's owner watches the count
}

// The owner of a layer (CTA layer mod G) finalises it once every contribution has arrived:
// all contributions are reduced in a fixed order and the layer's scale is published.
__device__ __forceinline__ void finalize_norm(const FusedArgs &a, int layer, int lane)
{
    if (lane == 0) a.cnt_n[layer] = 0u;           // ready for the next call
    const long long s0 = __ldg(a.slot_base + layer);
    const int ns = (int)(__ldg(a.slot_base + layer + 1) - s0);
    // Every lane sums its slots (lane, lane+32, ...) in order, eight workers at a time so that many
    // independent loads are in flight; then a fixed butterfly across the lanes.
    float nu = 0.0f;
    bool bad = false;
    for (int i0 = 0; i0 < a.M; i0 += 8) {
        double acc[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
#pragma unroll 2
        for (int s = lane; s < ns; s += 32) {
            const double *p = a.npart + (s0 + s) * a.M + i0;
            double v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (i0 + j < a.M) ? __ldcg(p + j) : 0.0;
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += v[j];
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (i0 + j < a.M) {
                const float nrm = (float)sqrt(dat_warp_sum(acc[j]));
                if (lane == 0) a.worker_norms[(long long)(i0 + j) * a.h + layer] = nrm;
                bad |= !isfinite(nrm);
                nu = (i0 + j == 0 || nrm > nu) ? nrm : nu;
            }
        }
    }
    if (lane == 0) {
        a.scales[layer] = nu;
        const float qmul = (nu == 0.0f) ? 0.0f : a.S_f / nu;
        const float dq = (nu == 0.0f) ? 0.0f : nu / a.SM_f;
        if (a.scales_out) a.scales_out[layer] = nu;
        if (bad) atomicOr(a.status, DAT_STATUS_NONFINITE);
        PROF_LAYER(layer, 0);
        unsigned long long *w = a.flags + 3 * (long long)layer;
        st_release64(w, ((unsigned long long)a.epoch << 32) | __float_as_uint(qmul));
        st_release64(w + 1, ((unsigned long long)a.epoch << 32) | __float_as_uint(dq));
    }
}

// Q: the same for the sums of theta^2 and m'^2; completing a layer publishes its step length.
__device__ __forceinline__ void finish_quant(const FusedArgs &a, Shared &sh, int layer, long long slot, int buf,
                                             bool flush, int lane)
{
    if (lane < 2) {
        double s = sh.acc_q[lane];
#pragma unroll
        for (int w = 0; w < F_CW; ++w) s += sh.red_q[buf][w][lane];
        sh.acc_q[lane] = s;
    }
    __syncwarp();
    if (!flush) return;
    if (!DAT_CHECK(slot >= 0 && slot < a.n_slots && layer >= 0 && layer < a.h, 9, slot)) return;
    if (lane < 2) { a.qpart[slot * 2 + lane] = sh.acc_q[lane]; sh.acc_q[lane] = 0.0; }
    __threadfence();
    __syncwarp();
    if (lane == 0) red_add(a.cnt_q + layer);
}

__device__ __forceinline__ void finalize_quant(const FusedArgs &a, int layer, int lane)
{
    if (lane == 0) a.cnt_q[layer] = 0u;
    const long long s0 = __ldg(a.slot_base + layer);
    const int ns = (int)(__ldg(a.slot_base + layer + 1) - s0);
    double x = 0.0, y = 0.0;
#pragma unroll 4
    for (int s = lane; s < ns; s += 32) {
        const double2 v = __ldcg(reinterpret_cast<const double2 *>(a.qpart + (s0 + s) * 2));
        x += v.x;
        y += v.y;
    }
    x = dat_warp_sum(x);
    y = dat_warp_sum(y);
    if (lane == 0) {
        const float n_theta = (float)sqrt(x), n_u = (float)sqrt(y);
        const float tau = fminf(fmaxf(n_theta, a.c_l), a.c_u);
        const float ratio = (n_u == 0.0f) ? 0.0f : tau / n_u;
        const float neg_a = -(a.lr * ratio);
        if (a.norms_out) { a.norms_out[2 * layer] = n_theta; a.norms_out[2 * layer + 1] = n_u; }
        if (!isfinite(n_theta) || !isfinite(n_u)) atomicOr(a.status, DAT_STATUS_NONFINITE);
        PROF_LAYER(layer, 1);
        st_release64(a.flags + 3 * (long long)layer + 2, ((unsigned long long)a.epoch << 32) | __float_as_uint(neg_a));
    }
}

// Serves both hand-off rings in turn (non-blocking tests) and finalises the layers this CTA owns
// (layer mod G == CTA) as their contribution counts fill up, until both rings have said END and
// every owned layer is done.
__device__ __forceinline__ void reducer(const FusedArgs &a, Shared &sh, bool have_norm)
{
    const int lane = threadIdx.x & 31;
    uint32_t kn = 0, kq = 0;
    bool done_n = !have_norm, done_q = false;
    int own_n = have_norm ? (int)blockIdx.x : a.h, own_q = (int)blockIdx.x;     // next owned layer to finalise
    uint32_t want_n = (own_n < a.h) ? __ldg(a.expect + own_n) : 0u;
    uint32_t want_q = (own_q < a.h) ? __ldg(a.expect + a.h + own_q) : 0u;
    long long t_last = clock64();
    uint32_t round = 0;
    while (!(done_n && done_q) || own_n < a.h || own_q < a.h) {
        bool progress = false;
        if (!done_n) {
            const uint32_t b = kn % F_REDN;
            if (mbar_test_wait(&sh.nred_full[b], (kn / F_REDN) & 1u)) {
                PROF_T0();
                if (sh.ndesc[b].kind == ITEM_END) done_n = true;
                else {
                    finish_norm(a, sh, sh.ndesc[b].layer, sh.ndesc[b].slot, (int)b, sh.ndesc[b].flush != 0, lane);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.nred_empty[b]);
                }
                kn++;
                progress = true;
                PROF_ADD(5);
            }
        }
        if (!done_q) {
            const uint32_t b = kq % F_RED;
            if (mbar_test_wait(&sh.qred_full[b], (kq / F_RED) & 1u)) {
                PROF_T0();
                if (sh.qdesc[b].kind == ITEM_END) done_q = true;
                else {
                    finish_quant(a, sh, sh.qdesc[b].layer, sh.qdesc[b].slot, (int)b, sh.qdesc[b].flush != 0, lane);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.qred_empty[b]);
                }
                kq++;
                progress = true;
                PROF_ADD(5);
            }
        }
        // owned layers: look at the counts when idle, and every few rounds when busy
        if (!progress || (++round & 3u) == 0u) {
            if (own_n < a.h && ld_acquire(a.cnt_n + own_n) == want_n) {
                PROF_T0();
                finalize_norm(a, own_n, lane);
                own_n += (int)gridDim.x;
                want_n = (own_n < a.h) ? __ldg(a.expect + own_n) : 0u;
                progress = true;
                PROF_ADD(5);
            }
            if (own_q < a.h && ld_acquire(a.cnt_q + own_q) == want_q) {
                PROF_T0();
                finalize_quant(a, own_q, lane);
                own_q += (int)gridDim.x;
                want_q = (own_q < a.h) ? __ldg(a.expect + a.h + own_q) : 0u;
                progress = true;
                PROF_ADD(5);
            }
        }
        if (progress) {
            t_last = clock64();
        } else {
            if (*(volatile int *)&sh.abort_flag || (ld_acquire(a.status) & DAT_STATUS_TIMEOUT)) { atomicExch(&sh.abort_flag, 1); return; }
            if (clock64() - t_last > F_WAIT_CYCLES) { raise_timeout(sh, a.status); return; }
            __nanosleep(40);
        }
    }
}

// ---- consumer warps -----------------------------------------------------------------------------------
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

// The F_ROWS worker rows of one chunk of a full tile, from the stage.
template <bool IDENTITY, bool FULL>
__device__ __forceinline__ void rows_quant(const FusedArgs &a, const float *st, int chunk, int rows, long long e0,
                                           int ct, float qmul, int sum[4], float facc[4])
{
    const float S1_f = a.S_f + 1.0f;
#pragma unroll
    for (int r = 0; r < F_ROWS; ++r) {
        if (FULL || r < rows) {
            const float4 f = *reinterpret_cast<const float4 *>(st + r * FT + 4 * ct);
            const float v[4] = {f.x, f.y, f.z, f.w};
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

// The same for a tile at a layer boundary: masked global loads, one row at a time.
template <bool IDENTITY>
__device__ __noinline__ void rows_quant_masked(const FusedArgs &a, int chunk, int rows, long long e0, long long lo,
                                               long long hi, float qmul, int sum[4], float facc[4])
{
    const float S1_f = a.S_f + 1.0f;
#pragma unroll 1
    for (int r = 0; r < rows; ++r) {
        float v[4];
        dat_load4(a.gp.p[chunk * F_ROWS + r], e0, lo, hi, v);
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

// Eight warps; consumer thread ct owns elements 4ct..4ct+3 of every tile.  Everything a stage
// needs to know comes from its header, so the consumers touch global memory only for the
// results (and for the masked loads of boundary tiles).
template <bool IDENTITY>
__device__ __forceinline__ void consumer(const FusedArgs &a, Shared &sh, const float *stages, const float *nbuf)
{
    const int ct = threadIdx.x, lane = ct & 31, warp = ct >> 5;
    uint32_t taken = 0, nred = 0;                // stage ring, its hand-offs
    uint32_t nseq = 0, nred_n = 0;               // norm ring, its hand-offs
    bool n_done = IDENTITY, q_done = false;
    double nacc[2 * F_ROWS] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};     // running sums of squares (M <= 8)
    double qss0 = 0.0, qss1 = 0.0;               // running sums of theta^2 and m'^2 until the next flush
    int sum[4] = {0, 0, 0, 0};
    float facc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    const float Mf = (float)a.M;
    for (;;) {
        const uint32_t slot = taken % F_STAGES, use = taken / F_STAGES;
        if (threadIdx.x == 0) PROF_TRACE(0, taken, 0, clock64());
        // take whatever is ready, a norm pass first (other CTAs' flags wait for those)
        int pick = -1;
        { PROF_T0();
        long long t0 = 0;
        for (uint32_t spins = 1;; ++spins) {
            if (!n_done && mbar_test_wait(&sh.nfull[nseq % F_NBUF], (nseq / F_NBUF) & 1u)) { pick = 0; break; }
            if (!q_done && mbar_test_wait(&sh.full[slot], use & 1u)) { pick = 1; break; }
            if (n_done && q_done) return;
            __nanosleep(32);
            if ((spins & 63u) == 0u) {
                if (*(volatile int *)&sh.abort_flag) return;
                if (t0 == 0) t0 = clock64();
                else if (clock64() - t0 > F_WAIT_CYCLES) { raise_timeout(sh, a.status); return; }
            }
        }
        PROF_ADD(0); }
        if (pick == 0) {
            const int r = norm_consume(a, sh, nbuf, nseq, nred_n, ct, nacc);
            if (r < 0) return;
            if (r == 0) n_done = true; else ++nseq;
            continue;
        }
        PROF_T0();
        const StageHdr &H = sh.hdr[slot];
        const uint32_t kind = H.kind;
        if (threadIdx.x == 0) { PROF_TRACE(0, taken, 1, clock64()); PROF_TRACE(0, taken, 2, kind | (H.flags << 4) | ((unsigned long long)H.layer << 16)); }
        taken++;
        const uint32_t rb = nred % F_RED, ruse = nred / F_RED;
        if (kind == ITEM_END) {
            if (!wait_mbar(sh, &sh.qred_empty[rb], (ruse & 1u) ^ 1u, a.status)) return;
            if (ct == 0) sh.qdesc[rb].kind = ITEM_END;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.qred_full[rb]);
            q_done = true;
            continue;
        }
        const uint32_t flags = H.flags;
        const bool fast = flags & HDR_FAST, last_chunk = flags & HDR_LAST_CHUNK;
        const int chunk = H.chunk;
        const long long lo = H.lo, hi = H.hi, e0 = H.begin + 4 * (long long)ct;
        const float f0 = H.f0, f1 = H.f1;
        const float *st = stages + (size_t)slot * F_STAGE_FLOATS;
        if (!DAT_CHECK(kind <= ITEM_U && chunk >= 0 && chunk * F_ROWS < a.M && lo >= 0 && lo < hi && hi <= a.d, 7, chunk)) return;

        if (kind == ITEM_Q) {
            const int rows = min(F_ROWS, a.M - chunk * F_ROWS);
            if (chunk == 0) {
#pragma unroll
                for (int j = 0; j < 4; ++j) { sum[j] = 0; facc[j] = 0.0f; }
            }
            if (fast && rows == F_ROWS) rows_quant<IDENTITY, true>(a, st, chunk, rows, e0, ct, f0, sum, facc);
            else if (fast) rows_quant<IDENTITY, false>(a, st, chunk, rows, e0, ct, f0, sum, facc);
            else rows_quant_masked<IDENTITY>(a, chunk, rows, e0, lo, hi, f0, sum, facc);
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
            const uint32_t hflush = flags & HDR_FLUSH;
            const int hlayer = H.layer;
            const long long hslot = H.slot;
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
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                m[j] = __fmaf_rn(a.mu, m[j], __fmaf_rn(a.wd, th[j], ghat[j]));
                qss0 = fma((double)th[j], (double)th[j], qss0);
                qss1 = fma((double)m[j], (double)m[j], qss1);
            }
            if (e0 < hi && DAT_CHECK(lo >= 0 && hi <= a.d && e0 >= 0, 5, e0)) dat_store4(a.mom, e0, lo, hi, m);
            if (hflush) {
                // the CTA's contribution to the layer is due: reduce across lanes and hand over
                const double ss0 = dat_warp_sum(qss0), ss1 = dat_warp_sum(qss1);
                qss0 = 0.0;
                qss1 = 0.0;
                { PROF_T0();
                if (!wait_mbar(sh, &sh.qred_empty[rb], (ruse & 1u) ^ 1u, a.status)) return;
                PROF_ADD(13); }
                if (lane == 0) { sh.red_q[rb][warp][0] = ss0; sh.red_q[rb][warp][1] = ss1; }
                if (ct == 0) {
                    sh.qdesc[rb].kind = ITEM_Q; sh.qdesc[rb].flush = 1u;
                    sh.qdesc[rb].layer = hlayer; sh.qdesc[rb].slot = hslot;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.qred_full[rb]);
                nred++;
            }
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
            if (e0 < hi && DAT_CHECK(lo >= 0 && hi <= a.d && e0 >= 0, 6, e0)) dat_store4(a.theta, e0, lo, hi, th);
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
    float *nbuf = stages + (size_t)F_STAGES * F_STAGE_FLOATS;
    Shared &sh = *reinterpret_cast<Shared *>(smem_raw + (size_t)F_STAGES * F_STAGE_BYTES + (size_t)F_NBUF * F_NBUF_FLOATS * 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < F_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], F_CW); }
        for (int b = 0; b < F_NBUF; ++b) { mbar_init(&sh.nfull[b], 1); mbar_init(&sh.nempty[b], F_CW); }
        for (int b = 0; b < F_REDN; ++b) { mbar_init(&sh.nred_full[b], F_CW); mbar_init(&sh.nred_empty[b], 1); }
        for (int b = 0; b < F_RED; ++b) { mbar_init(&sh.qred_full[b], F_CW); mbar_init(&sh.qred_empty[b], 1); }
        for (int s = 0; s < F_STAGES; ++s) sh.hdr[s].kind = ITEM_END;
        for (int b = 0; b < F_NBUF; ++b) sh.nhdr[b].kind = ITEM_END;
#ifdef DAT_PROF
        for (int k = 0; k < 16; ++k) sh.prof[k] = 0;
#endif
        sh.abort_flag = 0;
        sh.q_pos = 0;
        sh.n_issued = 0;
        sh.acc_q[0] = sh.acc_q[1] = 0.0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < DAT_MAX_WORKERS) sh.acc_n[threadIdx.x] = 0.0;
    __syncthreads();

    PROF_T0();
    uint32_t issued = 0;
    const int warp = threadIdx.x >> 5;
    if (warp < F_CW) consumer<IDENTITY>(a, sh, stages, nbuf);
    else if (warp < F_CW + F_NW) { if (!IDENTITY) norm_issuer(a, sh, nbuf); }
    else if (warp == F_CW + F_NW) issued = producer<IDENTITY>(a, sh, stages);
    else reducer(a, sh, !IDENTITY);
    PROF_ADD(9);
    __syncthreads();
#ifdef DAT_PROF
    if (a.prof && threadIdx.x < 16) a.prof[blockIdx.x * 16 + threadIdx.x] += sh.prof[threadIdx.x];
#endif

    if (threadIdx.x == F_CT && !IDENTITY && *(volatile int *)&sh.abort_flag) {
        // after an abort the norm warps' last copies may still be in flight: wait (bounded) for the
        // last use of each of their buffers
        const uint32_t n = (uint32_t)sh.n_issued, first = n > F_NBUF ? n - F_NBUF : 0;
        for (uint32_t q = first; q < n; ++q) {
            const long long t0 = clock64();
            while (!mbar_test_wait(&sh.nfull[q % F_NBUF], (q / F_NBUF) & 1u) && clock64() - t0 < F_WAIT_CYCLES) {}
        }
    }
    if (threadIdx.x == F_CT + F_NT) {
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
#ifdef DAT_SELFCHECK
static long long *g_dat_check_log = nullptr;
extern "C" void dat_selfcheck_set_log(long long *device_buffer) { g_dat_check_log = device_buffer; }
#endif
#ifdef DAT_PROF
static unsigned long long *g_dat_prof = nullptr;
extern "C" void dat_prof_set_buffer(unsigned long long *device_buffer) { g_dat_prof = device_buffer; }
#endif

void dat_fused_destroy(dat_plan_t *plan)
{
    FusedSchedule *f = plan->fused;
    if (!f) return;
    void *ptrs[] = {f->d_recs, f->d_cta_first, f->d_slot_base, f->d_expect, f->d_sync, f->d_flags, f->d_npart, f->d_qpart};
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
    f->smem_bytes = (size_t)F_STAGES * F_STAGE_BYTES + (size_t)F_NBUF * F_NBUF_FLOATS * 4 + sizeof(Shared);

    int l2 = 0;
    cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, plan->device);
    f->window_bytes = l2 > 0 ? (int64_t)l2 / 10 * 7 : (int64_t)32 << 20;
    f->slack = 4 * (int64_t)G;
#ifdef DAT_PROF
    if (const char *e = getenv("DAT_FUSED_WINDOW_MB")) f->window_bytes = (int64_t)atoi(e) << 20;
    if (const char *e = getenv("DAT_FUSED_SLACK")) f->slack = atoi(e);
    if (const char *e = getenv("DAT_FUSED_NLEAD")) f->nlead = atoi(e);
#endif

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
        f->n_slots = ns;
        if (nt > (int64_t)ITEM_TILE_MASK) return DAT_ERR_UNSUPPORTED;

        // how far N may run ahead of Q: the gradient tiles in between must stay in L2
        const int64_t tile_bytes = (int64_t)FT * 4 * plan->M;
        const int64_t max_lag = std::max<int64_t>(f->window_bytes / tile_bytes, 2 * (int64_t)G);
        items.reserve((size_t)nt * 3);
        build_items(items, tile_base, h, identity, f->slack, max_lag);
        // Records, grouped by CTA (item i belongs to CTA i mod G).  For N and Q items the record
        // names the slot of the CTA's running sums: layers with at most G tiles use one slot per
        // tile and flush at once; in larger layers a CTA accumulates over its tiles of the layer
        // and flushes with its last one (slot = the CTA's index).  expect[] counts the flushes.
        auto layer_of = [&](int64_t tile) {
            return (int64_t)(std::upper_bound(tile_base.begin(), tile_base.end(), tile) - tile_base.begin()) - 1;
        };
        const int64_t n_items = (int64_t)items.size();
        std::vector<int64_t> cta_first((size_t)G + 1, 0);
        for (int c = 0; c < G; ++c) cta_first[c + 1] = cta_first[c] + (n_items > c ? (n_items - 1 - c) / G + 1 : 0);
        std::vector<uint4> recs((size_t)n_items);
        std::vector<int64_t> last_rec[2] = {std::vector<int64_t>((size_t)G, -1), std::vector<int64_t>((size_t)G, -1)};
        std::vector<int> last_layer[2] = {std::vector<int>((size_t)G, -1), std::vector<int>((size_t)G, -1)};
        for (int64_t i = 0; i < n_items; ++i) {
            const uint32_t type = items[i] >> 30;
            const int64_t tile = items[i] & ITEM_TILE_MASK;
            const int cta = (int)(i % G);
            const int64_t r = cta_first[cta] + i / G;
            const int l = (int)layer_of(tile);
            const int64_t lo = plan->offsets[l], hi = plan->offsets[l + 1];
            const int64_t begin = (lo & ~(int64_t)3) + (tile - tile_base[l]) * FT;
            const bool fast = begin >= lo && begin + FT <= hi;
            uint32_t info = type | (fast ? REC_FAST : 0u) | ((uint32_t)l << 8);
            uint32_t slot = 0;
            if (type != ITEM_U) {
                const int k = (type == ITEM_N) ? 0 : 1;
                const int64_t ntl = tile_base[l + 1] - tile_base[l];
                if (last_rec[k][cta] >= 0 && last_layer[k][cta] != l) {     // the CTA moved on to another layer
                    recs[last_rec[k][cta]].x |= REC_FLUSH;
                    expect[k * h + last_layer[k][cta]]++;
                    last_rec[k][cta] = -1;
                }
                if (ntl <= G) {
                    slot = (uint32_t)(slot_base[l] + (tile - tile_base[l]));
                    info |= REC_FLUSH;
                    expect[k * h + l]++;
                } else {
                    slot = (uint32_t)(slot_base[l] + cta);
                    last_rec[k][cta] = r;
                    last_layer[k][cta] = l;
                }
            }
            recs[r] = make_uint4(info, slot, (uint32_t)begin, (uint32_t)((uint64_t)begin >> 32));
        }
        for (int k = 0; k < 2; ++k)
            for (int c = 0; c < G; ++c)
                if (last_rec[k][c] >= 0) { recs[last_rec[k][c]].x |= REC_FLUSH; expect[k * h + last_layer[k][c]]++; }
        if (ns > 0xFFFFFFFFll || h >= (1 << 24)) return DAT_ERR_UNSUPPORTED;
        f->n_items = n_items;
        f->sync_words = (size_t)h * 2 + 64;
        cudaError_t e = upload(&f->d_recs, recs);
        if (e == cudaSuccess) e = upload(&f->d_cta_first, cta_first);
        if (e == cudaSuccess) e = upload(&f->d_slot_base, slot_base);
        if (e == cudaSuccess) e = upload(&f->d_expect, expect);
        if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_sync, f->sync_words * 4);
        if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_flags, (size_t)h * 3 * 8);
        if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_npart, (size_t)ns * plan->M * 8);
        if (e == cudaSuccess) e = cudaMalloc((void **)&f->d_qpart, (size_t)ns * 16);
        if (e == cudaSuccess) e = cudaMemset(f->d_sync, 0, f->sync_words * 4);
        if (e == cudaSuccess) e = cudaMemset(f->d_flags, 0, (size_t)h * 3 * 8);
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
    a.slot_base = f->d_slot_base;
    a.cta_first = f->d_cta_first;
    a.recs = f->d_recs;
    a.expect = f->d_expect;
    a.npart = f->d_npart;
    a.qpart = f->d_qpart;
    const size_t h = (size_t)plan->h;
    a.cnt_n = f->d_sync;
    a.cnt_q = f->d_sync + h;
    a.done = f->d_sync + 2 * h;
    a.flags = f->d_flags;
    a.status = plan->d_status;
    a.worker_norms = plan->d_worker_norms;
    a.scales = plan->d_scales;
    a.code_sum = identity ? nullptr : code_sum_out;
    a.norms_out = layer_norms_out;
    a.scales_out = identity ? nullptr : scales_out;
    a.h = (int)plan->h;
    a.M = plan->M;
    a.nlead = f->nlead;
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
#ifdef DAT_SELFCHECK
    a.d = plan->d;
    a.n_slots = f->n_slots;
    a.check_log = g_dat_check_log;
#endif
    void *params[] = {(void *)&a};
    const void *fn = identity ? (const void *)k_fused_step<true> : (const void *)k_fused_step<false>;
    DAT_CUDA(plan, cudaLaunchCooperativeKernel(fn, dim3((unsigned)f->grid), dim3(F_THREADS), params, f->smem_bytes,
                                               (cudaStream_t)stream));
    plan->launches++;
    return DAT_OK;
}
