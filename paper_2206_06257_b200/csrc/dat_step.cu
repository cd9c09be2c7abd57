// dat_step: Steps 7, 9 and 12 of Algorithm A1 in ONE persistent kernel of self-feeding warps.
//
// The flat vector is cut into per-layer tiles of FT elements.  Every tile passes through three
// work items:
//   N  read the M gradient tiles, fp64 sums of squares per worker.  When a layer's last
//      contribution has arrived, nu_l, S/nu_l and nu_l/(S*M) are published  [||g||_2 of Eq. rand_q]
//   Q  (needs nu_l) re-read the gradient tiles -- still in L2 for layers that fit -- draw the
//      stochastic levels (Eq. xi), sum the signed codes over the workers and scale (Eq. grad_agg),
//      form m' = mu*m + g_hat + wd*theta, store m', fp64 sums of theta^2 and m'^2.  When a layer
//      is complete, a_l = lr*tau(||theta_l||)/||u_l|| is published                      [Eq. 3]
//   U  (needs a_l) theta -= a_l * m'                                                    [Eq. 3]
//
// The host lays the items out as one list in which N runs ahead of Q and Q ahead of U by just
// enough for the dependencies; layers are taken largest first, so that the end of the list,
// where nothing is left to overlap with, belongs to the small ones.  Within a layer the Q items
// walk the tiles in the opposite direction of the N items (and the U items in the opposite
// direction of the Q items), so that a layer larger than L2 still finds its most recently read
// part there.  A tile's three items go
// to the same CTA (tile index mod G; one CTA per SM); every CTA takes its items in list order.
//
// Inside a CTA every COMPUTE warp owns a fixed 256-element slice of each tile and feeds itself:
// it walks the CTA's item records, moves its slice of up to eight gradient rows (plus the theta
// and m rows) into its own shared-memory slots with asynchronous copies (cp.async, 16 bytes per
// lane, one group per batch), one batch ahead of the batch it is working on, and consumes the
// batches in order.  Compute warps never wait for each other;
// their running sums (squares per worker; theta^2 and m'^2) stay in registers across the tiles
// of a layer and are handed to the CTA's REDUCER warp only when the CTA's contribution to the
// layer is due.  The reducer warp adds the warps' sums in a fixed order, publishes the CTA's
// contribution and counts it; the reducer of the layer's owner CTA (its position in the processing order, mod G) watches the
// count and, when it is complete, reduces all contributions in a fixed order and releases the
// layer's result words.  Slices that touch a layer boundary are read with ordinary masked loads.
//
// An item depends only on items earlier in the list, every CTA's records are in list order, a
// warp never blocks on a layer's result while it holds unconsumed batches that the result could
// depend on, and all CTAs are co-resident (cooperative launch): the list cannot deadlock.  Every
// wait -- on an mbarrier, on a result word, on a hand-off buffer -- is bounded all the same: when
// one runs out the thread sets DAT_STATUS_TIMEOUT and the CTA's abort flag, every other waiter
// sees it and leaves, each warp waits for its own copies in flight, and the kernel
// returns; the last CTA out clears the dependency counters.
#include <algorithm>
#include <cstdlib>
#include <new>

#include "dat_internal.cuh"

#ifndef F_W
#define F_W 11                                   // compute warps per CTA (with the reducer warp: three warps per scheduler)
#endif
#define F_SLICE 256                              // elements of a tile per compute warp; lane j owns 8j..8j+7
#define FT (F_W * F_SLICE)                       // elements per fused tile
#define F_RB 8                                   // gradient rows per batch
#define F_ROW_BYTES (F_SLICE * 4)
#define F_SLOT_ROWS (F_RB + 2)                   // gradient rows + theta row + momentum row
#define F_SLOT_BYTES (F_SLOT_ROWS * F_ROW_BYTES)
#ifndef F_NSLOT
#define F_NSLOT 2                                // slots per compute warp: one batch in use, one in flight
#endif
#define F_THREADS ((F_W + 1) * 32)               // + the reducer warp
static_assert(F_NSLOT == 2, "the compute warps' loop keeps exactly two batch descriptors");
#define F_KQ 4                                   // hand-off buffers, compute warps -> reducer, Q sums
#define F_KN_MAX 4                               // the same for N sums (M values per warp; as many as fit)
#define F_CTAS_PER_SM 1
#ifndef F_Q_UNROLL
#define F_Q_UNROLL 2                             // rows of a Q batch whose Philox chains the compiler may interleave
#endif
#ifndef F_N_UNROLL
#define F_N_UNROLL 8                             // 16-byte reads of an N batch in flight per lane
#endif
#define F_PRAGMA(x) _Pragma(#x)
#define F_UNROLL(n) F_PRAGMA(unroll n)
#ifndef F_LARGEST_FIRST
#define F_LARGEST_FIRST 1                        // process the layers in descending size
#endif
#ifndef F_L2_HINTS
#define F_L2_HINTS 1                             // L2 eviction policies on the asynchronous copies
#endif
#define F_WAIT_CYCLES (1ll << 31)                // bound of every device-side wait (about a second)

enum { ITEM_N = 0u, ITEM_Q = 1u, ITEM_U = 2u, ITEM_END = 3u };
#define ITEM_TILE_MASK 0x3FFFFFFFu

struct FusedSchedule {
    uint2 *d_recs = nullptr;          // the item records, grouped by CTA
    uint32_t *d_rec_slots = nullptr;  // per record: partial-sum slot
    int64_t *d_cta_first = nullptr;   // G+1: first record of each CTA
    int64_t n_items = 0;
    int64_t *d_slot_base = nullptr;   // h+1, partial-sum slots per layer
    uint32_t *d_expect = nullptr;     // 2h: contributions expected per layer (N, Q)
    int *d_order = nullptr;           // h: processing order, position -> layer
    uint32_t *d_sync = nullptr;       // cnt_n[h] cnt_q[h] done[1]
    unsigned long long *d_flags = nullptr;   // per layer: (epoch, S/nu) (epoch, nu/(S*M)) (epoch, -a_l)
    double *d_npart = nullptr;        // slots * M
    double *d_qpart = nullptr;        // slots * 2
    size_t sync_words = 0;
    int64_t n_slots = 0;
    uint32_t epoch = 0;
    int grid = 0;
    int kn = 1;                       // hand-off buffers for N sums
    int64_t slack = 0;
    int64_t window_bytes = 0;
    size_t smem_bytes = 0;
};

struct FusedArgs {
    GradPtrs gp;
    PhiloxKeys keys;
    float *theta, *mom;
    const int64_t *off, *slot_base, *cta_first;
    const uint2 *recs;
    const uint32_t *rec_slots;                   // per record: partial-sum slot (N, Q items)
    const uint32_t *expect;
    const int *order;                            // processing order: position -> layer
    double *npart, *qpart;
    uint32_t *cnt_n, *cnt_q, *done, *status;
    unsigned long long *flags;                   // 3 words per layer, each (epoch << 32) | float bits
    float *worker_norms, *scales;
    int32_t *code_sum;
    float *norms_out, *scales_out;
    int h, M, kn;
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

// What a warp knows about a batch it has started (registers).
struct Batch {
    uint32_t x = 0;                              // the record's word, with the slice's mode in bits 4-5
    uint32_t aux = 0;                            // rows | chunk << 8 | last << 16
    int pos = 0;                                 // the record's index in the CTA's list (names the slot on a flush)
    long long begin = 0;                         // first element of the warp's slice
    unsigned long long w0 = 0, w1 = 0;           // the layer's result words as they stood when the batch was started
};
enum { MODE_EMPTY = 0u, MODE_FAST = 1u, MODE_MASKED = 2u };

// What the compute warps hand to the reducer warp with a buffer of per-warp sums.
struct RedDesc {
    uint32_t kind;                               // ITEM_N, ITEM_Q or ITEM_END
    int layer;
    long long slot;
};

#ifdef DAT_PROF
// counters (compute warp 0 and the reducer warp of every CTA):
// 0 wait_copy 1 N 2 Q 3 U 4 issue 5 reducer work 6 wait_scale 7 wait_step 8 wait_handoff 9 total
#define PROF_T0() const long long prof_t0 = clock64()
#define PROF_ADD(k) do { if (a.prof && (threadIdx.x == 0 || threadIdx.x == F_W * 32)) sh.prof[(k)] += (unsigned long long)(clock64() - prof_t0); } while (0)
#define PROF_MARK(v) const long long v = clock64()
#define PROF_SPAN(k, v0, v1) do { if (a.prof && threadIdx.x == 0) sh.prof[(k)] += (unsigned long long)((v1) - (v0)); } while (0)
#define PROF_LAYER(layer, col) do { if (a.prof) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); a.prof[296 * 16 + (layer) * 4 + (col)] = t_; } } while (0)
#else
#define PROF_MARK(v) do {} while (0)
#define PROF_SPAN(k, v0, v1) do {} while (0)
#define PROF_LAYER(layer, col) do {} while (0)
#define PROF_T0() do {} while (0)
#define PROF_ADD(k) do {} while (0)
#endif

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

// Fixed part of the shared memory; the slots come before it, the N hand-off buffers after it.
struct Shared {
    unsigned long long nred_full[F_KN_MAX], nred_empty[F_KN_MAX]; // compute warps -> reducer, N sums
    unsigned long long qred_full[F_KQ], qred_empty[F_KQ];         // compute warps -> reducer, Q sums
    RedDesc ndesc[F_KN_MAX], qdesc[F_KQ];
    double red_q[F_KQ][F_W][2];                  // per-warp sums of theta^2 and m'^2
#ifdef DAT_PROF
    unsigned long long prof[16];
#endif
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
// global -> shared asynchronous copy of 16 bytes per lane (both addresses 16-byte aligned);
// the copies of a batch form one group, and a warp waits for its own groups in order.
// `policy` is an L2 eviction policy (createpolicy): what is read for the last time should not push
// out what is still waiting for its second pass.
__device__ __forceinline__ void cp_async16(uint32_t dst_shared, const void *src, unsigned long long policy)
{
#if F_L2_HINTS
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst_shared), "l"(src), "l"(policy) : "memory");
#else
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_shared), "l"(src) : "memory");
#endif
}
struct L2Policies {
    unsigned long long keep, normal, stream;     // evict last / normal / first
};
__device__ __forceinline__ L2Policies make_policies()
{
    L2Policies p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p.keep));
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p.normal));
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p.stream));
    return p;
}
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int PENDING>
__device__ __forceinline__ void cp_async_wait()      // until at most PENDING of this thread's groups are in flight
{
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
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
// Per-layer result words: (epoch << 32) | float bits.  Valid once the epoch matches.
__device__ __forceinline__ unsigned long long ld_acquire64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_release64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ float4 lds128(const unsigned char *p)
{
    return *reinterpret_cast<const float4 *>(p);
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
        __nanosleep(64);
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

// ---- the item list -----------------------------------------------------------------------------
// One 8-byte record per item, written by the host, grouped by CTA in list order:
//   x = kind | flush << 2 | fast << 3 | layer << 8
//   y = (first element of the tile) / 8   (tiles start on multiples of 8: a lane's eight elements
//       share one Philox block)
// and, in a second array read only on a flush, the partial-sum slot of the item (N, Q).
// "fast" = a full tile inside its layer: every slice is moved by asynchronous copies.  In other
// tiles each warp compares its slice with the layer's bounds.  A warp fetches 32 records with
// one coalesced load.
#define REC_FLUSH 4u
#define REC_FAST 8u
#define REC_MODE_SHIFT 4                         // bits 4-5 are free in the record: the batch keeps its mode there

// ---- compute warps: starting batches ---------------------------------------------------------------
// A warp's cursor over the CTA's records, one batch (item, chunk of F_RB workers) at a time.
struct Walk {
    long long first;                             // this CTA's records
    int n;
    int pos = 0, chunk = 0;                      // next batch: record, group of workers
    int win_base = -1;                           // lane j holds record win_base + j
    uint2 win;
    int q_pf_layer = -1, u_pf_layer = -1;        // layers whose result words a started batch already carries
};

enum { ISSUE_OK = 1, ISSUE_NONE = 0, ISSUE_DEFER = -1 };

// Starts the warp's next batch in the slot at shared address `dst` (already offset by 16 bytes
// per lane): every lane copies 16 bytes of each half of each row of the slice (gradient rows of
// the batch's workers; the theta and m rows with an item's last batch), one group per batch.
// `gl` holds, for M <= F_RB, the lane's byte pointers into the gradient buffers.  Nothing here
// waits: the first Q (U) batch of a layer takes along a relaxed read of the layer's scale (step
// length) words, to be looked at when the batch is consumed.  A U batch may be started before its
// layer's step length exists: the m' it copies was written by this very warp when it consumed the
// tile's Q item (a tile's three items go to the same CTA, a slice to the same warp) -- unless that
// Q batch is the one still waiting to be consumed (`pending_q` = its first element, else -1):
// then ISSUE_DEFER is returned and the U batch is started after it.
template <int NCH>
__device__ __forceinline__ int issue_next(const FusedArgs &a, Walk &w, uint32_t dst, long long pending_q, int warp_off, int lane, const char *const (&gl)[F_RB], const char *th_l,
                                          const char *mo_l, const L2Policies &pol, Batch &out)
{
    if (w.pos >= w.n) return ISSUE_NONE;
    if (w.win_base != (w.pos & ~31)) {
        w.win_base = w.pos & ~31;
        w.win = (w.win_base + lane < w.n) ? __ldg(a.recs + w.first + w.win_base + lane) : make_uint2(0, 0);
    }
    const uint32_t x = __shfl_sync(0xFFFFFFFFu, w.win.x, w.pos & 31), y = __shfl_sync(0xFFFFFFFFu, w.win.y, w.pos & 31);
    const uint32_t kind = x & 3u;
    const int layer = (int)(x >> 8);
    const long long s0 = ((long long)y << 3) + warp_off;
    if (kind == ITEM_U && s0 == pending_q) return ISSUE_DEFER;
    out.w0 = 0;
    out.w1 = 0;
    if (kind == ITEM_Q && w.q_pf_layer != layer) {
        w.q_pf_layer = layer;
        out.w0 = ld_relaxed64(a.flags + 3 * (long long)layer);
        out.w1 = ld_relaxed64(a.flags + 3 * (long long)layer + 1);
    } else if (kind == ITEM_U && w.u_pf_layer != layer) {
        w.u_pf_layer = layer;
        out.w0 = ld_relaxed64(a.flags + 3 * (long long)layer + 2);
    }
    uint32_t mode = MODE_FAST;
    if (!(x & REC_FAST)) {
        const long long lo = __ldg(a.off + layer), hi = __ldg(a.off + layer + 1);
        if (s0 >= hi || s0 + F_SLICE <= lo) mode = MODE_EMPTY;
        else if (s0 < lo || s0 + F_SLICE > hi) mode = MODE_MASKED;
    }
    int c = 0, nr = (kind == ITEM_U) ? 0 : a.M;
    bool last = true;
    if (NCH > 1) {
        c = w.chunk;
        nr = (kind == ITEM_U) ? 0 : min(F_RB, a.M - c * F_RB);
        last = (kind == ITEM_U) || (c == (a.M + F_RB - 1) / F_RB - 1);
    }
    out.x = (x & ~((3u << REC_MODE_SHIFT) | (last ? 0u : REC_FLUSH))) | (mode << REC_MODE_SHIFT);
    out.aux = (uint32_t)nr | ((uint32_t)c << 8) | (last ? 0x10000u : 0u);
    out.pos = w.pos;
    out.begin = s0;
    if (mode == MODE_FAST && DAT_CHECK(s0 >= 0 && s0 + F_SLICE <= a.d && (s0 & 7) == 0 && c * F_RB + nr <= a.M, 2, s0)) {
        // N reads a gradient tile for the first time (keep it for the Q pass), Q for the last;
        // theta is read again by the U pass; m (Q) and m' (U) are not read again.
        const long long eb = s0 * 4;
        const unsigned long long pg = (kind == ITEM_N) ? pol.keep : pol.stream;
#pragma unroll
        for (int r = 0; r < F_RB; ++r) {
            if (r < nr) {
                const char *src = (NCH == 1 ? gl[r] : reinterpret_cast<const char *>(a.gp.p[c * F_RB + r]) + lane * 16) + eb;
                cp_async16(dst + r * F_ROW_BYTES, src, pg);
                cp_async16(dst + r * F_ROW_BYTES + F_ROW_BYTES / 2, src + F_ROW_BYTES / 2, pg);
            }
        }
        if (last && kind != ITEM_N) {
            const unsigned long long pt = (kind == ITEM_Q) ? pol.normal : pol.stream;
            cp_async16(dst + F_RB * F_ROW_BYTES, th_l + eb, pt);
            cp_async16(dst + F_RB * F_ROW_BYTES + F_ROW_BYTES / 2, th_l + eb + F_ROW_BYTES / 2, pt);
            cp_async16(dst + (F_RB + 1) * F_ROW_BYTES, mo_l + eb, pol.stream);
            cp_async16(dst + (F_RB + 1) * F_ROW_BYTES + F_ROW_BYTES / 2, mo_l + eb + F_ROW_BYTES / 2, pol.stream);
        }
    }
    cp_async_commit();                           // one group per batch, empty for slices without copies
    if (last) { w.chunk = 0; w.pos++; } else w.chunk = c + 1;
    return ISSUE_OK;
}

// ---- compute warps: consuming batches ---------------------------------------------------------------
// N batch from a slot: lane j adds the exact fp64 squares of quarter (j & 3) of gradient row
// (j >> 2).  The 16-byte reads are rotated by the lane index so that the eight lanes of a
// shared-memory phase hit eight different bank groups.
__device__ __forceinline__ double norm_fast(const unsigned char *slot, int nr, int lane)
{
    const int row = lane >> 2;
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    if (row < nr) {
        const unsigned char *p = slot + row * F_ROW_BYTES + (lane & 3) * (F_ROW_BYTES / 4);
        F_UNROLL(F_N_UNROLL)
        for (int i = 0; i < F_ROW_BYTES / 64; ++i) {
            const float4 f = lds128(p + (((i + lane) & (F_ROW_BYTES / 64 - 1)) << 4));
            s0 = fma((double)f.x, (double)f.x, s0);
            s1 = fma((double)f.y, (double)f.y, s1);
            s2 = fma((double)f.z, (double)f.z, s2);
            s3 = fma((double)f.w, (double)f.w, s3);
        }
    }
    return (s0 + s1) + (s2 + s3);
}

// The same for a slice at a layer boundary: masked scalar loads from global memory.
__device__ __noinline__ double norm_masked(const FusedArgs &a, int chunk, int nr, long long s0, long long lo, long long hi,
                                           int lane)
{
    const int row = lane >> 2;
    double s = 0.0;
    if (row < nr) {
        const float *g = a.gp.p[chunk * F_RB + row];
        const long long e0 = s0 + (lane & 3) * (F_SLICE / 4);
        for (int i = 0; i < F_SLICE / 4; ++i) {
            const long long e = e0 + i;
            if (e >= lo && e < hi) { const float x = g[e]; s = fma((double)x, (double)x, s); }
        }
    }
    return s;
}

// Per-plan constants of the scaled form of Eq. xi used on full slices.  With S + 1 = 2^b,
//   y' = sat(fma(|g|, t 2^-b, u1 2^-b)) = min(fma(|g|, t, u1), S + 1) 2^-b   (scaling by a power of
// two commutes with the rounding), and fma_rz(y', 2^b, 2^23 - 1) = 2^23 + floor(y) - 1 exactly:
// the clamp and the floor ride on the two multiply-adds.  The signed level is then added to a
// float sum (|sum| <= 64 * 65535 < 2^24: exact).  Not valid when t 2^-b is subnormal (norms
// beyond 2^126 / 2^b): such layers take the plain form.
struct QuantConst {
    float two_b, inv_two_b, t_min;               // 2^b, 2^-b, smallest t with t 2^-b normal
    float c0, c1;                                // 16-bit u: u1 2^-b = fma(2^23 + half, c0, c1)
    uint32_t ubits;                              // 23-bit u: exponent bits of u1 2^-b
};

// Q batch from a slot: the gradient rows of the lane's eight consecutive elements e0 .. e0+7.
// One Philox block (16-bit u) or two (23-bit u) per row.
template <bool IDENTITY, bool RNG16, bool FULL>
__device__ __forceinline__ void rows_quant(const FusedArgs &a, const QuantConst &qc, const unsigned char *slot, int chunk,
                                           int nr, long long e0, int lane, float ts, float acc[8])
{
    F_UNROLL(F_Q_UNROLL)
    for (int r = 0; r < F_RB; ++r) {
        if (FULL || r < nr) {
            const float4 f0 = lds128(slot + r * F_ROW_BYTES + lane * 32);
            const float4 f1 = lds128(slot + r * F_ROW_BYTES + lane * 32 + 16);
            const float v[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
            if (IDENTITY) {
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] += v[j];
            } else {
                const uint32_t worker = (uint32_t)(chunk * F_RB + r);
                uint32_t w[8];
                if (RNG16) {
                    dat_random_words((uint64_t)e0 >> 3, worker, a.keys, w);
                } else {
                    dat_random_words((uint64_t)e0 >> 2, worker, a.keys, w);
                    dat_random_words(((uint64_t)e0 >> 2) + 1, worker, a.keys, w + 4);
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float u1s;
                    if (RNG16) {
                        const uint32_t fb = __byte_perm(w[j >> 1], 0x4B000000u, (j & 1) ? 0x7632 : 0x7610);
                        u1s = __fmaf_rn(__uint_as_float(fb), qc.c0, qc.c1);
                    } else {
                        u1s = __uint_as_float(qc.ubits | (w[j] & 0x007FFFFFu));
                    }
                    const float ys = __saturatef(__fmaf_rn(fabsf(v[j]), ts, u1s));
                    const float lf = __fmaf_rz(ys, qc.two_b, 8388607.0f) - 8388608.0f;
                    const float sg = __uint_as_float((__float_as_uint(v[j]) & 0x80000000u) | 0x3F800000u);
                    acc[j] = __fmaf_rn(lf, sg, acc[j]);
                }
            }
        }
    }
}

// The plain form, one row and four elements at a time: for slices at a layer boundary (masked
// global loads, slot == nullptr) and for layers whose scale is outside the range of the scaled form.
template <bool IDENTITY>
__device__ __noinline__ void rows_quant_plain(const FusedArgs &a, const unsigned char *slot, int chunk, int nr,
                                              long long e0, long long lo, long long hi, int lane, float qmul, bool rng16,
                                              float acc[8])
{
    const float S1_f = a.S_f + 1.0f;
#pragma unroll 1
    for (int r = 0; r < nr; ++r) {
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            const long long ee = e0 + 4 * half;
            float v[4];
            if (slot) {
                const float4 f = lds128(slot + r * F_ROW_BYTES + lane * 32 + half * 16);
                v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
            } else {
                dat_load4(a.gp.p[chunk * F_RB + r], ee, lo, hi, v);
            }
            float add[4];
            if (IDENTITY) {
#pragma unroll
                for (int j = 0; j < 4; ++j) add[j] = v[j];
            } else {
                float u1[4];
                dat_u1x4((uint64_t)ee, (uint32_t)(chunk * F_RB + r), a.keys, rng16, u1);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float lf = (float)dat_level_u1(v[j], qmul, S1_f, u1[j]);
                    add[j] = (v[j] < 0.0f) ? -lf : lf;
                }
            }
            if (half == 0) {
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[j] += add[j];
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[4 + j] += add[j];
            }
        }
    }
}

// theta and m of the lane's eight elements: from the slot's last two rows or masked from global memory.
__device__ __forceinline__ void load_params(const FusedArgs &a, const unsigned char *slot, bool fast, long long e0,
                                            long long lo, long long hi, int lane, float th[8], float m[8])
{
    if (fast) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const float4 t4 = lds128(slot + F_RB * F_ROW_BYTES + lane * 32 + 16 * k);
            const float4 m4 = lds128(slot + (F_RB + 1) * F_ROW_BYTES + lane * 32 + 16 * k);
            th[4 * k] = t4.x; th[4 * k + 1] = t4.y; th[4 * k + 2] = t4.z; th[4 * k + 3] = t4.w;
            m[4 * k] = m4.x; m[4 * k + 1] = m4.y; m[4 * k + 2] = m4.z; m[4 * k + 3] = m4.w;
        }
    } else {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            dat_load4(a.theta, e0 + 4 * k, lo, hi, th + 4 * k);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long e = e0 + 4 * k + j;
                m[4 * k + j] = (e >= lo && e < hi) ? __ldcg(a.mom + e) : 0.0f;
            }
        }
    }
}

// One compute warp.  NCH = number of worker groups whose running sums of squares it keeps
// (1 for M <= F_RB, else DAT_MAX_WORKERS / F_RB).
template <bool IDENTITY, int NCH, bool RNG16>
__device__ __forceinline__ void compute_warp(const FusedArgs &a, Shared &sh, unsigned char *slots, double *red_n)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    Walk w;
    w.first = __ldg(a.cta_first + blockIdx.x);
    w.n = (int)(__ldg(a.cta_first + blockIdx.x + 1) - w.first);
    uint32_t nf_n = 0, nf_q = 0;                 // hand-offs to the reducer
    double nacc[NCH];                            // running sums of squares: row (lane >> 2) of each group, quarter (lane & 3)
#pragma unroll
    for (int c = 0; c < NCH; ++c) nacc[c] = 0.0;
    double qss0 = 0.0, qss1 = 0.0;               // running sums of theta^2 and m'^2 until the next flush
    float acc[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};   // signed level sums (or gradient sums) of the item
    int q_layer = -1;                            // layer whose scale this warp has seen
    float q_f[2] = {0.0f, 0.0f};
    float ts = 0.0f;                             // S/nu * 2^-b of that layer
    bool plain = false;                          // that layer's scale is outside the range of the scaled form
    const float Mf = (float)a.M;
    QuantConst qc;
    qc.two_b = a.S_f + 1.0f;
    qc.inv_two_b = 1.0f / qc.two_b;
    qc.t_min = 1.17549435e-38f * qc.two_b;       // 2^-126 * 2^b
    qc.c0 = qc.inv_two_b * (1.0f / 65536.0f);
    qc.c1 = -127.0f * qc.inv_two_b;
    qc.ubits = __float_as_uint(qc.inv_two_b);

    // the lane's view of the inputs: byte pointers offset by its 16 bytes of every half row
    const char *gl[F_RB];
#pragma unroll
    for (int r = 0; r < F_RB; ++r) gl[r] = reinterpret_cast<const char *>(a.gp.p[r < a.M ? r : 0]) + lane * 16;
    const char *th_l = reinterpret_cast<const char *>(a.theta) + lane * 16;
    const char *mo_l = reinterpret_cast<const char *>(a.mom) + lane * 16;
    const int warp_off = warp * F_SLICE;
    const uint32_t slot_u32 = smem_u32(slots) + lane * 16;
    const L2Policies pol = make_policies();

    Batch cur, nxt;                              // the batch being consumed, the one in flight behind it
    uint32_t par = 0;                            // slot of the next batch to start
    int u_layer = -1;                            // layer whose step length this warp has seen
    float u_f = 0.0f;
    bool have_nxt = false;
    for (;;) {
        if (!have_nxt) {                         // nothing in flight: start the batch to work on
            PROF_T0();
            const int r = issue_next<NCH>(a, w, slot_u32 + par * F_SLOT_BYTES, -1, warp_off, lane, gl, th_l, mo_l, pol, nxt);
            PROF_ADD(4);
            if (r != ISSUE_OK) break;            // end of the list
            par ^= 1u;
        }
        cur = nxt;
        {   // start the batch after it, into the slot that the previous round has finished with
            PROF_T0();
            const long long pending_q = ((cur.x & 3u) == ITEM_Q) ? cur.begin : -1;
            have_nxt = issue_next<NCH>(a, w, slot_u32 + par * F_SLOT_BYTES, pending_q, warp_off, lane, gl, th_l, mo_l, pol, nxt) == ISSUE_OK;
            PROF_ADD(4);
            if (have_nxt) par ^= 1u;
        }
        { PROF_T0();
        if (have_nxt) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncwarp();                            // the other lanes' copies of this batch have landed too
        PROF_ADD(0); }
        const unsigned char *sl = slots + (size_t)(par ^ (have_nxt ? 0u : 1u)) * F_SLOT_BYTES;
        const Batch h0 = cur;
        const long long s0 = h0.begin;
        const uint32_t info = h0.x, kind = info & 3u, mode = (info >> REC_MODE_SHIFT) & 3u;
        const int layer = (int)(info >> 8);
        const int chunk = (NCH == 1) ? 0 : (int)((h0.aux >> 8) & 255u), nr = (NCH == 1) ? a.M : (int)(h0.aux & 255u);
        const bool last = (NCH == 1) || (h0.aux & 0x10000u);
        const long long e0 = s0 + 8 * lane;
        long long lo = s0, hi = s0 + F_SLICE;
        if (mode == MODE_MASKED) { lo = __ldg(a.off + layer); hi = __ldg(a.off + layer + 1); }
        if (!DAT_CHECK(kind <= ITEM_U && layer >= 0 && layer < a.h && (kind == ITEM_U || chunk * F_RB + nr <= a.M), 7, info)) { atomicExch(&sh.abort_flag, 1); break; }

        if (kind == ITEM_N) {
            PROF_T0();
            if (mode != MODE_EMPTY) {
                const double s = (mode == MODE_FAST) ? norm_fast(sl, nr, lane) : norm_masked(a, chunk, nr, s0, lo, hi, lane);
#pragma unroll
                for (int c = 0; c < NCH; ++c)
                    if (NCH == 1 || c == chunk) nacc[c] += s;
            }
            PROF_ADD(1);
            if (info & REC_FLUSH) {
                // the CTA's contribution to the layer is due: quarters -> rows, then hand over
                const uint32_t rb = nf_n % (uint32_t)a.kn, ruse = nf_n / (uint32_t)a.kn;
                { PROF_T0();
                if (!wait_mbar(sh, &sh.nred_empty[rb], (ruse & 1u) ^ 1u, a.status)) break;
                PROF_ADD(8); }
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    double v = nacc[c];
                    v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
                    v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
                    const int i = c * F_RB + (lane >> 2);
                    if ((lane & 3) == 0 && i < a.M) red_n[((size_t)rb * F_W + warp) * a.M + i] = v;
                    nacc[c] = 0.0;
                }
                if (threadIdx.x == 0) { sh.ndesc[rb].kind = ITEM_N; sh.ndesc[rb].layer = layer; sh.ndesc[rb].slot = __ldg(a.rec_slots + w.first + h0.pos); }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.nred_full[rb]);
                nf_n++;
            }
        } else if (kind == ITEM_Q) {
            PROF_T0();
            if (chunk == 0) {
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
                if (!IDENTITY && q_layer != layer) {
                    PROF_T0();
                    if ((uint32_t)(h0.w0 >> 32) == a.epoch && (uint32_t)(h0.w1 >> 32) == a.epoch) {
                        q_f[0] = __uint_as_float((uint32_t)h0.w0);       // the words were there when the batch was started
                        q_f[1] = __uint_as_float((uint32_t)h0.w1);
                    } else if (!wait_words(sh, a.flags + 3 * (long long)layer, 2, a.epoch, a.status, q_f)) break;
                    q_layer = layer;
                    ts = q_f[0] * qc.inv_two_b;
                    plain = (q_f[0] != 0.0f) && !(q_f[0] >= qc.t_min && q_f[0] <= 3.402823466e38f);
                    PROF_ADD(6);
                }
            }
            if (mode == MODE_FAST && (IDENTITY || !plain)) {
                if (nr == F_RB) rows_quant<IDENTITY, RNG16, true>(a, qc, sl, chunk, nr, e0, lane, ts, acc);
                else rows_quant<IDENTITY, RNG16, false>(a, qc, sl, chunk, nr, e0, lane, ts, acc);
            } else if (mode != MODE_EMPTY) {
                rows_quant_plain<IDENTITY>(a, mode == MODE_FAST ? sl : nullptr, chunk, nr, e0, lo, hi, lane, q_f[0], RNG16, acc);
            }
            if (last) {
                if (mode != MODE_EMPTY) {
                    float th[8], m[8];
                    load_params(a, sl, mode == MODE_FAST, e0, lo, hi, lane, th, m);
                    if (!IDENTITY && a.code_sum) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (e0 + j >= lo && e0 + j < hi) a.code_sum[e0 + j] = (int)acc[j];
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float ghat = IDENTITY ? acc[j] / Mf : acc[j] * q_f[1];
                        m[j] = __fmaf_rn(a.mu, m[j], __fmaf_rn(a.wd, th[j], ghat));
                        qss0 = fma((double)th[j], (double)th[j], qss0);
                        qss1 = fma((double)m[j], (double)m[j], qss1);
                    }
                    if (DAT_CHECK(lo >= 0 && hi <= a.d && e0 >= 0, 5, e0)) {
                        if (e0 < hi) dat_store4(a.mom, e0, lo, hi, m);
                        if (e0 + 4 < hi) dat_store4(a.mom, e0 + 4, lo, hi, m + 4);
                    }
                }
                if (info & REC_FLUSH) {
                    const double ss0 = dat_warp_sum(qss0), ss1 = dat_warp_sum(qss1);
                    qss0 = 0.0;
                    qss1 = 0.0;
                    const uint32_t rb = nf_q % F_KQ, ruse = nf_q / F_KQ;
                    { PROF_T0();
                    if (!wait_mbar(sh, &sh.qred_empty[rb], (ruse & 1u) ^ 1u, a.status)) break;
                    PROF_ADD(8); }
                    if (lane == 0) { sh.red_q[rb][warp][0] = ss0; sh.red_q[rb][warp][1] = ss1; }
                    if (threadIdx.x == 0) { sh.qdesc[rb].kind = ITEM_Q; sh.qdesc[rb].layer = layer; sh.qdesc[rb].slot = __ldg(a.rec_slots + w.first + h0.pos); }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.qred_full[rb]);
                    nf_q++;
                }
            }
            PROF_ADD(2);
        } else {
            PROF_T0();
            if (u_layer != layer) {
                PROF_T0();
                if ((uint32_t)(h0.w0 >> 32) == a.epoch) {
                    u_f = __uint_as_float((uint32_t)h0.w0);
                } else {
                    float f[2];
                    if (!wait_words(sh, a.flags + 3 * (long long)layer + 2, 1, a.epoch, a.status, f)) break;
                    u_f = f[0];
                }
                u_layer = layer;
                PROF_ADD(7);
            }
            if (mode != MODE_EMPTY) {
                const float na = u_f;
                float th[8], m[8];
                load_params(a, sl, mode == MODE_FAST, e0, lo, hi, lane, th, m);
#pragma unroll
                for (int j = 0; j < 8; ++j) th[j] = __fmaf_rn(na, m[j], th[j]);
                if (DAT_CHECK(lo >= 0 && hi <= a.d && e0 >= 0, 6, e0)) {
                    if (e0 < hi) dat_store4(a.theta, e0, lo, hi, th);
                    if (e0 + 4 < hi) dat_store4(a.theta, e0 + 4, lo, hi, th + 4);
                }
            }
            PROF_ADD(3);
        }
        __syncwarp();                            // every lane is done with the slot before it is refilled
    }

    cp_async_wait<0>();                          // nothing of this warp is in flight when the shared memory is given back
    if (*(volatile int *)&sh.abort_flag) return;
    // tell the reducer that this warp has nothing more to hand over
    if (!IDENTITY) {
        const uint32_t rb = nf_n % (uint32_t)a.kn, ruse = nf_n / (uint32_t)a.kn;
        if (!wait_mbar(sh, &sh.nred_empty[rb], (ruse & 1u) ^ 1u, a.status)) return;
        if (threadIdx.x == 0) sh.ndesc[rb].kind = ITEM_END;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.nred_full[rb]);
    }
    {
        const uint32_t rb = nf_q % F_KQ, ruse = nf_q / F_KQ;
        if (!wait_mbar(sh, &sh.qred_empty[rb], (ruse & 1u) ^ 1u, a.status)) return;
        if (threadIdx.x == 0) sh.qdesc[rb].kind = ITEM_END;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.qred_full[rb]);
    }
}

// ---- reducer warp ----------------------------------------------------------------------------------
// N: add the compute warps' sums in a fixed order, publish the CTA's contribution to the layer
// and count it (no answer needed: the layer's owner watches the count).
__device__ __forceinline__ void finish_norm(const FusedArgs &a, const double *red_n, int layer, long long slot, int buf,
                                            int lane)
{
    if (!DAT_CHECK(slot >= 0 && slot < a.n_slots && layer >= 0 && layer < a.h, 8, slot)) return;
    for (int i = lane; i < a.M; i += 32) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < F_W; ++w) s += red_n[((size_t)buf * F_W + w) * a.M + i];
        a.npart[slot * a.M + i] = s;
    }
    __threadfence();
    __syncwarp();
    if (lane == 0) red_add(a.cnt_n + layer);
}

// The owner of a layer (CTA = its position in the processing order mod G) finalises it once every contribution has arrived:
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
__device__ __forceinline__ void finish_quant(const FusedArgs &a, Shared &sh, int layer, long long slot, int buf, int lane)
{
    if (!DAT_CHECK(slot >= 0 && slot < a.n_slots && layer >= 0 && layer < a.h, 9, slot)) return;
    if (lane < 2) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < F_W; ++w) s += sh.red_q[buf][w][lane];
        a.qpart[slot * 2 + lane] = s;
    }
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
// (position mod G == CTA) as their contribution counts fill up, until both rings have said END and
// every owned layer is done.
__device__ __forceinline__ void reducer(const FusedArgs &a, Shared &sh, const double *red_n, bool have_norm)
{
    const int lane = threadIdx.x & 31;
    uint32_t kn = 0, kq = 0;
    bool done_n = !have_norm, done_q = false;
    // Ownership follows the processing order: this CTA owns the layers at positions c, c + G, ...
    // of that order, so the next one to complete is always the one it looks at.
    int pos_n = have_norm ? (int)blockIdx.x : a.h, pos_q = (int)blockIdx.x;
    int own_n = (pos_n < a.h) ? __ldg(a.order + pos_n) : 0, own_q = (pos_q < a.h) ? __ldg(a.order + pos_q) : 0;
    uint32_t want_n = (pos_n < a.h) ? __ldg(a.expect + own_n) : 0u;
    uint32_t want_q = (pos_q < a.h) ? __ldg(a.expect + a.h + own_q) : 0u;
    long long t_last = clock64();
    uint32_t round = 0;
    while (!(done_n && done_q) || pos_n < a.h || pos_q < a.h) {
        bool progress = false;
        if (!done_n) {
            const uint32_t b = kn % (uint32_t)a.kn;
            if (mbar_test_wait(&sh.nred_full[b], (kn / (uint32_t)a.kn) & 1u)) {
                PROF_T0();
                if (sh.ndesc[b].kind == ITEM_END) done_n = true;
                else {
                    finish_norm(a, red_n, sh.ndesc[b].layer, sh.ndesc[b].slot, (int)b, lane);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.nred_empty[b]);
                }
                kn++;
                progress = true;
                PROF_ADD(5);
            }
        }
        if (!done_q) {
            const uint32_t b = kq % F_KQ;
            if (mbar_test_wait(&sh.qred_full[b], (kq / F_KQ) & 1u)) {
                PROF_T0();
                if (sh.qdesc[b].kind == ITEM_END) done_q = true;
                else {
                    finish_quant(a, sh, sh.qdesc[b].layer, sh.qdesc[b].slot, (int)b, lane);
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
            if (pos_n < a.h && ld_acquire(a.cnt_n + own_n) == want_n) {
                PROF_T0();
                finalize_norm(a, own_n, lane);
                pos_n += (int)gridDim.x;
                own_n = (pos_n < a.h) ? __ldg(a.order + pos_n) : 0;
                want_n = (pos_n < a.h) ? __ldg(a.expect + own_n) : 0u;
                progress = true;
                PROF_ADD(5);
            }
            if (pos_q < a.h && ld_acquire(a.cnt_q + own_q) == want_q) {
                PROF_T0();
                finalize_quant(a, own_q, lane);
                pos_q += (int)gridDim.x;
                own_q = (pos_q < a.h) ? __ldg(a.order + pos_q) : 0;
                want_q = (pos_q < a.h) ? __ldg(a.expect + a.h + own_q) : 0u;
                progress = true;
                PROF_ADD(5);
            }
        }
        if (progress) {
            t_last = clock64();
        } else {
            if (*(volatile int *)&sh.abort_flag || (ld_acquire(a.status) & DAT_STATUS_TIMEOUT)) { atomicExch(&sh.abort_flag, 1); return; }
            if (clock64() - t_last > F_WAIT_CYCLES) { raise_timeout(sh, a.status); return; }
            __nanosleep(400);
        }
    }
}

template <bool IDENTITY, int NCH, bool RNG16>
__global__ void __launch_bounds__(F_THREADS, F_CTAS_PER_SM)
k_fused_step(const __grid_constant__ FusedArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Shared &sh = *reinterpret_cast<Shared *>(smem_raw + (size_t)F_W * F_NSLOT * F_SLOT_BYTES);
    double *red_n = reinterpret_cast<double *>(smem_raw + (size_t)F_W * F_NSLOT * F_SLOT_BYTES + sizeof(Shared));

    if (threadIdx.x == 0) {
        for (int b = 0; b < F_KN_MAX; ++b) { mbar_init(&sh.nred_full[b], F_W); mbar_init(&sh.nred_empty[b], 1); }
        for (int b = 0; b < F_KQ; ++b) { mbar_init(&sh.qred_full[b], F_W); mbar_init(&sh.qred_empty[b], 1); }
#ifdef DAT_PROF
        for (int k = 0; k < 16; ++k) sh.prof[k] = 0;
#endif
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    PROF_T0();
    const int warp = threadIdx.x >> 5;
    if (warp < F_W) compute_warp<IDENTITY, NCH, RNG16>(a, sh, smem_raw + (size_t)warp * F_NSLOT * F_SLOT_BYTES, red_n);
    else reducer(a, sh, red_n, !IDENTITY);
    PROF_ADD(9);
    __syncthreads();
#ifdef DAT_PROF
    if (a.prof && threadIdx.x < 16) a.prof[blockIdx.x * 16 + threadIdx.x] += sh.prof[threadIdx.x];
#endif

    if (threadIdx.x == 0) {
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
    void *ptrs[] = {f->d_recs, f->d_rec_slots, f->d_order, f->d_cta_first, f->d_slot_base, f->d_expect, f->d_sync, f->d_flags, f->d_npart, f->d_qpart};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    delete f;
    plan->fused = nullptr;
}

// The item list: three pointers walk the layers in order.  N runs ahead; a Q tile may be
// emitted once every N tile of its layer was emitted at least `slack` N-items ago (time for the
// stragglers, the reduction and the result words to land), and N may not run more than `max_lag`
// tiles ahead of Q (what L2 can keep) unless Q itself is waiting; U follows Q in the same way.
// Eligible kinds are emitted in turn, so that HBM streaming (N) and the L2/ALU-bound work (Q, U)
// interleave one to one.  Inside a layer N and U walk the tiles upwards and Q downwards: what a
// pass touched last is what the next pass over the layer touches first.
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
        if (q_ok) {
            const int64_t tile = identity ? q : tile_base[lq] + (tile_base[lq + 1] - 1 - q);
            items.push_back(((uint32_t)ITEM_Q << 30) | (uint32_t)tile);
            q++;
        }
        if (u_ok) {
            const int64_t tile = identity ? tile_base[lu] + (tile_base[lu + 1] - 1 - u) : u;
            items.push_back(((uint32_t)ITEM_U << 30) | (uint32_t)tile);
            u++;
        }
    }
}

template <typename T>
static cudaError_t upload(T **dst, const std::vector<T> &src)
{
    cudaError_t e = cudaMalloc((void **)dst, std::max<size_t>(src.size(), 1) * sizeof(T));
    if (e != cudaSuccess) return e;
    return cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
}

static const void *fused_kernel(const dat_plan_t *plan)
{
    if (plan->bits == 32)       // more than F_RB workers: an item is taken in groups of F_RB rows
        return plan->M <= F_RB ? (const void *)k_fused_step<true, 1, false> : (const void *)k_fused_step<true, DAT_MAX_WORKERS / F_RB, false>;
    const bool rng16 = (plan->rng_bits == 16);
    if (plan->M <= F_RB) return rng16 ? (const void *)k_fused_step<false, 1, true> : (const void *)k_fused_step<false, 1, false>;
    return rng16 ? (const void *)k_fused_step<false, DAT_MAX_WORKERS / F_RB, true>
                 : (const void *)k_fused_step<false, DAT_MAX_WORKERS / F_RB, false>;
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

    // shared memory: the slots, the fixed part, and as many N hand-off buffers as still fit
    int smem_sm = 0, smem_reserved = 0;
    cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, plan->device);
    cudaDeviceGetAttribute(&smem_reserved, cudaDevAttrReservedSharedMemoryPerBlock, plan->device);
    const size_t fixed = (size_t)F_W * F_NSLOT * F_SLOT_BYTES + sizeof(Shared);
    const size_t per_cta = (size_t)smem_sm / F_CTAS_PER_SM > (size_t)smem_reserved ? (size_t)smem_sm / F_CTAS_PER_SM - smem_reserved : 0;
    const size_t one_kn = (size_t)F_W * plan->M * sizeof(double);
    if (per_cta < fixed + one_kn) return DAT_ERR_UNSUPPORTED;
    f->kn = (int)std::min<size_t>((per_cta - fixed) / one_kn, F_KN_MAX);
    f->smem_bytes = fixed + (size_t)f->kn * one_kn;

    int l2 = 0;
    cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, plan->device);
    f->window_bytes = l2 > 0 ? (int64_t)l2 / 5 * 8 : (int64_t)128 << 20;      // N leads Q by at most 1.6 x L2 of gradient rows
    f->slack = 8 * (int64_t)G;
#ifdef DAT_PROF
    if (const char *e = getenv("DAT_FUSED_WINDOW_MB")) f->window_bytes = (int64_t)atoi(e) << 20;
    if (const char *e = getenv("DAT_FUSED_SLACK")) f->slack = atoi(e);
#endif

    std::vector<uint32_t> items;
    std::vector<int64_t> tile_base(h + 1), slot_base(h + 1);
    std::vector<uint32_t> expect(2 * h, 0);
    try {
        // Layers are processed largest first (results do not depend on the order): the end of the
        // list, where Q and U have no N left to overlap with, then belongs to the small layers.
        std::vector<int64_t> ntiles(h), order(h);
        int64_t nt = 0, ns = 0;
        for (int64_t l = 0; l < h; ++l) {
            slot_base[l] = ns;
            const int64_t a = plan->offsets[l] & ~(int64_t)7;
            ntiles[l] = (plan->offsets[l + 1] - a + FT - 1) / FT;
            ns += std::min<int64_t>(ntiles[l], G);
            order[l] = l;
        }
#if F_LARGEST_FIRST
        std::stable_sort(order.begin(), order.end(), [&](int64_t x, int64_t y) { return ntiles[x] > ntiles[y]; });
#endif
        for (int64_t k = 0; k < h; ++k) {           // tile_base is indexed by position in the processing order
            tile_base[k] = nt;
            nt += ntiles[order[k]];
        }
        tile_base[h] = nt;
        slot_base[h] = ns;
        f->n_slots = ns;
        if (nt > (int64_t)ITEM_TILE_MASK || plan->d > ((int64_t)1 << 35)) return DAT_ERR_UNSUPPORTED;   // records hold element / 8 in 32 bits

        // how far N may run ahead of Q (measured: the step is fastest when N is not held back to L2 size)
        const int64_t tile_bytes = (int64_t)FT * 4 * plan->M;
        const int64_t max_lag = std::max<int64_t>(f->window_bytes / tile_bytes, 2 * (int64_t)G);
        items.reserve((size_t)nt * 3);
        build_items(items, tile_base, h, identity, f->slack, max_lag);

        // Records, grouped by CTA: a tile's items all go to CTA (tile mod G), in list order.  For
        // N and Q items the record names the slot of the CTA's running sums: layers with at most
        // G tiles use one slot per tile and flush at once; in larger layers a CTA accumulates over
        // its tiles of the layer and flushes with its last one (slot = the CTA's index).
        // expect[] counts the flushes.
        auto layer_of = [&](int64_t tile) {
            return (int64_t)(std::upper_bound(tile_base.begin(), tile_base.end(), tile) - tile_base.begin()) - 1;
        };
        const int64_t n_items = (int64_t)items.size();
        std::vector<int64_t> cta_first((size_t)G + 1, 0), fill((size_t)G, 0);
        for (int64_t i = 0; i < n_items; ++i) cta_first[(items[i] & ITEM_TILE_MASK) % G + 1]++;
        for (int c = 0; c < G; ++c) cta_first[c + 1] += cta_first[c];
        std::vector<uint2> recs((size_t)n_items);
        std::vector<uint32_t> rec_slots((size_t)n_items, 0u);
        std::vector<int64_t> last_rec[2] = {std::vector<int64_t>((size_t)G, -1), std::vector<int64_t>((size_t)G, -1)};
        std::vector<int> last_layer[2] = {std::vector<int>((size_t)G, -1), std::vector<int>((size_t)G, -1)};
        for (int64_t i = 0; i < n_items; ++i) {
            const uint32_t type = items[i] >> 30;
            const int64_t tile = items[i] & ITEM_TILE_MASK;
            const int cta = (int)(tile % G);
            const int64_t r = cta_first[cta] + fill[cta]++;
            const int64_t k_pos = layer_of(tile);
            const int l = (int)order[k_pos];
            const int64_t lo = plan->offsets[l], hi = plan->offsets[l + 1];
            const int64_t begin = (lo & ~(int64_t)7) + (tile - tile_base[k_pos]) * FT;
            const bool fast = begin >= lo && begin + FT <= hi;
            uint32_t info = type | (fast ? REC_FAST : 0u) | ((uint32_t)l << 8);
            uint32_t slot = 0;
            if (type != ITEM_U) {
                const int k = (type == ITEM_N) ? 0 : 1;
                const int64_t ntl = ntiles[l];
                if (last_rec[k][cta] >= 0 && last_layer[k][cta] != l) {     // the CTA moved on to another layer
                    recs[last_rec[k][cta]].x |= REC_FLUSH;
                    expect[k * h + last_layer[k][cta]]++;
                    last_rec[k][cta] = -1;
                }
                if (ntl <= G) {
                    slot = (uint32_t)(slot_base[l] + (tile - tile_base[k_pos]));
                    info |= REC_FLUSH;
                    expect[k * h + l]++;
                } else {
                    slot = (uint32_t)(slot_base[l] + cta);
                    last_rec[k][cta] = r;
                    last_layer[k][cta] = l;
                }
            }
            recs[r] = make_uint2(info, (uint32_t)(begin >> 3));
            rec_slots[r] = slot;
        }
        for (int k = 0; k < 2; ++k)
            for (int c = 0; c < G; ++c)
                if (last_rec[k][c] >= 0) { recs[last_rec[k][c]].x |= REC_FLUSH; expect[k * h + last_layer[k][c]]++; }
        if (ns > 0xFFFFFFFFll || h >= (1 << 24)) return DAT_ERR_UNSUPPORTED;
        f->n_items = n_items;
        f->sync_words = (size_t)h * 2 + 64;
        cudaError_t e = upload(&f->d_recs, recs);
        if (e == cudaSuccess) e = upload(&f->d_rec_slots, rec_slots);
        if (e == cudaSuccess) e = upload(&f->d_cta_first, cta_first);
        if (e == cudaSuccess) e = upload(&f->d_slot_base, slot_base);
        if (e == cudaSuccess) e = upload(&f->d_expect, expect);
        if (e == cudaSuccess) { std::vector<int> order32(order.begin(), order.end()); e = upload(&f->d_order, order32); }
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

    const void *fn = fused_kernel(plan);
    DAT_CUDA(plan, cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)f->smem_bytes));
    int per_sm = 0;
    DAT_CUDA(plan, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, F_THREADS, f->smem_bytes));
    if (per_sm < F_CTAS_PER_SM) return DAT_ERR_UNSUPPORTED;      // the list needs all CTAs resident
    return DAT_OK;
}

extern "C" int dat_step_sweep(dat_plan_t *plan, float *theta, float *mom, const float *const *grads,
                              uint64_t seed, uint64_t step, const dat_hparams_t *hp,
                              int32_t *code_sum_out, float *layer_norms_out, float *scales_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta || !mom || !hp) return DAT_ERR_ARG;
    if (plan->scale_mode != DAT_SCALE_SHARED_MAX && plan->bits != 32) return DAT_ERR_UNSUPPORTED;   // the fused sweep sums integer codes
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
    a.rec_slots = f->d_rec_slots;
    a.expect = f->d_expect;
    a.order = f->d_order;
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
    a.kn = f->kn;
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
    DAT_CUDA(plan, cudaLaunchCooperativeKernel(fused_kernel(plan), dim3((unsigned)f->grid), dim3(F_THREADS), params,
                                               f->smem_bytes, (cudaStream_t)stream));
    plan->launches++;
    return DAT_OK;
}
