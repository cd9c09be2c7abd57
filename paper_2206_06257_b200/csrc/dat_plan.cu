// Plan object, argument validation, status word and the host-buffer entry point.
#include <cmath>
#include <new>

#include "dat_internal.cuh"

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool dat_aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int dat_cuda_fail(dat_plan_t *plan, cudaError_t e)
{
    if (plan) plan->last_cuda = (int)e;
    (void)cudaGetLastError();   // clear the sticky-less error state for the next call
    return DAT_ERR_CUDA;
}

int dat_check_plan(dat_plan_t *plan)
{
    if (!plan) return DAT_ERR_ARG;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return dat_cuda_fail(plan, e);
    if (dev != plan->device) return DAT_ERR_ARG;
    return DAT_OK;
}

int dat_check_grads(const dat_plan_t *plan, const float *const *grads, GradPtrs *out)
{
    if (!grads) return DAT_ERR_ARG;
    for (int i = 0; i < plan->M; ++i) {
        if (!grads[i]) return DAT_ERR_ARG;
        if (!dat_aligned16(grads[i])) return DAT_ERR_ALIGN;
        out->p[i] = grads[i];
    }
    for (int i = plan->M; i < DAT_MAX_WORKERS; ++i) out->p[i] = nullptr;
    return DAT_OK;
}

LambConst dat_lamb_const(const dat_lamb_hparams_t *hp, int64_t t)
{
    LambConst c;
    c.beta1 = hp->beta1;
    c.beta2 = hp->beta2;
    c.om1 = 1.0f - hp->beta1;
    c.om2 = 1.0f - hp->beta2;
    c.bc1 = (float)(1.0 - pow((double)hp->beta1, (double)t));      // 1 - beta^t in double, rounded once
    c.bc2 = (float)(1.0 - pow((double)hp->beta2, (double)t));
    c.zeta = hp->zeta;
    c.wd = hp->weight_decay;
    return c;
}

PhiloxKeys dat_make_keys(uint64_t seed, uint64_t step)
{
    PhiloxKeys k;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)step;
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = k0;
        k.k1[r] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    k.seed_hi = (uint32_t)(seed >> 32);
    return k;
}

extern "C" int dat_plan_create(dat_plan_t **out, int64_t num_layers, const int64_t *layer_offsets,
                               int num_workers, int bits, int scale_mode, int rng_bits)
{
    if (!out) return DAT_ERR_ARG;
    *out = nullptr;
    if (!layer_offsets || num_layers < 1 || num_layers > (1 << 24)) return DAT_ERR_ARG;
    if (num_workers < 1 || num_workers > DAT_MAX_WORKERS) return DAT_ERR_ARG;
    if (!(bits == 1 || bits == 2 || bits == 4 || bits == 8 || bits == 16 || bits == 32)) return DAT_ERR_BITS;
    if (scale_mode != DAT_SCALE_SHARED_MAX && scale_mode != DAT_SCALE_PER_WORKER) return DAT_ERR_ARG;
    if (rng_bits != DAT_RNG_BITS_16 && rng_bits != DAT_RNG_BITS_23) return DAT_ERR_ARG;
    if (layer_offsets[0] != 0) return DAT_ERR_LAYOUT;
    for (int64_t l = 0; l < num_layers; ++l)
        if (layer_offsets[l + 1] <= layer_offsets[l]) return DAT_ERR_LAYOUT;
    if (layer_offsets[num_layers] > ((int64_t)1 << 40)) return DAT_ERR_ARG;

    dat_plan_t *p = new (std::nothrow) dat_plan_t();
    if (!p) return DAT_ERR_NOMEM;
    cudaError_t e = cudaGetDevice(&p->device);
    if (e != cudaSuccess) { delete p; (void)cudaGetLastError(); return DAT_ERR_CUDA; }
    e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
    if (e != cudaSuccess) { delete p; (void)cudaGetLastError(); return DAT_ERR_CUDA; }

    p->h = num_layers;
    p->d = layer_offsets[num_layers];
    p->M = num_workers;
    p->bits = bits;
    p->scale_mode = scale_mode;
    p->rng_bits = rng_bits;
    p->S = (bits == 32) ? 0u : (uint32_t)((1ull << bits) - 1ull);
    try {
        p->offsets.assign(layer_offsets, layer_offsets + num_layers + 1);
        p->tile_base.resize(num_layers + 1);
    } catch (...) { delete p; return DAT_ERR_NOMEM; }
    int64_t nt = 0;
    for (int64_t l = 0; l < num_layers; ++l) {
        p->tile_base[l] = nt;
        const int64_t a = p->offsets[l] & ~(int64_t)3;
        nt += (p->offsets[l + 1] - a + DAT_TILE - 1) / DAT_TILE;
    }
    p->tile_base[num_layers] = nt;
    p->n_tiles = nt;
    const int eff_bits = (bits == 32) ? 0 : bits;
    p->level_bytes = (int64_t)align_up((size_t)((p->d * eff_bits + 7) / 8), 16);
    p->sign_bytes = (bits == 32) ? 0 : (int64_t)align_up((size_t)((p->d + 7) / 8), 16);

    // carve the workspace
    const size_t h1 = (size_t)num_layers + 1, h = (size_t)num_layers;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t o_off = take(h1 * 8), o_tb = take(h1 * 8);
    const size_t o_part = take((size_t)nt * (size_t)(num_workers > 2 ? num_workers : 2) * 8);
    const size_t o_wn = take((size_t)num_workers * h * 4);
    const size_t o_sc = take(h * 4), o_qm = take((size_t)num_workers * h * 4), o_dq = take(h * 4), o_sa = take(h * 4);
    const size_t o_nr = take(2 * h * 4), o_st = take(256);
    p->ws_bytes = off;
    e = cudaMalloc((void **)&p->ws, p->ws_bytes);
    if (e != cudaSuccess) { delete p; (void)cudaGetLastError(); return DAT_ERR_NOMEM; }
    p->d_offsets = (int64_t *)(p->ws + o_off);
    p->d_tile_base = (int64_t *)(p->ws + o_tb);
    p->d_partials = (double *)(p->ws + o_part);
    p->d_worker_norms = (float *)(p->ws + o_wn);
    p->d_scales = (float *)(p->ws + o_sc);
    p->d_qmul = (float *)(p->ws + o_qm);
    p->d_dq = (float *)(p->ws + o_dq);
    p->d_step_a = (float *)(p->ws + o_sa);
    p->d_norms = (float *)(p->ws + o_nr);
    p->d_status = (uint32_t *)(p->ws + o_st);
    e = cudaMemset(p->ws, 0, p->ws_bytes);
    if (e == cudaSuccess) e = cudaMemcpy(p->d_offsets, p->offsets.data(), h1 * 8, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(p->d_tile_base, p->tile_base.data(), h1 * 8, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(p->ws);
        delete p;
        (void)cudaGetLastError();
        return DAT_ERR_CUDA;
    }
    const int rc = dat_pipe_build(p);
    if (rc != DAT_OK) {
        dat_pipe_destroy(p);
        cudaFree(p->ws);
        delete p;
        return rc;
    }
    *out = p;
    return DAT_OK;
}

extern "C" int dat_plan_set_origin(dat_plan_t *plan, int64_t elem_base, int64_t worker_base)
{
    if (!plan || elem_base < 0 || (elem_base & 7) || worker_base < 0 || worker_base + plan->M > ((int64_t)1 << 32)) return DAT_ERR_ARG;
    plan->elem_base = elem_base;
    plan->worker_base = (uint32_t)worker_base;
    return DAT_OK;
}

extern "C" int dat_plan_destroy(dat_plan_t *plan)
{
    if (!plan) return DAT_OK;
    int rc = DAT_OK;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != plan->device) cudaSetDevice(plan->device);
    if (cudaDeviceSynchronize() != cudaSuccess) rc = DAT_ERR_CUDA;
    dat_pipe_destroy(plan);
    if (plan->stage) cudaFree(plan->stage);
    if (plan->d_tile_base8) cudaFree(plan->d_tile_base8);
    if (plan->d_partials8) cudaFree(plan->d_partials8);
    if (plan->ws) cudaFree(plan->ws);
    if (prev >= 0 && prev != plan->device) cudaSetDevice(prev);
    (void)cudaGetLastError();
    delete plan;
    return rc;
}

extern "C" int dat_plan_sizes(const dat_plan_t *plan, int64_t *level_bytes_per_worker,
                              int64_t *sign_bytes_per_worker, int64_t *num_scales,
                              int64_t *workspace_bytes)
{
    if (!plan) return DAT_ERR_ARG;
    if (level_bytes_per_worker) *level_bytes_per_worker = plan->level_bytes;
    if (sign_bytes_per_worker) *sign_bytes_per_worker = plan->sign_bytes;
    if (num_scales) *num_scales = (plan->scale_mode == DAT_SCALE_PER_WORKER) ? plan->h * plan->M : plan->h;
    if (workspace_bytes) *workspace_bytes = (int64_t)plan->ws_bytes;
    return DAT_OK;
}

extern "C" int dat_get_status(dat_plan_t *plan, uint32_t *flags_out, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!flags_out) return DAT_ERR_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    uint32_t v = 0;
    DAT_CUDA(plan, cudaMemcpyAsync(&v, plan->d_status, sizeof v, cudaMemcpyDeviceToHost, s));
    DAT_CUDA(plan, cudaMemsetAsync(plan->d_status, 0, sizeof v, s));
    DAT_CUDA(plan, cudaStreamSynchronize(s));
    if (v & DAT_STATUS_TIMEOUT) {       // the call that gave up left its counters mid-way
        DAT_CUDA(plan, dat_pipe_reset(plan, s));
        DAT_CUDA(plan, cudaStreamSynchronize(s));
    }
    *flags_out = v;
    return DAT_OK;
}

extern "C" int64_t dat_plan_launch_count(const dat_plan_t *plan) { return plan ? plan->launches : 0; }

extern "C" int dat_last_cuda_error(const dat_plan_t *plan) { return plan ? plan->last_cuda : 0; }

extern "C" const char *dat_strerror(int code)
{
    switch (code) {
    case DAT_OK: return "ok";
    case DAT_ERR_ARG: return "invalid argument (null pointer, size or value out of range, wrong device)";
    case DAT_ERR_ALIGN: return "device pointer is not 16-byte aligned";
    case DAT_ERR_BITS: return "bits must be one of 1, 2, 4, 8, 16 (or 32 where no codes are involved)";
    case DAT_ERR_LAYOUT: return "layer offsets must start at 0 and increase strictly";
    case DAT_ERR_CUDA: return "a CUDA runtime call failed";
    case DAT_ERR_NOMEM: return "out of memory";
    case DAT_ERR_UNSUPPORTED: return "not implemented in this build";
    case DAT_ERR_TOO_LARGE: return "problem exceeds the fixed capacity of this entry point (see DAT_STATIC_MAX_*)";
    default: return "unknown error code";
    }
}

extern "C" int dat_step_host(dat_plan_t *plan, float *theta_host, float *mom_host,
                             const float *const *grads_host, uint64_t seed, uint64_t step,
                             const dat_hparams_t *hp, void *stream)
{
    int rc = dat_check_plan(plan);
    if (rc != DAT_OK) return rc;
    if (!theta_host || !mom_host || !grads_host || !hp) return DAT_ERR_ARG;
    for (int i = 0; i < plan->M; ++i)
        if (!grads_host[i]) return DAT_ERR_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    // every staged vector starts on a 256-byte boundary
    const size_t stride = align_up((size_t)plan->d * 4, 256) / 4;
    if (!plan->stage) {
        cudaError_t e = cudaMalloc((void **)&plan->stage, (size_t)(plan->M + 2) * stride * 4);
        if (e != cudaSuccess) { plan->stage = nullptr; plan->last_cuda = (int)e; (void)cudaGetLastError(); return DAT_ERR_NOMEM; }
    }
    const size_t bytes = (size_t)plan->d * 4;
    float *d_theta = plan->stage, *d_mom = plan->stage + stride;
    const float *d_grads[DAT_MAX_WORKERS];
    DAT_CUDA(plan, cudaMemcpyAsync(d_theta, theta_host, bytes, cudaMemcpyHostToDevice, s));
    DAT_CUDA(plan, cudaMemcpyAsync(d_mom, mom_host, bytes, cudaMemcpyHostToDevice, s));
    for (int i = 0; i < plan->M; ++i) {
        float *g = plan->stage + (size_t)(i + 2) * stride;
        DAT_CUDA(plan, cudaMemcpyAsync(g, grads_host[i], bytes, cudaMemcpyHostToDevice, s));
        d_grads[i] = g;
    }
    rc = dat_step(plan, d_theta, d_mom, d_grads, seed, step, hp, nullptr, nullptr, nullptr, stream);
    if (rc != DAT_OK) return rc;
    DAT_CUDA(plan, cudaMemcpyAsync(theta_host, d_theta, bytes, cudaMemcpyDeviceToHost, s));
    DAT_CUDA(plan, cudaMemcpyAsync(mom_host, d_mom, bytes, cudaMemcpyDeviceToHost, s));
    DAT_CUDA(plan, cudaStreamSynchronize(s));
    return DAT_OK;
}
