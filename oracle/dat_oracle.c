/*
 * dat_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-threaded CPU statement of the data-parallel hot path of
 * the outer-minimisation step of Distributed Adversarial Training (DAT):
 *
 *   M workers' per-layer fp32 gradients
 *     -> randomized b-bit quantizer Q(.)            (Appendix "Additional details on
 *                                                     gradient quantization", Eq. rand_q, Eq. xi;
 *                                                     Algorithm A1 Step 7)
 *     -> aggregation g_hat = (1/M) sum_i Q(g^(i))   (Algorithm A1 Step 9, Eq. grad_agg)
 *     -> layer-wise adaptive learning rate update   (Eq. ada_learn / Eq. 3; Algorithm A1
 *                                                     Step 12, Eq. outer_min)
 *
 * Only the tests, the smoke check and the CPU-baseline timing may call this file.
 * It shares no code, header, table or constant generator with the CUDA path.
 *
 * Every function follows the algorithm's steps in the paper's order, element by
 * element; there is no blocking, fusion or reordering.  Build WITHOUT fast-math and
 * with floating-point contraction off (see oracle/build.py): each fp32 operation
 * written below is exactly one IEEE-754 round-to-nearest operation, and fmaf() is
 * used only where a fused multiply-add is meant.
 *
 * Conventions fixed here where the paper is silent or inconsistent (each is also
 * listed with its reason in the design notes of the repository):
 *   R1  2^b levels {0,...,S}, S = 2^b - 1, grid step 1/S (the paper says "s = 2^b
 *       levels" but its xi takes s+1 values; b bits hold exactly 2^b values).
 *   R2  One quantizer norm per layer (a "layer" is one tensor of the caller's offset
 *       table).  Default mode SHARED_MAX: nu_l = max_i ||g_l^(i)||_2, so that the M
 *       workers' integer codes live on one grid and can be summed as integers.
 *       PER_WORKER mode is Eq. grad_agg / Eq. rand_q taken literally per layer.
 *   R3  Randomness: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), keyed on
 *       (seed, step, worker, element); 23-bit uniform u from the low 23 bits of the
 *       element's word; level = floor(x + u), evaluated as floor(x + (1 + u)) - 1.
 *   R4  Descent direction u_t (which Eq. 3 leaves to "the optimizer employed"):
 *       heavy-ball momentum with coupled weight decay, u = m' = mu*m + g_hat + wd*theta.
 *   R5  Zero norms: tau(0) = c_l (0 by default, so an all-zero tensor does not move);
 *       ||u_l|| = 0 gives ratio 0; nu = 0 gives all levels 0.
 *   R6  tau uses the OLD parameters theta_t, as Eq. 3 is written.
 *
 * Pins (tests/test_oracle_*.py): Philox known-answer vectors; level in
 * {floor(x), floor(x)+1}; exact cases (power-of-two single element, S^2 equal
 * elements); unbiasedness and the QSGD variance bound by Monte Carlo; scale
 * invariance under 2^k; b = 32 equals the worker average; M = 1; the LALR closed
 * form on hand-sized layers and the step-length invariant; zero-norm conventions;
 * bit budget; pack/unpack against numpy.packbits.
 * The exact fp32 rounding order of the quantizer's x = |g|*S/nu, of the dequantize
 * factor and of the update is a choice of this file: "parity unpinned" for those
 * last-bit choices (the paper fixes none).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define DAT_ORACLE_SCALE_SHARED_MAX 0
#define DAT_ORACLE_SCALE_PER_WORKER 1

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (published definition, SC'11 paper, Sec. 3.3 and Table 2).   */
/* ------------------------------------------------------------------------- */

void dat_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2],
                              uint32_t out[4])
{
    const uint32_t mult0 = 0xD2511F53u, mult1 = 0xCD9E8D57u;   /* round multipliers */
    const uint32_t weyl0 = 0x9E3779B9u, weyl1 = 0xBB67AE85u;   /* key schedule      */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += weyl0; k1 += weyl1; }
        uint64_t p0 = (uint64_t)mult0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)mult1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32 random bits of element e (global index in the flat parameter vector) of
 * worker `worker` at (seed, step).  Four consecutive elements share one Philox
 * block: counter = (lo(e/4), hi(e/4), worker, hi(seed)), key = (lo(seed), step).   */
uint32_t dat_oracle_random_word(uint64_t seed, uint64_t step, uint32_t worker, uint64_t e)
{
    uint64_t q = e >> 2;
    uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), worker, (uint32_t)(seed >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)step };
    uint32_t out[4];
    dat_oracle_philox4x32_10(ctr, key, out);
    return out[e & 3u];
}

/* 1 + u, with u uniform on {0, 2^-23, ..., 1 - 2^-23} taken from the low 23 bits of a word:
 * the bits become the mantissa of a float in [1, 2) (exact, no arithmetic). */
float dat_oracle_uniform12(uint32_t w)
{
    uint32_t bits = 0x3F800000u | (w & 0x007FFFFFu);
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

/* The quantizer's random number 1 + u of element e of `worker` at (seed, step), for the two
 * resolutions of u the method is run with (the paper fixes neither generator nor resolution):
 *   rng_bits = 23: u = (low 23 bits of dat_oracle_random_word) / 2^23 -- one Philox block per
 *                  four consecutive elements;
 *   rng_bits = 16: one Philox block per EIGHT consecutive elements: counter
 *                  (lo(e/8), hi(e/8), worker, hi(seed)), same key; element e takes word
 *                  (e/2) mod 4, its low half if e is even and its high half if e is odd;
 *                  u = half / 2^16 (exact in a float).
 * P(level rounds up) then matches the fractional part of x to within 2^-23 resp. 2^-16.      */
float dat_oracle_uniform12_at(uint64_t seed, uint64_t step, uint32_t worker, uint64_t e, int rng_bits)
{
    if (rng_bits != 16)
        return dat_oracle_uniform12(dat_oracle_random_word(seed, step, worker, e));
    uint64_t q = e >> 3;
    uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), worker, (uint32_t)(seed >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)step };
    uint32_t out[4];
    dat_oracle_philox4x32_10(ctr, key, out);
    uint32_t w = out[(e >> 1) & 3u];
    uint32_t half = (e & 1u) ? (w >> 16) : (w & 0xFFFFu);
    return 1.0f + (float)half * (1.0f / 65536.0f);
}

/* ------------------------------------------------------------------------- */
/* S1: quantizer norms.  ||g||_2 of Eq. rand_q, one per (worker, layer).       */
/* ------------------------------------------------------------------------- */

/* worker_norms[i*h + l] = (float) sqrt( sum_j (double)g_j^2 ), j ascending.     */
void dat_oracle_worker_norms(int64_t h, const int64_t *offsets, int64_t l0, int64_t l1,
                             int M, const float *const *grads, float *worker_norms)
{
    for (int i = 0; i < M; ++i)
        for (int64_t l = l0; l < l1; ++l) {
            double ss = 0.0;
            for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e) {
                double g = (double)grads[i][e];
                ss += g * g;
            }
            worker_norms[(int64_t)i * h + l] = (float)sqrt(ss);
        }
}

/* The scales the quantizer uses.  SHARED_MAX: scales[l] = max_i norm(i,l) (h values).
 * PER_WORKER: scales[i*h + l] = norm(i,l) (M*h values).                             */
void dat_oracle_scales(int64_t h, int64_t l0, int64_t l1, int M, int scale_mode,
                       const float *worker_norms, float *scales)
{
    for (int64_t l = l0; l < l1; ++l) {
        if (scale_mode == DAT_ORACLE_SCALE_PER_WORKER) {
            for (int i = 0; i < M; ++i)
                scales[(int64_t)i * h + l] = worker_norms[(int64_t)i * h + l];
        } else {
            float nu = worker_norms[l];
            for (int i = 1; i < M; ++i) {
                float v = worker_norms[(int64_t)i * h + l];
                if (v > nu) nu = v;
            }
            scales[l] = nu;
        }
    }
}

static float scale_of(const float *scales, int scale_mode, int64_t h, int i, int64_t l)
{
    return (scale_mode == DAT_ORACLE_SCALE_PER_WORKER) ? scales[(int64_t)i * h + l] : scales[l];
}

/* ------------------------------------------------------------------------- */
/* S2: the randomized quantizer (Eq. rand_q, Eq. xi), element by element.      */
/* ------------------------------------------------------------------------- */

/* With S = 2^b - 1 and x = S*|g_e|/nu in [0, S]: xi = level/S where
 * level = floor(x) + 1 with probability x - floor(x), else floor(x).
 * Drawn as level = floor(x + u), u uniform on [0,1).  The random bits give u1 = 1 + u
 * directly, so the draw is written level = floor(x + u1) - 1; x + u1 is ONE fused
 * operation fmaf(|g|, S/nu, u1), so x itself is never rounded.  The clamp (of x + u1 to
 * S + 1, i.e. of the level to S) covers the two ways the sum can exceed it: rounding at
 * x = S, and caller-supplied scales smaller than max|g|.
 * level[i][e] in {0..S}; neg[i][e] = 1 iff g < 0 (so -0.0 and NaN give 0).       */
void dat_oracle_quantize(int64_t h, const int64_t *offsets, int64_t l0, int64_t l1,
                         int M, int bits, int scale_mode,
                         const float *const *grads, uint64_t seed, uint64_t step, int rng_bits,
                         const float *scales,
                         uint32_t *const *level, uint8_t *const *neg)
{
    const uint32_t S = (uint32_t)((1ull << bits) - 1ull);
    const float S_f = (float)S;
    for (int i = 0; i < M; ++i)
        for (int64_t l = l0; l < l1; ++l) {
            float nu = scale_of(scales, scale_mode, h, i, l);
            float t = (nu == 0.0f) ? 0.0f : S_f / nu;
            for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e) {
                float g = grads[i][e];
                float u1 = dat_oracle_uniform12_at(seed, step, (uint32_t)i, (uint64_t)e, rng_bits);
                float y = fminf(fmaf(fabsf(g), t, u1), S_f + 1.0f);
                level[i][e] = (uint32_t)floorf(y) - 1u;
                neg[i][e] = (uint8_t)(g < 0.0f);
            }
        }
}

/* Algorithm A1 Step 10 (two-sided quantisation, the parameter-server setting): before the
 * server sends the aggregate back it quantizes it once more, g_hat <- Q(g_hat).  Q is the same
 * quantizer applied to ONE vector: the scale of layer l is ||g_hat_l||_2 itself (or scales_in[l]
 * if given), the random numbers come from the stream of index `stream` (by convention M, the
 * first index no worker uses; the paper does not say where the server's randomness comes from),
 * and the receiver's value is nu_l * sign * level / S.
 * Outputs: scales[l], level[e], neg[e], and g_hat overwritten with the de-quantised value.    */
void dat_oracle_requantize(int64_t h, const int64_t *offsets, int64_t l0, int64_t l1, int bits,
                           uint64_t seed, uint64_t step, int rng_bits, uint32_t stream,
                           const float *scales_in, float *g_hat, float *scales,
                           uint32_t *level, uint8_t *neg)
{
    const uint32_t S = (uint32_t)((1ull << bits) - 1ull);
    const float S_f = (float)S;
    (void)h;
    for (int64_t l = l0; l < l1; ++l) {
        float nu;
        if (scales_in) {
            nu = scales_in[l];
        } else {
            double ss = 0.0;
            for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e)
                ss += (double)g_hat[e] * (double)g_hat[e];
            nu = (float)sqrt(ss);
        }
        scales[l] = nu;
        float t = (nu == 0.0f) ? 0.0f : S_f / nu;
        float factor = (nu == 0.0f) ? 0.0f : nu / S_f;
        for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e) {
            float g = g_hat[e];
            float u1 = dat_oracle_uniform12_at(seed, step, stream, (uint64_t)e, rng_bits);
            float y = fminf(fmaf(fabsf(g), t, u1), S_f + 1.0f);
            uint32_t lev = (uint32_t)floorf(y) - 1u;
            level[e] = lev;
            neg[e] = (uint8_t)(g < 0.0f);
            g_hat[e] = (float)(neg[e] ? -(int32_t)lev : (int32_t)lev) * factor;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* S3: the transmitted message.  32 bits per norm, 1 sign bit and b level bits */
/* per element ("(32 + d + b d) bits", with one norm per layer).               */
/* ------------------------------------------------------------------------- */

/* Both planes are flat little-endian bit streams over the global element index e:
 * level plane: element e occupies bits [(e*b) mod 8, +b) of byte floor(e*b/8)
 *              (b in {1,2,4,8}); b = 16: bytes 2e (low) and 2e+1 (high).
 * sign plane : bit (e mod 8) of byte floor(e/8); 1 = negative.
 * Plane sizes are rounded up to a multiple of 16 bytes; the padding is zero.    */
int64_t dat_oracle_level_plane_bytes(int64_t d, int bits)
{
    int64_t n = (d * (int64_t)bits + 7) / 8;
    return (n + 15) / 16 * 16;
}

int64_t dat_oracle_sign_plane_bytes(int64_t d)
{
    int64_t n = (d + 7) / 8;
    return (n + 15) / 16 * 16;
}

void dat_oracle_pack(int64_t d, int bits, const uint32_t *level, const uint8_t *neg,
                     uint8_t *level_plane, uint8_t *sign_plane)
{
    memset(level_plane, 0, (size_t)dat_oracle_level_plane_bytes(d, bits));
    memset(sign_plane, 0, (size_t)dat_oracle_sign_plane_bytes(d));
    for (int64_t e = 0; e < d; ++e) {
        int64_t bitpos = e * (int64_t)bits;
        if (bits == 16) {
            level_plane[2 * e] = (uint8_t)(level[e] & 0xFFu);
            level_plane[2 * e + 1] = (uint8_t)(level[e] >> 8);
        } else {
            level_plane[bitpos >> 3] |= (uint8_t)(level[e] << (bitpos & 7));
        }
        sign_plane[e >> 3] |= (uint8_t)((neg[e] & 1u) << (e & 7));
    }
}

void dat_oracle_unpack(int64_t d, int bits, const uint8_t *level_plane,
                       const uint8_t *sign_plane, uint32_t *level, uint8_t *neg)
{
    const uint32_t mask = (uint32_t)((1ull << bits) - 1ull);
    for (int64_t e = 0; e < d; ++e) {
        int64_t bitpos = e * (int64_t)bits;
        if (bits == 16)
            level[e] = (uint32_t)level_plane[2 * e] | ((uint32_t)level_plane[2 * e + 1] << 8);
        else
            level[e] = ((uint32_t)level_plane[bitpos >> 3] >> (bitpos & 7)) & mask;
        neg[e] = (uint8_t)((sign_plane[e >> 3] >> (e & 7)) & 1u);
    }
}

/* ------------------------------------------------------------------------- */
/* S4-S5: aggregation at the server (Eq. grad_agg) and dequantisation.         */
/* ------------------------------------------------------------------------- */

/* SHARED_MAX: all Q(g^(i)) of a layer share nu_l, so
 *   g_hat_e = (1/M) sum_i nu_l * sign * level/S = (sum_i signed level) * nu_l/(S*M):
 *   an exact int32 sum, then one fp32 factor per layer and one multiply per element.
 * PER_WORKER: g_hat_e = (sum_i nu_{i,l} * signed level_i) / (S*M), accumulated in
 *   fp32 with fmaf in ascending worker order; no integer sum exists, code_sum is
 *   left untouched.                                                              */
void dat_oracle_aggregate(int64_t h, const int64_t *offsets, int64_t l0, int64_t l1,
                          int M, int bits, int scale_mode,
                          const uint32_t *const *level, const uint8_t *const *neg,
                          const float *scales, int32_t *code_sum, float *g_hat)
{
    const uint32_t S = (uint32_t)((1ull << bits) - 1ull);
    const float SM_f = (float)((uint64_t)S * (uint64_t)M);
    for (int64_t l = l0; l < l1; ++l) {
        if (scale_mode == DAT_ORACLE_SCALE_PER_WORKER) {
            for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e) {
                float acc = 0.0f;
                for (int i = 0; i < M; ++i) {
                    float code = (float)level[i][e];
                    if (neg[i][e]) code = -code;
                    acc = fmaf(scales[(int64_t)i * h + l], code, acc);
                }
                g_hat[e] = acc / SM_f;
            }
        } else {
            float nu = scales[l];
            float factor = (nu == 0.0f) ? 0.0f : nu / SM_f;
            for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e) {
                int32_t sum = 0;
                for (int i = 0; i < M; ++i)
                    sum += neg[i][e] ? -(int32_t)level[i][e] : (int32_t)level[i][e];
                if (code_sum) code_sum[e] = sum;
                g_hat[e] = (float)sum * factor;
            }
        }
    }
}

/* b = 32 means "no quantisation": Q is the identity and Eq. grad_agg is the plain
 * worker average, accumulated in fp32 in ascending worker order.                  */
void dat_oracle_average(const int64_t *offsets, int64_t l0, int64_t l1, int M,
                        const float *const *grads, float *g_hat)
{
    for (int64_t e = offsets[l0]; e < offsets[l1]; ++e) {
        float acc = 0.0f;
        for (int i = 0; i < M; ++i) acc += grads[i][e];
        g_hat[e] = acc / (float)M;
    }
}

/* ------------------------------------------------------------------------- */
/* S6-S8: the LALR update, Eq. 3, layer by layer.                              */
/* ------------------------------------------------------------------------- */

/* u = m' = mu*m + (g_hat + wd*theta);  theta' = theta - tau(||theta||)*lr/||u|| * u
 * with tau(x) = min{max{x, c_l}, c_u}.  Norms: fp64 sum of exact squares, ascending,
 * rounded once to fp32.  layer_norms (nullable): [2l] = ||theta_l||, [2l+1] = ||u_l||. */
void dat_oracle_lalr(const int64_t *offsets, int64_t l0, int64_t l1,
                     float *theta, float *mom, const float *g_hat,
                     float lr, float mu, float wd, float c_l, float c_u,
                     float *layer_norms)
{
    for (int64_t l = l0; l < l1; ++l) {
        double ss_theta = 0.0, ss_u = 0.0;
        for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e) {
            float m_new = fmaf(mu, mom[e], fmaf(wd, theta[e], g_hat[e]));
            mom[e] = m_new;
            ss_theta += (double)theta[e] * (double)theta[e];
            ss_u += (double)m_new * (double)m_new;
        }
        float n_theta = (float)sqrt(ss_theta);
        float n_u = (float)sqrt(ss_u);
        float tau = fminf(fmaxf(n_theta, c_l), c_u);
        float ratio = (n_u == 0.0f) ? 0.0f : tau / n_u;
        float a = lr * ratio;
        for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e)
            theta[e] = fmaf(-a, mom[e], theta[e]);
        if (layer_norms) { layer_norms[2 * l] = n_theta; layer_norms[2 * l + 1] = n_u; }
    }
}

/* ------------------------------------------------------------------------- */
/* Algorithm A2 (LAMB) as the outer-minimisation oracle: the direction u_t is    */
/* Adam's, the update is again Eq. upth = Eq. 3, layer by layer.                 */
/* ------------------------------------------------------------------------- */

/* t = 1, 2, ... is the iteration count of the bias corrections.  Per element (fp32, one rounding
 * per listed operation):
 *   m' = fma(beta1, m, (1-beta1) * g)            v' = fma(beta2, v, (1-beta2) * (g*g))
 *   m^ = m' / (1 - beta1^t)                      v^ = v' / (1 - beta2^t)
 *   u  = fma(wd, theta, m^ / (sqrt(v^) + zeta))
 * then theta' = theta - (lr * tau(||theta_l||) / ||u_l||) * u with the norms of the layer in fp64.
 * Readings: the algorithm as printed overwrites m_t, v_t with their bias-corrected values; they are
 * taken as temporaries (m^, v^), as in the LAMB paper it cites, and m', v' are the stored moments.
 * The printed algorithm has no weight decay while the experiments set one; it enters as in the LAMB
 * paper (added to the ratio), so wd = 0 is the algorithm exactly as printed.
 * 1 - beta^t is formed in double and rounded to float once.                                       */
void dat_oracle_lamb(const int64_t *offsets, int64_t l0, int64_t l1,
                     float *theta, float *mom, float *var, const float *g_hat,
                     float lr, float beta1, float beta2, float zeta, float wd, float c_l, float c_u,
                     int64_t t, float *layer_norms)
{
    const float om1 = 1.0f - beta1, om2 = 1.0f - beta2;
    const float bc1 = (float)(1.0 - pow((double)beta1, (double)t));
    const float bc2 = (float)(1.0 - pow((double)beta2, (double)t));
    for (int64_t l = l0; l < l1; ++l) {
        int64_t n = offsets[l + 1] - offsets[l];
        float *u = (float *)malloc((size_t)n * sizeof(float));
        double ss_theta = 0.0, ss_u = 0.0;
        for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e) {
            float g = g_hat[e];
            float m_new = fmaf(beta1, mom[e], om1 * g);
            float v_new = fmaf(beta2, var[e], om2 * (g * g));
            mom[e] = m_new;
            var[e] = v_new;
            float m_hat = m_new / bc1;
            float v_hat = v_new / bc2;
            float ue = fmaf(wd, theta[e], m_hat / (sqrtf(v_hat) + zeta));
            u[e - offsets[l]] = ue;
            ss_theta += (double)theta[e] * (double)theta[e];
            ss_u += (double)ue * (double)ue;
        }
        float n_theta = (float)sqrt(ss_theta);
        float n_u = (float)sqrt(ss_u);
        float tau = fminf(fmaxf(n_theta, c_l), c_u);
        float ratio = (n_u == 0.0f) ? 0.0f : tau / n_u;
        float a = lr * ratio;
        for (int64_t e = offsets[l]; e < offsets[l + 1]; ++e)
            theta[e] = fmaf(-a, u[e - offsets[l]], theta[e]);
        if (layer_norms) { layer_norms[2 * l] = n_theta; layer_norms[2 * l + 1] = n_u; }
        free(u);
    }
}

/* ------------------------------------------------------------------------- */
/* One whole step for layers [l0, l1): S1 -> S2 -> S4/S5 -> S6-S8, one layer   */
/* at a time (temporary code arrays hold one layer).  scales_in (nullable)      */
/* replaces the computed scales (same indexing).  code_sum, layer_norms,        */
/* scales_out are nullable outputs.  Returns 0, or -1 if out of memory.         */
/* ------------------------------------------------------------------------- */
int dat_oracle_step(int64_t h, const int64_t *offsets, int64_t l0, int64_t l1,
                    int M, int bits, int scale_mode,
                    float *theta, float *mom, const float *const *grads,
                    uint64_t seed, uint64_t step, int rng_bits, const float *scales_in,
                    float lr, float mu, float wd, float c_l, float c_u,
                    int32_t *code_sum, float *layer_norms, float *scales_out)
{
    int64_t n_scales = (scale_mode == DAT_ORACLE_SCALE_PER_WORKER) ? (int64_t)M * h : h;
    float *norms = (float *)calloc((size_t)M * (size_t)h, sizeof(float));
    float *scales = (float *)calloc((size_t)n_scales, sizeof(float));
    uint32_t **level = (uint32_t **)calloc((size_t)M, sizeof(uint32_t *));
    uint8_t **neg = (uint8_t **)calloc((size_t)M, sizeof(uint8_t *));
    float *g_hat = NULL;
    int rc = -1;
    if (!norms || !scales || !level || !neg) goto done;

    int64_t n_max = 0;
    for (int64_t l = l0; l < l1; ++l)
        if (offsets[l + 1] - offsets[l] > n_max) n_max = offsets[l + 1] - offsets[l];
    uint32_t *level_store = (uint32_t *)malloc((size_t)M * (size_t)(n_max + 1) * sizeof(uint32_t));
    uint8_t *neg_store = (uint8_t *)malloc((size_t)M * (size_t)(n_max + 1));
    g_hat = (float *)malloc((size_t)(n_max + 1) * sizeof(float));
    if (!level_store || !neg_store || !g_hat) { free(level_store); free(neg_store); goto done; }

    for (int64_t l = l0; l < l1; ++l) {
        int64_t base = offsets[l];
        /* The per-layer temporaries are addressed with the global index e, like
         * every other array here: shift their base pointers by the layer offset. */
        for (int i = 0; i < M; ++i) {
            level[i] = level_store + (int64_t)i * n_max - base;
            neg[i] = neg_store + (int64_t)i * n_max - base;
        }
        float *g_hat_l = g_hat - base;
        if (bits == 32) {
            dat_oracle_average(offsets, l, l + 1, M, grads, g_hat_l);
        } else {
            if (scales_in) {
                if (scale_mode == DAT_ORACLE_SCALE_PER_WORKER)
                    for (int i = 0; i < M; ++i) scales[(int64_t)i * h + l] = scales_in[(int64_t)i * h + l];
                else
                    scales[l] = scales_in[l];
            } else {
                dat_oracle_worker_norms(h, offsets, l, l + 1, M, grads, norms);
                dat_oracle_scales(h, l, l + 1, M, scale_mode, norms, scales);
            }
            dat_oracle_quantize(h, offsets, l, l + 1, M, bits, scale_mode, grads, seed, step, rng_bits, scales,
                                (uint32_t *const *)level, (uint8_t *const *)neg);
            dat_oracle_aggregate(h, offsets, l, l + 1, M, bits, scale_mode,
                                 (const uint32_t *const *)level, (const uint8_t *const *)neg,
                                 scales, code_sum, g_hat_l);
        }
        dat_oracle_lalr(offsets, l, l + 1, theta, mom, g_hat_l, lr, mu, wd, c_l, c_u, layer_norms);
    }
    if (scales_out && bits != 32) {
        if (scale_mode == DAT_ORACLE_SCALE_PER_WORKER) {
            for (int i = 0; i < M; ++i)
                for (int64_t l = l0; l < l1; ++l) scales_out[(int64_t)i * h + l] = scales[(int64_t)i * h + l];
        } else {
            for (int64_t l = l0; l < l1; ++l) scales_out[l] = scales[l];
        }
    }
    free(level_store);
    free(neg_store);
    rc = 0;
done:
    free(norms); free(scales); free(level); free(neg); free(g_hat);
    return rc;
}
