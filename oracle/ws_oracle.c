/*
 * ws_oracle.c - CPU oracle for the sharded weight update.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header or table with
 * the CUDA path and must never be linked into, or called from, the product.
 *
 * All floating-point work is done in double and every stored fp32 output is
 * rounded exactly once (the cast at the store).  Nothing here is blocked,
 * fused or reordered beyond what the cited passage states.  The OpenMP
 * pragmas only split loops whose iterations are independent; every
 * reduction (gradient sum over replicas, norm sums) runs in one fixed,
 * ascending order on one thread.
 *
 * What the paper fixes and where:
 *   - replicas sum their gradients and apply the same update      (Section 2.2)
 *   - reduce-scatter leaves replica r one fully reduced shard, the
 *     update runs on that shard, all-gather rebuilds the weights  (Section 2.2,
 *     "Sharding with decomposed all-reduce")
 *   - a tensor is reformatted (dimensions combined, then padded so
 *     that it divides by the shard count) and dynamic-sliced by
 *     replica id; gradient, weight and slots use one format        (Section 4.1)
 *   - reduces over sharded data mask pads with the identity by
 *     comparing element locations with the pad area, then combine
 *     per-replica partial results                                  (Section 4.1,
 *     "Non-elementwise operators")
 *   - one combined shard holds one shard of every tensor           (Section 5.2,
 *     "Batched communication operators")
 *   - update in fp32, full weight gathered in bfloat16             (Section 4.2)
 * The paper cites but does not print the optimizer formulas; the readings
 * used here are: momentum-SGD with L2 decay added to the gradient
 * (m' = mu m + g + wd w; w' = w - lr m'), Adam with bias correction and eps
 * outside the root, LAMB = Adam direction plus decoupled decay, scaled per
 * tensor by ||w|| / ||u|| (1 when either norm is zero).  LARS (the optimizer
 * of the paper's ResNet-50 runs, Table 1; formula from the LARS paper it cites):
 * local rate lambda = eta ||w|| / (||g|| + beta ||w||) per tensor (1 when either
 * norm is zero), v' = mu v + lr lambda (g + beta w), w' = w - v'.
 * Adafactor (the paper's second example of an optimizer with reduce operators, Section 4.1;
 * formula from the Adafactor paper it cites, the variant with factored second moments,
 * update clipping, relative step size, increasing decay and no momentum): for a
 * rows x cols matrix with summed gradient G and beta = 1 - t^-c,
 *   Rv' = beta Rv + (1-beta) rowsum(G^2 + eps1),  Cv' = beta Cv + (1-beta) colsum(G^2 + eps1),
 *   V = Rv' Cv'^T / sum(Rv'),  U = G / sqrt(V),  U^ = U / max(1, RMS(U)/d),
 *   w' = w - max(eps2, RMS(w)) min(lr, 1/sqrt(t)) U^;
 * a vector keeps the full v' = beta v + (1-beta)(g^2 + eps1) and uses V = v'.  A tensor of
 * more than two dimensions is the matrix of its last dimension (columns) against all the
 * leading ones together (rows).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { WSO_SGDM = 0, WSO_ADAM = 1, WSO_LAMB = 2, WSO_LARS = 3 };
enum { WSO_F32 = 0, WSO_BF16 = 1 };

typedef struct {
    int32_t opt;
    double lr, beta1, beta2, eps, weight_decay, momentum, grad_scale;
    int64_t step; /* 1-based index of the update being applied */
    double trust_coeff; /* LARS eta */
    double eps2, clip_threshold, decay_exponent; /* Adafactor: eps_2, d, c of beta2_t = 1 - t^-c */
} wso_hyper;

/* ---------------------------------------------------------------- bf16 -- */

/* bfloat16 is the upper half of an IEEE binary32; widening is exact. */
double wso_bf16_to_double(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* binary32 -> bfloat16, round to nearest, ties to even (Section 4.2 is silent
 * on the mode; nearest-even is the reading).  NaN stays NaN (quiet). */
uint16_t wso_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u && (u & 0x007fffffu) != 0u)
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lower = u & 0xffffu;      /* the 16 bits that are dropped */
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1u;
    return (uint16_t)upper;
}

static double load_grad(const void *p, int32_t dtype, int64_t i) {
    if (dtype == WSO_BF16) return wso_bf16_to_double(((const uint16_t *)p)[i]);
    return (double)((const float *)p)[i];
}

/* ---------------------------------------------------------------- plan -- */

/* Sharding format of tensor t (Section 4.1): all dimensions are combined
 * (row-major flatten, free on linear memory), the shard count R divides the
 * flattened length after padding, and every shard ("piece") is additionally
 * rounded up to a multiple of A elements.  One combined shard is one piece of
 * every tensor, in tensor order (Section 5.2).  Returns S, the combined shard
 * length; piece[t] = p_t, off[t] = start of tensor t's piece inside a shard. */
int64_t wso_plan(const int64_t *numel, int32_t T, int32_t R, int32_t A,
                 int64_t *piece, int64_t *off) {
    int64_t S = 0;
    for (int32_t t = 0; t < T; ++t) {
        int64_t per = (numel[t] + R - 1) / R;      /* ceil(n_t / R)        */
        int64_t p = ((per + A - 1) / A) * A;       /* up to a multiple of A */
        piece[t] = p;
        off[t] = S;
        S += p;
    }
    return S;
}

/* ------------------------------------------------------- pack / unpack -- */

/* flat[r*S + off_t + q] = X_t[r*p_t + q] when that location exists in the
 * tensor, else an all-zero-bits pad (Section 4.1: pad, then dynamic-slice by
 * replica id).  elem_bytes is 4 or 2; data are copied as bits. */
void wso_pack(const void *const *tensors, const int64_t *numel, const int64_t *piece,
              const int64_t *off, int32_t T, int32_t R, int64_t S, int32_t elem_bytes,
              void *flat) {
    /* (small inputs stay on the calling thread: waking a team costs more than the copy) */
#pragma omp parallel for collapse(2) schedule(dynamic) if ((int64_t)R * S > (1 << 18))
    for (int32_t r = 0; r < R; ++r)
        for (int32_t t = 0; t < T; ++t)
            for (int64_t q = 0; q < piece[t]; ++q) {
                int64_t loc = (int64_t)r * piece[t] + q;
                char *dst = (char *)flat + ((int64_t)r * S + off[t] + q) * elem_bytes;
                if (loc < numel[t])
                    memcpy(dst, (const char *)tensors[t] + loc * elem_bytes, (size_t)elem_bytes);
                else
                    memset(dst, 0, (size_t)elem_bytes);
            }
}

/* X_t[i] = gathered[(i div p_t)*S + off_t + i mod p_t]  (reverse formatting
 * after the all-gather, Section 4.2). */
void wso_unpack(const void *flat, const int64_t *numel, const int64_t *piece,
                const int64_t *off, int32_t T, int64_t S, int32_t elem_bytes,
                void *const *tensors) {
    int64_t total = 0;
    for (int32_t t = 0; t < T; ++t) total += numel[t];
#pragma omp parallel for schedule(dynamic) if (total > (1 << 18))
    for (int32_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < numel[t]; ++i) {
            int64_t r = i / piece[t], q = i % piece[t];
            memcpy((char *)tensors[t] + i * elem_bytes,
                   (const char *)flat + (r * S + off[t] + q) * elem_bytes, (size_t)elem_bytes);
        }
}

/* -------------------------------------------------- per-element update -- */

typedef struct { double bc1, bc2; } bias_corr;

static bias_corr bias_of(const wso_hyper *h) {
    bias_corr b;
    b.bc1 = 1.0 - pow(h->beta1, (double)h->step);
    b.bc2 = 1.0 - pow(h->beta2, (double)h->step);
    return b;
}

/* momentum-SGD with weight decay. */
static void sgdm_elem(const wso_hyper *h, double g, double *w, double *m) {
    double gp = g + h->weight_decay * (*w);
    double mn = h->momentum * (*m) + gp;
    *m = mn;
    *w = *w - h->lr * mn;
}

/* Adam moments; returns the bias-corrected direction mhat / (sqrt(vhat)+eps). */
static double adam_moments(const wso_hyper *h, bias_corr b, double g, double *m, double *v) {
    double mn = h->beta1 * (*m) + (1.0 - h->beta1) * g;
    double vn = h->beta2 * (*v) + (1.0 - h->beta2) * g * g;
    *m = mn;
    *v = vn;
    return (mn / b.bc1) / (sqrt(vn / b.bc2) + h->eps);
}

/* ------------------------------------------- unsharded definition (O) -- */

/* The plain definition the sharded method must reproduce (Section 3.1: every
 * replica would compute the same values): all-reduce = sum the R gradient
 * copies of a whole tensor, then apply the optimizer to the whole tensor.
 * grads[k] is replica k's gradient for THIS tensor (n elements).  w, m, v are
 * updated in place (v unused for SGDM).  *rho receives the LAMB trust ratio
 * (1 for the other optimizers). */
void wso_update_tensor(const wso_hyper *h, int64_t n, int32_t R, const void *const *grads,
                       int32_t g_dtype, float *w, float *m, float *v, double *rho) {
    bias_corr b = bias_of(h);
    if (rho) *rho = 1.0;
    if (h->opt == WSO_SGDM || h->opt == WSO_ADAM) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < n; ++i) {
            double g = 0.0;
            for (int32_t k = 0; k < R; ++k) g += load_grad(grads[k], g_dtype, i);
            g *= h->grad_scale;
            double wd = (double)w[i], md = (double)m[i];
            if (h->opt == WSO_SGDM) {
                sgdm_elem(h, g, &wd, &md);
            } else {
                double vd = (double)v[i];
                double dir = adam_moments(h, b, g, &md, &vd);
                wd = wd - h->lr * dir;
                v[i] = (float)vd;
            }
            m[i] = (float)md;
            w[i] = (float)wd;
        }
        return;
    }
    /* LAMB: u over the whole tensor, then the two norms, then the step. */
    double *u = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double g = 0.0;
        for (int32_t k = 0; k < R; ++k) g += load_grad(grads[k], g_dtype, i);
        g *= h->grad_scale;
        double md = (double)m[i], vd = (double)v[i];
        double dir = adam_moments(h, b, g, &md, &vd);
        u[i] = dir + h->weight_decay * (double)w[i];
        m[i] = (float)md;
        v[i] = (float)vd;
    }
    double a = 0.0, bb = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        a += (double)w[i] * (double)w[i];
        bb += u[i] * u[i];
    }
    double ratio = (a > 0.0 && bb > 0.0) ? sqrt(a) / sqrt(bb) : 1.0;
    if (rho) *rho = ratio;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) w[i] = (float)((double)w[i] - h->lr * ratio * u[i]);
    free(u);
}

/* ------------------------------------------ sharded route, step by step -- */

/* The method's own steps on packed buffers, in the paper's order:
 *   for every shard r: reduce the R gradient copies of slice r (reduce-scatter
 *   arithmetic), masking pads by location; update the 1/R slice of w, m, v;
 *   LAMB: per-(shard, tensor) partial sums of w^2 and u^2 over valid
 *   locations, combined over shards in ascending r (the scalar all-reduce),
 *   then the step; write w' into slot r of the gathered layout (fp32, or
 *   bf16 rounded from the fp32 master).
 * gpacked[k]: gradient copy k, packed, R*S elements, pads arbitrary; there are
 *   K copies.  K == R in the basic scheme; with partial sharding (Section 5.2:
 *   groups of replicas each shard R ways, then an all-reduce across groups adds
 *   the groups' partial results) K = groups * R and shard r sums all K slices.
 * w, m, v: [R][S] fp32 shard-major, updated in place, pads written +0.
 * gathered: [R][S] of out_dtype, or NULL.  rho: T doubles or NULL.
 * partials: [R][T][2] doubles (a, b) or NULL. */
void wso_sharded_update(const wso_hyper *h, int32_t T, const int64_t *numel,
                        const int64_t *piece, const int64_t *off, int64_t S, int32_t R,
                        int32_t K, const void *const *gpacked, int32_t g_dtype, float *w, float *m,
                        float *v, void *gathered, int32_t out_dtype, double *rho,
                        double *partials) {
    bias_corr b = bias_of(h);
    int lamb = (h->opt == WSO_LAMB);
    double *u = NULL, *part = NULL;
    if (lamb) {
        u = (double *)calloc((size_t)R * (size_t)S + 1, sizeof(double));
        part = (double *)calloc((size_t)R * (size_t)T * 2 + 1, sizeof(double));
    }
    /* (shard, tensor) iterations touch disjoint positions and own one pair of partial sums each,
     * accumulated in ascending q on whichever thread runs the iteration: the result does not
     * depend on the number of threads */
#pragma omp parallel for collapse(2) schedule(dynamic) if ((int64_t)R * S > (1 << 18))
    for (int32_t r = 0; r < R; ++r) {
        for (int32_t t = 0; t < T; ++t) {
            double pa = 0.0, pb = 0.0;
            for (int64_t q = 0; q < piece[t]; ++q) {
                int64_t j = (int64_t)r * S + off[t] + q;   /* position in [R][S] */
                int64_t loc = (int64_t)r * piece[t] + q;   /* iota + start offset */
                if (loc >= numel[t]) {                      /* pad: identity / +0 */
                    w[j] = 0.0f;
                    m[j] = 0.0f;
                    if (v) v[j] = 0.0f;
                    continue;
                }
                double g = 0.0;
                for (int32_t k = 0; k < K; ++k) g += load_grad(gpacked[k], g_dtype, j);
                g *= h->grad_scale;
                double wd = (double)w[j], md = (double)m[j];
                if (h->opt == WSO_SGDM) {
                    sgdm_elem(h, g, &wd, &md);
                    w[j] = (float)wd;
                } else {
                    double vd = (double)v[j];
                    double dir = adam_moments(h, b, g, &md, &vd);
                    v[j] = (float)vd;
                    if (lamb) {
                        double uu = dir + h->weight_decay * wd;
                        u[j] = uu;
                        pa += wd * wd;
                        pb += uu * uu;
                    } else {
                        w[j] = (float)(wd - h->lr * dir);
                    }
                }
                m[j] = (float)md;
            }
            if (lamb) {
                part[((size_t)r * T + t) * 2 + 0] = pa;
                part[((size_t)r * T + t) * 2 + 1] = pb;
            }
        }
    }
    /* per tensor: combine the shards' partials in ascending r, then apply (tensors are independent) */
#pragma omp parallel for schedule(dynamic) if ((int64_t)R * S > (1 << 18))
    for (int32_t t = 0; t < T; ++t) {
        double ratio = 1.0;
        if (lamb) {
            double a = 0.0, bb = 0.0;
            for (int32_t r = 0; r < R; ++r) {              /* combine partials */
                a += part[((size_t)r * T + t) * 2 + 0];
                bb += part[((size_t)r * T + t) * 2 + 1];
            }
            ratio = (a > 0.0 && bb > 0.0) ? sqrt(a) / sqrt(bb) : 1.0;
            for (int32_t r = 0; r < R; ++r)
                for (int64_t q = 0; q < piece[t]; ++q) {
                    int64_t j = (int64_t)r * S + off[t] + q;
                    if ((int64_t)r * piece[t] + q >= numel[t]) continue;
                    w[j] = (float)((double)w[j] - h->lr * ratio * u[j]);
                }
        }
        if (rho) rho[t] = ratio;
    }
    if (partials && lamb) memcpy(partials, part, sizeof(double) * (size_t)R * T * 2);
    if (gathered) {
        int64_t G = (int64_t)R * S;
        if (out_dtype == WSO_BF16) {
#pragma omp parallel for schedule(static) if (G > (1 << 18))
            for (int64_t j = 0; j < G; ++j) ((uint16_t *)gathered)[j] = wso_f32_to_bf16(w[j]);
        } else {
            memcpy(gathered, w, sizeof(float) * (size_t)G);
        }
    }
    free(u);
    free(part);
}

/* Reduce step alone (reduce-scatter arithmetic for shard r): out[j] =
 * grad_scale * sum_k G_k[r*S + j] over valid locations, 0 on pads; rounded
 * once to fp32. */
void wso_shard_reduce(int32_t T, const int64_t *numel, const int64_t *piece, const int64_t *off,
                      int64_t S, int32_t K, int32_t r, const void *const *gpacked,
                      int32_t g_dtype, double grad_scale, float *out) {
    for (int32_t t = 0; t < T; ++t)
        for (int64_t q = 0; q < piece[t]; ++q) {
            int64_t loc = (int64_t)r * piece[t] + q;
            double g = 0.0;
            if (loc < numel[t]) {
                for (int32_t k = 0; k < K; ++k)
                    g += load_grad(gpacked[k], g_dtype, (int64_t)r * S + off[t] + q);
                g *= grad_scale;
            }
            out[off[t] + q] = (float)g;
        }
}

/* ------------------------------------------------------------------ LARS -- */

static double lars_rate(const wso_hyper *h, double a /* sum w^2 */, double b /* sum g^2 */) {
    if (!(a > 0.0 && b > 0.0)) return 1.0;
    return h->trust_coeff * sqrt(a) / (sqrt(b) + h->weight_decay * sqrt(a));
}

/* Unsharded LARS on one whole tensor: all-reduce (sum) the K gradient copies, take the norms
 * of the weight and of the summed gradient over the whole tensor, then the momentum step with
 * the tensor's local rate.  m is the momentum buffer v of the LARS paper.  In place. */
void wso_lars_tensor(const wso_hyper *h, int64_t n, int32_t K, const void *const *grads,
                     int32_t g_dtype, float *w, float *m, double *rate) {
    double *g = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double a = 0.0, b = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double s = 0.0;
        for (int32_t k = 0; k < K; ++k) s += load_grad(grads[k], g_dtype, i);
        g[i] = s * h->grad_scale;
        a += (double)w[i] * (double)w[i];
        b += g[i] * g[i];
    }
    double lam = lars_rate(h, a, b);
    if (rate) *rate = lam;
    for (int64_t i = 0; i < n; ++i) {
        double wd = (double)w[i];
        double vn = h->momentum * (double)m[i] + h->lr * lam * (g[i] + h->weight_decay * wd);
        m[i] = (float)vn;
        w[i] = (float)(wd - vn);
    }
    free(g);
}

/* Sharded LARS, step by step (same buffers and conventions as wso_sharded_update): per shard,
 * reduce the K copies of the slice with pads masked by location and take per-(shard, tensor)
 * partial sums of w^2 and g^2; combine the partials over shards in ascending r (the scalar
 * all-reduce of Section 4.1); then every shard applies the step with its tensors' rates. */
void wso_lars_sharded(const wso_hyper *h, int32_t T, const int64_t *numel, const int64_t *piece,
                      const int64_t *off, int64_t S, int32_t R, int32_t K,
                      const void *const *gpacked, int32_t g_dtype, float *w, float *m,
                      void *gathered, int32_t out_dtype, double *rate) {
    double *g = (double *)calloc((size_t)R * (size_t)S + 1, sizeof(double));
    double *part = (double *)calloc((size_t)R * (size_t)T * 2 + 1, sizeof(double));
    for (int32_t r = 0; r < R; ++r)
        for (int32_t t = 0; t < T; ++t) {
            double pa = 0.0, pb = 0.0;
            for (int64_t q = 0; q < piece[t]; ++q) {
                int64_t j = (int64_t)r * S + off[t] + q;
                if ((int64_t)r * piece[t] + q >= numel[t]) continue;   /* pad: identity */
                double s = 0.0;
                for (int32_t k = 0; k < K; ++k) s += load_grad(gpacked[k], g_dtype, j);
                g[j] = s * h->grad_scale;
                pa += (double)w[j] * (double)w[j];
                pb += g[j] * g[j];
            }
            part[((size_t)r * T + t) * 2 + 0] = pa;
            part[((size_t)r * T + t) * 2 + 1] = pb;
        }
    for (int32_t t = 0; t < T; ++t) {
        double a = 0.0, b = 0.0;
        for (int32_t r = 0; r < R; ++r) {
            a += part[((size_t)r * T + t) * 2 + 0];
            b += part[((size_t)r * T + t) * 2 + 1];
        }
        double lam = lars_rate(h, a, b);
        if (rate) rate[t] = lam;
        for (int32_t r = 0; r < R; ++r)
            for (int64_t q = 0; q < piece[t]; ++q) {
                int64_t j = (int64_t)r * S + off[t] + q;
                if ((int64_t)r * piece[t] + q >= numel[t]) {
                    w[j] = 0.0f;
                    m[j] = 0.0f;
                    continue;
                }
                double wd = (double)w[j];
                double vn = h->momentum * (double)m[j] + h->lr * lam * (g[j] + h->weight_decay * wd);
                m[j] = (float)vn;
                w[j] = (float)(wd - vn);
            }
    }
    if (gathered) {
        int64_t G = (int64_t)R * S;
        if (out_dtype == WSO_BF16)
            for (int64_t j = 0; j < G; ++j) ((uint16_t *)gathered)[j] = wso_f32_to_bf16(w[j]);
        else
            memcpy(gathered, w, sizeof(float) * (size_t)G);
    }
    free(g);
    free(part);
}

/* ------------------------------------------- concatenated (flat) layout -- */

/* Section 5.2, "Batched communication operators": for a combined all-reduce the input tensors
 * are concatenated in their full shapes and the internal shards are partitions of the
 * concatenation, whatever tensor a boundary falls in.  As a sharding layout for the update:
 * tensor t starts at cat[t] (each start rounded up to a multiple of A elements), the
 * concatenation of length C = cat[T] is cut into R shards of S = A * ceil(ceil(C / R) / A)
 * elements, and shard r is positions [r S, (r+1) S).  Returns S. */
int64_t wso_plan_flat(const int64_t *numel, int32_t T, int32_t R, int32_t A, int64_t *cat) {
    int64_t c = 0;
    for (int32_t t = 0; t < T; ++t) {
        cat[t] = c;
        c = ((c + numel[t] + A - 1) / A) * A;
    }
    cat[T] = c;
    int64_t per = (c + R - 1) / R;
    return ((per + A - 1) / A) * A;
}

/* Sharded route over an explicit position map: tmap[p] is the tensor that owns position p of the
 * [R][S] layout (or -1 for padding).  Per shard r: reduce the K gradient copies of the slice with
 * pads masked by location, update the slice; for the norm-based optimizers take per-(shard, tensor)
 * partial sums, combine them over shards in ascending r, then apply.  Same buffers, outputs and
 * conventions as wso_sharded_update / wso_lars_sharded; serves any layout that has a map. */
void wso_sharded_update_map(const wso_hyper *h, int32_t T, const int32_t *tmap, int64_t S, int32_t R,
                            int32_t K, const void *const *gpacked, int32_t g_dtype, float *w, float *m,
                            float *v, void *gathered, int32_t out_dtype, double *rho) {
    bias_corr b = bias_of(h);
    const int lamb = (h->opt == WSO_LAMB), lars = (h->opt == WSO_LARS);
    const int64_t G = (int64_t)R * S;
    double *u = (double *)calloc((size_t)G + 1, sizeof(double));       /* LAMB: u;  LARS: summed gradient */
    double *part = (double *)calloc((size_t)R * (size_t)T * 2 + 1, sizeof(double));
    for (int32_t r = 0; r < R; ++r)
        for (int64_t q = 0; q < S; ++q) {
            const int64_t j = (int64_t)r * S + q;
            const int32_t t = tmap[j];
            if (t < 0) {                                              /* pad */
                w[j] = 0.0f;
                m[j] = 0.0f;
                if (v) v[j] = 0.0f;
                continue;
            }
            double g = 0.0;
            for (int32_t k = 0; k < K; ++k) g += load_grad(gpacked[k], g_dtype, j);
            g *= h->grad_scale;
            double wd = (double)w[j], md = (double)m[j];
            double *pa = &part[((size_t)r * T + t) * 2];
            if (h->opt == WSO_SGDM) {
                sgdm_elem(h, g, &wd, &md);
                w[j] = (float)wd;
                m[j] = (float)md;
            } else if (lars) {
                u[j] = g;
                pa[0] += wd * wd;
                pa[1] += g * g;
            } else {
                double vd = (double)v[j];
                double dir = adam_moments(h, b, g, &md, &vd);
                v[j] = (float)vd;
                m[j] = (float)md;
                if (lamb) {
                    u[j] = dir + h->weight_decay * wd;
                    pa[0] += wd * wd;
                    pa[1] += u[j] * u[j];
                } else {
                    w[j] = (float)(wd - h->lr * dir);
                }
            }
        }
    double *ratio = (double *)calloc((size_t)T + 1, sizeof(double));
    for (int32_t t = 0; t < T; ++t) {
        double a = 0.0, bb = 0.0;
        for (int32_t r = 0; r < R; ++r) {
            a += part[((size_t)r * T + t) * 2 + 0];
            bb += part[((size_t)r * T + t) * 2 + 1];
        }
        ratio[t] = 1.0;
        if (lamb) ratio[t] = (a > 0.0 && bb > 0.0) ? sqrt(a) / sqrt(bb) : 1.0;
        if (lars) ratio[t] = lars_rate(h, a, bb);
        if (rho) rho[t] = ratio[t];
    }
    if (lamb || lars)
        for (int64_t j = 0; j < G; ++j) {
            const int32_t t = tmap[j];
            if (t < 0) continue;
            const double wd = (double)w[j];
            if (lamb) {
                w[j] = (float)(wd - h->lr * ratio[t] * u[j]);
            } else {
                const double vn = h->momentum * (double)m[j] + h->lr * ratio[t] * (u[j] + h->weight_decay * wd);
                m[j] = (float)vn;
                w[j] = (float)(wd - vn);
            }
        }
    if (gathered) {
        if (out_dtype == WSO_BF16)
            for (int64_t j = 0; j < G; ++j) ((uint16_t *)gathered)[j] = wso_f32_to_bf16(w[j]);
        else
            memcpy(gathered, w, sizeof(float) * (size_t)G);
    }
    free(ratio);
    free(u);
    free(part);
}

/* ------------------------------------------- one replica's share, phase by phase -- */

/* The sharded LAMB / LARS update as ONE replica runs it on real replicas (Section 2.2: after the
 * reduce-scatter replica r holds the fully reduced gradient of shard r; Section 4.1: every replica
 * reduces what its shard holds, masking pads by location, and the replicas then combine their
 * partial results).  These are wso_sharded_update / wso_lars_sharded cut at the two points where
 * the replicas exchange data; running them for r = 0..R-1 around a sum of the partials over r
 * (ascending) gives bit for bit the same result.
 *   gslice : the reduced gradient of shard r, S elements (what the reduce-scatter delivered)
 *   w, m, v: the replica's S-element shards
 *   part   : [T][2] this shard's partial sums (sum w^2, sum u^2; LARS: sum w^2, sum g^2)
 *   u      : S doubles kept between the two phases (LAMB: the step direction; LARS: the scaled gradient) */
void wso_lamb_shard_partial(const wso_hyper *h, int32_t T, const int64_t *numel, const int64_t *piece,
                            const int64_t *off, int32_t r, const void *gslice, int32_t g_dtype,
                            const float *w, float *m, float *v, double *part, double *u) {
    bias_corr b = bias_of(h);
    for (int32_t t = 0; t < T; ++t) {
        double pa = 0.0, pb = 0.0;
        for (int64_t q = 0; q < piece[t]; ++q) {
            int64_t j = off[t] + q;
            if ((int64_t)r * piece[t] + q >= numel[t]) {     /* pad: identity / +0 */
                m[j] = 0.0f;
                v[j] = 0.0f;
                u[j] = 0.0;
                continue;
            }
            double g = load_grad(gslice, g_dtype, j) * h->grad_scale;
            double wd = (double)w[j], md = (double)m[j], vd = (double)v[j];
            double dir = adam_moments(h, b, g, &md, &vd);
            double uu = dir + h->weight_decay * wd;
            m[j] = (float)md;
            v[j] = (float)vd;
            u[j] = uu;
            pa += wd * wd;
            pb += uu * uu;
        }
        part[2 * t + 0] = pa;
        part[2 * t + 1] = pb;
    }
}

void wso_lars_shard_partial(const wso_hyper *h, int32_t T, const int64_t *numel, const int64_t *piece,
                            const int64_t *off, int32_t r, const void *gslice, int32_t g_dtype,
                            const float *w, double *part, double *u) {
    for (int32_t t = 0; t < T; ++t) {
        double pa = 0.0, pb = 0.0;
        for (int64_t q = 0; q < piece[t]; ++q) {
            int64_t j = off[t] + q;
            if ((int64_t)r * piece[t] + q >= numel[t]) {
                u[j] = 0.0;
                continue;
            }
            double g = load_grad(gslice, g_dtype, j) * h->grad_scale;
            u[j] = g;
            pa += (double)w[j] * (double)w[j];
            pb += g * g;
        }
        part[2 * t + 0] = pa;
        part[2 * t + 1] = pb;
    }
}

/* The per-tensor ratio from the combined sums: LAMB's trust ratio or LARS's local rate. */
double wso_norm_ratio(const wso_hyper *h, double a, double b) {
    if (h->opt == WSO_LARS) return lars_rate(h, a, b);
    return (a > 0.0 && b > 0.0) ? sqrt(a) / sqrt(b) : 1.0;
}

/* Phase 2 for shard r with the tensors' ratios; writes the shard's slot of the gathered layout
 * (S elements of out_dtype) when slot != NULL.  m is read and written by LARS only. */
void wso_norm_shard_apply(const wso_hyper *h, int32_t T, const int64_t *numel, const int64_t *piece,
                          const int64_t *off, int64_t S, int32_t r, const double *ratio, const double *u,
                          float *w, float *m, void *slot, int32_t out_dtype) {
    for (int32_t t = 0; t < T; ++t)
        for (int64_t q = 0; q < piece[t]; ++q) {
            int64_t j = off[t] + q;
            if ((int64_t)r * piece[t] + q >= numel[t]) {
                w[j] = 0.0f;
                if (h->opt == WSO_LARS) m[j] = 0.0f;
                continue;
            }
            double wd = (double)w[j];
            if (h->opt == WSO_LARS) {
                double vn = h->momentum * (double)m[j] + h->lr * ratio[t] * (u[j] + h->weight_decay * wd);
                m[j] = (float)vn;
                w[j] = (float)(wd - vn);
            } else {
                w[j] = (float)(wd - h->lr * ratio[t] * u[j]);
            }
        }
    if (slot) {
        if (out_dtype == WSO_BF16)
            for (int64_t j = 0; j < S; ++j) ((uint16_t *)slot)[j] = wso_f32_to_bf16(w[j]);
        else
            memcpy(slot, w, sizeof(float) * (size_t)S);
    }
}

/* ------------------------------------------------------------- Adafactor -- */

static double af_decay(const wso_hyper *h) { return 1.0 - pow((double)h->step, -h->decay_exponent); }

static double af_rho(const wso_hyper *h) {
    double r = 1.0 / sqrt((double)h->step);
    return h->lr < r ? h->lr : r;
}

/* Unsharded Adafactor on one whole tensor, seen as rows x cols (cols == 0: a vector of `rows`
 * elements, not factored).  All-reduce (sum) the K gradient copies first.  vr: rows floats
 * (the vector's full second moment when cols == 0), vc: cols floats.  In place.
 * info (may be NULL): [0] step size alpha, [1] RMS(U), [2] sum(Rv'). */
void wso_adafactor_tensor(const wso_hyper *h, int64_t rows, int64_t cols, int32_t K,
                          const void *const *grads, int32_t g_dtype, float *w, float *vr, float *vc,
                          double *info) {
    const int64_t n = cols > 0 ? rows * cols : rows;
    double *g = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double *u = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    const double beta = af_decay(h);
    double sw = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double s = 0.0;
        for (int32_t k = 0; k < K; ++k) s += load_grad(grads[k], g_dtype, i);
        g[i] = s * h->grad_scale;
        sw += (double)w[i] * (double)w[i];
    }
    double sum_r = 0.0;
    if (cols > 0) {
        double *rv = (double *)malloc(sizeof(double) * (size_t)rows);
        double *cv = (double *)malloc(sizeof(double) * (size_t)cols);
        for (int64_t i = 0; i < rows; ++i) {
            double s = 0.0;
            for (int64_t j = 0; j < cols; ++j) s += g[i * cols + j] * g[i * cols + j] + h->eps;
            rv[i] = beta * (double)vr[i] + (1.0 - beta) * s;
            vr[i] = (float)rv[i];
            sum_r += rv[i];
        }
        for (int64_t j = 0; j < cols; ++j) {
            double s = 0.0;
            for (int64_t i = 0; i < rows; ++i) s += g[i * cols + j] * g[i * cols + j] + h->eps;
            cv[j] = beta * (double)vc[j] + (1.0 - beta) * s;
            vc[j] = (float)cv[j];
        }
        for (int64_t i = 0; i < rows; ++i)
            for (int64_t j = 0; j < cols; ++j) u[i * cols + j] = g[i * cols + j] / sqrt(rv[i] * cv[j] / sum_r);
        free(rv);
        free(cv);
    } else {
        for (int64_t i = 0; i < n; ++i) {
            double v = beta * (double)vr[i] + (1.0 - beta) * (g[i] * g[i] + h->eps);
            vr[i] = (float)v;
            u[i] = g[i] / sqrt(v);
        }
    }
    double su = 0.0;
    for (int64_t i = 0; i < n; ++i) su += u[i] * u[i];
    const double rms_u = n > 0 ? sqrt(su / (double)n) : 0.0;
    const double rms_w = n > 0 ? sqrt(sw / (double)n) : 0.0;
    const double clip = rms_u / h->clip_threshold > 1.0 ? rms_u / h->clip_threshold : 1.0;
    const double alpha = (h->eps2 > rms_w ? h->eps2 : rms_w) * af_rho(h);
    for (int64_t i = 0; i < n; ++i) w[i] = (float)((double)w[i] - alpha * (u[i] / clip));
    if (info) { info[0] = alpha; info[1] = rms_u; info[2] = sum_r; }
    free(g);
    free(u);
}

/* Sharded Adafactor, step by step on packed [R][S] buffers (conventions of wso_sharded_update;
 * K gradient copies).  The row and column reduces collapse a dimension that the sharding cuts,
 * so (Section 4.1, "Non-elementwise operators") every shard masks its pads by location, reduces
 * what it holds, and the per-shard results are combined over the shards (ascending r): here the
 * row sums, the column sums, sum w^2 and later sum U^2 of every tensor.  Tensor t is
 * rows[t] x cols[t] (cols 0: vector); its factored state starts at fstate[foff[t]]: rows[t]
 * floats then cols[t] floats.  info: T x 3 doubles as in wso_adafactor_tensor, or NULL. */
void wso_adafactor_sharded(const wso_hyper *h, int32_t T, const int64_t *numel, const int64_t *piece,
                           const int64_t *off, int64_t S, int32_t R, int32_t K,
                           const void *const *gpacked, int32_t g_dtype, const int64_t *rows,
                           const int64_t *cols, const int64_t *foff, float *w, float *fstate,
                           void *gathered, int32_t out_dtype, double *info) {
    const int64_t G = (int64_t)R * S;
    const double beta = af_decay(h);
    double *g = (double *)calloc((size_t)G + 1, sizeof(double));
    double *u = (double *)calloc((size_t)G + 1, sizeof(double));
    for (int32_t t = 0; t < T; ++t) {
        const int64_t n = numel[t], nr = rows[t], nc = cols[t];
        const int64_t nstate = nc > 0 ? nr + nc : nr;
        float *vr = fstate + foff[t], *vc = vr + nr;
        /* per-shard partial reduce results: [R][nstate] sums of g^2 + eps1, [R] sums of w^2 */
        double *part = (double *)calloc((size_t)R * (size_t)(nstate > 0 ? nstate : 1), sizeof(double));
        double *pw = (double *)calloc((size_t)R, sizeof(double));
        for (int32_t r = 0; r < R; ++r)
            for (int64_t q = 0; q < piece[t]; ++q) {
                const int64_t e = (int64_t)r * piece[t] + q;        /* location in the full tensor */
                const int64_t j = (int64_t)r * S + off[t] + q;
                if (e >= n) continue;                                /* pad: identity of the sum */
                double s = 0.0;
                for (int32_t k = 0; k < K; ++k) s += load_grad(gpacked[k], g_dtype, j);
                g[j] = s * h->grad_scale;
                const double x = g[j] * g[j] + h->eps;
                if (nc > 0) {
                    part[(size_t)r * nstate + (size_t)(e / nc)] += x;
                    part[(size_t)r * nstate + (size_t)(nr + e % nc)] += x;
                } else {
                    part[(size_t)r * nstate + (size_t)e] += x;
                }
                pw[r] += (double)w[j] * (double)w[j];
            }
        /* combine over shards, then the moving averages */
        double *st = (double *)calloc((size_t)(nstate > 0 ? nstate : 1), sizeof(double));
        double sw = 0.0, sum_r = 0.0;
        for (int32_t r = 0; r < R; ++r) sw += pw[r];
        for (int64_t i = 0; i < nstate; ++i) {
            double s = 0.0;
            for (int32_t r = 0; r < R; ++r) s += part[(size_t)r * nstate + (size_t)i];
            st[i] = beta * (double)vr[i] + (1.0 - beta) * s;
            vr[i] = (float)st[i];
            if (nc > 0 && i < nr) sum_r += st[i];
        }
        (void)vc;
        /* the update direction on every shard and its partial sum of squares */
        double su = 0.0;
        for (int32_t r = 0; r < R; ++r) {
            double p = 0.0;
            for (int64_t q = 0; q < piece[t]; ++q) {
                const int64_t e = (int64_t)r * piece[t] + q;
                const int64_t j = (int64_t)r * S + off[t] + q;
                if (e >= n) continue;
                const double V = nc > 0 ? st[e / nc] * st[nr + e % nc] / sum_r : st[e];
                u[j] = g[j] / sqrt(V);
                p += u[j] * u[j];
            }
            su += p;
        }
        const double rms_u = n > 0 ? sqrt(su / (double)n) : 0.0;
        const double rms_w = n > 0 ? sqrt(sw / (double)n) : 0.0;
        const double clip = rms_u / h->clip_threshold > 1.0 ? rms_u / h->clip_threshold : 1.0;
        const double alpha = (h->eps2 > rms_w ? h->eps2 : rms_w) * af_rho(h);
        for (int32_t r = 0; r < R; ++r)
            for (int64_t q = 0; q < piece[t]; ++q) {
                const int64_t e = (int64_t)r * piece[t] + q;
                const int64_t j = (int64_t)r * S + off[t] + q;
                w[j] = e < n ? (float)((double)w[j] - alpha * (u[j] / clip)) : 0.0f;
            }
        if (info) { info[3 * t] = alpha; info[3 * t + 1] = rms_u; info[3 * t + 2] = sum_r; }
        free(part);
        free(pw);
        free(st);
    }
    if (gathered) {
        if (out_dtype == WSO_BF16)
            for (int64_t j = 0; j < G; ++j) ((uint16_t *)gathered)[j] = wso_f32_to_bf16(w[j]);
        else
            memcpy(gathered, w, sizeof(float) * (size_t)G);
    }
    free(g);
    free(u);
}

/* Sharded Adafactor as ONE replica runs it, stage by stage (wso_adafactor_sharded cut where the
 * replicas exchange data; for r = 0..R-1 with the sums taken over r in ascending order the result is
 * bit for bit the same).  gslice / w: shard r's reduced gradient and weights (S elements).
 *   sums  : adds shard r's partial row / column sums of g^2 + eps1 into acc (laid out like the
 *           factored state: tensor t at foff[t], rows then columns) and leaves sum w^2 per tensor in
 *           pw[T]; keeps the scaled gradient in gk[S]
 *           -> the replicas add their acc arrays (all-reduce) and share their pw rows
 *   moments: from the combined acc: st = beta state + (1 - beta) acc (doubles, kept for the later
 *           stages), the fp32 state, and every tensor's sum of row accumulators
 *   sumsq : u = g / sqrt(V) on shard r, partial sums of u^2 per tensor
 *           -> the replicas share their rows again
 *   step  : alpha and the clipping divisor of a tensor from its combined sums
 *   apply : w' = w - alpha u / clip on shard r */
void wso_af_shard_sums(const wso_hyper *h, int32_t T, const int64_t *numel, const int64_t *piece,
                       const int64_t *off, int32_t r, const void *gslice, int32_t g_dtype, const float *w,
                       const int64_t *rows, const int64_t *cols, const int64_t *foff, double *acc, double *pw,
                       double *gk) {
    for (int32_t t = 0; t < T; ++t) {
        const int64_t n = numel[t], nr = rows[t], nc = cols[t];
        double sw = 0.0;
        for (int64_t q = 0; q < piece[t]; ++q) {
            const int64_t e = (int64_t)r * piece[t] + q, j = off[t] + q;
            gk[j] = 0.0;
            if (e >= n) continue;
            gk[j] = load_grad(gslice, g_dtype, j) * h->grad_scale;
            const double x = gk[j] * gk[j] + h->eps;
            if (nc > 0) {
                acc[foff[t] + e / nc] += x;
                acc[foff[t] + nr + e % nc] += x;
            } else {
                acc[foff[t] + e] += x;
            }
            sw += (double)w[j] * (double)w[j];
        }
        pw[t] = sw;
    }
}

void wso_af_moments(const wso_hyper *h, int32_t T, const int64_t *rows, const int64_t *cols, const int64_t *foff,
                    const double *acc, float *fstate, double *st, double *sum_r) {
    const double beta = af_decay(h);
    for (int32_t t = 0; t < T; ++t) {
        const int64_t nr = rows[t], nc = cols[t], nstate = nc > 0 ? nr + nc : nr;
        double s = 0.0;
        for (int64_t i = 0; i < nstate; ++i) {
            const double x = beta * (double)fstate[foff[t] + i] + (1.0 - beta) * acc[foff[t] + i];
            st[foff[t] + i] = x;
            fstate[foff[t] + i] = (float)x;
            if (nc > 0 && i < nr) s += x;
        }
        sum_r[t] = s;
    }
}

void wso_af_shard_sumsq(int32_t T, const int64_t *numel, const int64_t *piece, const int64_t *off, int32_t r,
                        const int64_t *rows, const int64_t *cols, const int64_t *foff, const double *st,
                        const double *sum_r, const double *gk, double *u, double *pu) {
    for (int32_t t = 0; t < T; ++t) {
        const int64_t n = numel[t], nr = rows[t], nc = cols[t];
        double p = 0.0;
        for (int64_t q = 0; q < piece[t]; ++q) {
            const int64_t e = (int64_t)r * piece[t] + q, j = off[t] + q;
            u[j] = 0.0;
            if (e >= n) continue;
            const double V = nc > 0 ? st[foff[t] + e / nc] * st[foff[t] + nr + e % nc] / sum_r[t] : st[foff[t] + e];
            u[j] = gk[j] / sqrt(V);
            p += u[j] * u[j];
        }
        pu[t] = p;
    }
}

void wso_af_step(const wso_hyper *h, int64_t n, double sw, double su, double *alpha, double *clip) {
    const double rms_u = n > 0 ? sqrt(su / (double)n) : 0.0;
    const double rms_w = n > 0 ? sqrt(sw / (double)n) : 0.0;
    *clip = rms_u / h->clip_threshold > 1.0 ? rms_u / h->clip_threshold : 1.0;
    *alpha = (h->eps2 > rms_w ? h->eps2 : rms_w) * af_rho(h);
}

void wso_af_shard_apply(int32_t T, const int64_t *numel, const int64_t *piece, const int64_t *off, int64_t S,
                        int32_t r, const double *alpha, const double *clip, const double *u, float *w, void *slot,
                        int32_t out_dtype) {
    for (int32_t t = 0; t < T; ++t)
        for (int64_t q = 0; q < piece[t]; ++q) {
            const int64_t e = (int64_t)r * piece[t] + q, j = off[t] + q;
            w[j] = e < numel[t] ? (float)((double)w[j] - alpha[t] * (u[j] / clip[t])) : 0.0f;
        }
    if (slot) {
        if (out_dtype == WSO_BF16)
            for (int64_t j = 0; j < S; ++j) ((uint16_t *)slot)[j] = wso_f32_to_bf16(w[j]);
        else
            memcpy(slot, w, sizeof(float) * (size_t)S);
    }
}

int32_t wso_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads the loops with independent iterations may use from now on (1 = the single-thread
 * timing of the benchmark); returns the previous setting.  Results do not depend on it. */
int32_t wso_set_num_threads(int32_t n) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    extern void omp_set_num_threads(int);
    int32_t prev = omp_get_max_threads();
    if (n >= 1) omp_set_num_threads(n);
    return prev;
#else
    (void)n;
    return 1;
#endif
}
