/*
 * CPU oracle for the FP32 GPT-2 training step.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision statement of what the training step computes:
 * the forward pass of a pre-LayerNorm GPT-2 decoder with tied embeddings, the
 * mean cross-entropy loss, the exact gradient of that loss with respect to every
 * parameter, global-norm gradient clipping and one AdamW update.  It shares no
 * code with the CUDA library and must never be linked, imported or called by it.
 *
 * The paper gives no equations for the model, the loss or the optimizer; it names
 * them (architecture-figure caption: pre-normalised decoder blocks, masked
 * multi-head self-attention, GELU feed-forward, residual connections, weight-tied
 * embeddings; hyper-parameter table: AdamW with beta1/beta2/eps/weight decay,
 * gradient clip 1.0, dropout 0; Algorithm 1: forward, cross-entropy against the
 * target, backward, optimizer step).  The mathematics below is therefore the
 * textbook definition of each named component, written without blocking, fusion
 * or reordering so it can be checked by eye.  All storage and accumulation is
 * `double`; inputs are FP32 values widened exactly by the caller.
 *
 * Every function here is pinned by tests that do not use this file's own
 * formulas: finite differences, closed forms, invariants, library routines.
 *
 * Conventions: row-major arrays; weights are [out, in]; N = B*T rows; the fused
 * QKV output has columns ordered q | k | v, each C wide, head h owning columns
 * h*d .. (h+1)*d-1 of its part.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_API __attribute__((visibility("default")))

ORC_API int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ embedding */

/* x[n,:] = wte[tok[n],:] + wpe[n mod T,:]  (architecture caption: token plus learned
 * position embedding feeding the first block).  With round_fp32 != 0 the sum is
 * formed as ONE IEEE single-precision addition of the two FP32 values, which is the
 * reference for the bit-exact comparison of the gather kernel. */
ORC_API void orc_embedding_fwd(const int32_t* tok, const double* wte, const double* wpe,
                               int64_t N, int64_t T, int64_t C, int round_fp32, double* x) {
#pragma omp parallel for
    for (int64_t n = 0; n < N; ++n) {
        const double* e = wte + (int64_t)tok[n] * C;
        const double* p = wpe + (n % T) * C;
        for (int64_t c = 0; c < C; ++c) {
            if (round_fp32) {
                volatile float a = (float)e[c], b = (float)p[c];
                volatile float s = a + b;
                x[n * C + c] = (double)s;
            } else {
                x[n * C + c] = e[c] + p[c];
            }
        }
    }
}

/* dwte[tok[n],:] += dx[n,:];  dwpe[n mod T,:] += dx[n,:]  (accumulating). */
ORC_API void orc_embedding_bwd(const int32_t* tok, const double* dx, int64_t N, int64_t T, int64_t C,
                               double* dwte, double* dwpe) {
    for (int64_t n = 0; n < N; ++n) {
        double* e = dwte + (int64_t)tok[n] * C;
        double* p = dwpe + (n % T) * C;
        for (int64_t c = 0; c < C; ++c) {
            e[c] += dx[n * C + c];
            p[c] += dx[n * C + c];
        }
    }
}

/* ------------------------------------------------------------------ LayerNorm */

/* y = g * (x - mean) / sqrt(var + eps) + b, mean and biased variance over the C
 * features of each row. */
ORC_API void orc_layernorm_fwd(const double* x, const double* g, const double* b, int64_t N, int64_t C,
                               double eps, double* y, double* mean, double* rstd) {
#pragma omp parallel for
    for (int64_t n = 0; n < N; ++n) {
        const double* xr = x + n * C;
        double mu = 0.0;
        for (int64_t c = 0; c < C; ++c) mu += xr[c];
        mu /= (double)C;
        double var = 0.0;
        for (int64_t c = 0; c < C; ++c) var += (xr[c] - mu) * (xr[c] - mu);
        var /= (double)C;
        double rs = 1.0 / sqrt(var + eps);
        for (int64_t c = 0; c < C; ++c) y[n * C + c] = g[c] * ((xr[c] - mu) * rs) + b[c];
        if (mean) mean[n] = mu;
        if (rstd) rstd[n] = rs;
    }
}

/* With xhat = (x - mean) * rstd and dxhat = dy * g:
 *   dx = rstd * (dxhat - mean_c(dxhat) - xhat * mean_c(dxhat * xhat))
 *   dg += sum_n dy * xhat,   db += sum_n dy.
 * dx is overwritten; dg and db accumulate. */
ORC_API void orc_layernorm_bwd(const double* dy, const double* x, const double* g, const double* mean,
                               const double* rstd, int64_t N, int64_t C, double* dx, double* dg,
                               double* db) {
#pragma omp parallel for
    for (int64_t n = 0; n < N; ++n) {
        const double* xr = x + n * C;
        const double* dyr = dy + n * C;
        double mu = mean[n], rs = rstd[n];
        double s1 = 0.0, s2 = 0.0;
        for (int64_t c = 0; c < C; ++c) {
            double xh = (xr[c] - mu) * rs;
            double dxh = dyr[c] * g[c];
            s1 += dxh;
            s2 += dxh * xh;
        }
        s1 /= (double)C;
        s2 /= (double)C;
        for (int64_t c = 0; c < C; ++c) {
            double xh = (xr[c] - mu) * rs;
            double dxh = dyr[c] * g[c];
            dx[n * C + c] = rs * (dxh - s1 - xh * s2);
        }
    }
    /* parameter gradients: column sums in row order (serial over n, parallel over c) */
#pragma omp parallel for
    for (int64_t c = 0; c < C; ++c) {
        double ag = 0.0, ab = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            double xh = (x[n * C + c] - mean[n]) * rstd[n];
            ag += dy[n * C + c] * xh;
            ab += dy[n * C + c];
        }
        dg[c] += ag;
        db[c] += ab;
    }
}

/* --------------------------------------------------------------------- linear */

/* y[n,o] = sum_i x[n,i] * w[o,i] + b[o]   (b may be NULL). */
ORC_API void orc_linear_fwd(const double* x, const double* w, const double* b, int64_t N, int64_t in,
                            int64_t out, double* y) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double* xr = x + n * in;
        for (int64_t o = 0; o < out; ++o) {
            const double* wr = w + o * in;
            double acc = 0.0;
#pragma omp simd reduction(+ : acc)
            for (int64_t i = 0; i < in; ++i) acc += xr[i] * wr[i];
            y[n * out + o] = acc + (b ? b[o] : 0.0);
        }
    }
}

/* dx[n,i] = sum_o dy[n,o] * w[o,i]  (overwritten; may be NULL);
 * dw[o,i] += sum_n dy[n,o] * x[n,i];  db[o] += sum_n dy[n,o]  (db may be NULL). */
ORC_API void orc_linear_bwd(const double* dy, const double* x, const double* w, int64_t N, int64_t in,
                            int64_t out, double* dx, double* dw, double* db) {
    if (dx) {
#pragma omp parallel for schedule(static)
        for (int64_t n = 0; n < N; ++n) {
            double* dxr = dx + n * in;
            for (int64_t i = 0; i < in; ++i) dxr[i] = 0.0;
            for (int64_t o = 0; o < out; ++o) {
                double d = dy[n * out + o];
                const double* wr = w + o * in;
                for (int64_t i = 0; i < in; ++i) dxr[i] += d * wr[i];
            }
        }
    }
    if (dw) {
#pragma omp parallel for schedule(static)
        for (int64_t o = 0; o < out; ++o) {
            double* dwr = dw + o * in;
            for (int64_t n = 0; n < N; ++n) {
                double d = dy[n * out + o];
                const double* xr = x + n * in;
                for (int64_t i = 0; i < in; ++i) dwr[i] += d * xr[i];
            }
        }
    }
    if (db) {
#pragma omp parallel for
        for (int64_t o = 0; o < out; ++o) {
            double a = 0.0;
            for (int64_t n = 0; n < N; ++n) a += dy[n * out + o];
            db[o] += a;
        }
    }
}

/* ------------------------------------------------------------------ attention */

/* Causal multi-head self-attention.  For sequence b, head h, query i:
 *   S_ij = q_i . k_j / sqrt(d)  for j <= i,  P_i: = softmax_j(S_i:),  o_i = sum_j P_ij v_j.
 * The full T x T probability matrix of each (b, h) is materialised.  `lse` (nullable,
 * [B,H,T]) receives log sum_j exp(S_ij); `probs` (nullable, [B,H,T,T]) receives P with
 * exact zeros above the diagonal. */
ORC_API void orc_attention_fwd(const double* qkv, int64_t B, int64_t T, int64_t C, int64_t H, double* o,
                               double* lse, double* probs) {
    const int64_t d = C / H;
    const double scale = 1.0 / sqrt((double)d);
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t h = 0; h < H; ++h) {
            double* P = (double*)malloc((size_t)T * sizeof(double));
            for (int64_t i = 0; i < T; ++i) {
                const double* q = qkv + (b * T + i) * 3 * C + h * d;
                double mx = -INFINITY;
                for (int64_t j = 0; j <= i; ++j) {
                    const double* k = qkv + (b * T + j) * 3 * C + C + h * d;
                    double s = 0.0;
                    for (int64_t c = 0; c < d; ++c) s += q[c] * k[c];
                    s *= scale;
                    P[j] = s;
                    if (s > mx) mx = s;
                }
                double sum = 0.0;
                for (int64_t j = 0; j <= i; ++j) {
                    P[j] = exp(P[j] - mx);
                    sum += P[j];
                }
                for (int64_t j = 0; j <= i; ++j) P[j] /= sum;
                double* orow = o + (b * T + i) * C + h * d;
                for (int64_t c = 0; c < d; ++c) orow[c] = 0.0;
                for (int64_t j = 0; j <= i; ++j) {
                    const double* v = qkv + (b * T + j) * 3 * C + 2 * C + h * d;
                    for (int64_t c = 0; c < d; ++c) orow[c] += P[j] * v[c];
                }
                if (lse) lse[(b * H + h) * T + i] = mx + log(sum);
                if (probs) {
                    double* pr = probs + ((b * H + h) * T + i) * T;
                    for (int64_t j = 0; j < T; ++j) pr[j] = (j <= i) ? P[j] : 0.0;
                }
            }
            free(P);
        }
    }
}

/* Exact backward of the above.  With P recomputed from q and k:
 *   dV_j = sum_i P_ij do_i;   dP_ij = do_i . v_j;
 *   dS_ij = P_ij (dP_ij - sum_k P_ik dP_ik);
 *   dq_i = sum_j dS_ij k_j / sqrt(d);   dk_j = sum_i dS_ij q_i / sqrt(d).
 * dqkv is overwritten. */
ORC_API void orc_attention_bwd(const double* qkv, const double* d_o, int64_t B, int64_t T, int64_t C,
                               int64_t H, double* dqkv) {
    const int64_t d = C / H;
    const double scale = 1.0 / sqrt((double)d);
    memset(dqkv, 0, (size_t)(B * T * 3 * C) * sizeof(double));
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t h = 0; h < H; ++h) {
            double* P = (double*)malloc((size_t)T * sizeof(double));
            double* dP = (double*)malloc((size_t)T * sizeof(double));
            for (int64_t i = 0; i < T; ++i) {
                const double* q = qkv + (b * T + i) * 3 * C + h * d;
                const double* doi = d_o + (b * T + i) * C + h * d;
                double mx = -INFINITY;
                for (int64_t j = 0; j <= i; ++j) {
                    const double* k = qkv + (b * T + j) * 3 * C + C + h * d;
                    double s = 0.0;
                    for (int64_t c = 0; c < d; ++c) s += q[c] * k[c];
                    s *= scale;
                    P[j] = s;
                    if (s > mx) mx = s;
                }
                double sum = 0.0;
                for (int64_t j = 0; j <= i; ++j) {
                    P[j] = exp(P[j] - mx);
                    sum += P[j];
                }
                double dot = 0.0;
                for (int64_t j = 0; j <= i; ++j) {
                    P[j] /= sum;
                    const double* v = qkv + (b * T + j) * 3 * C + 2 * C + h * d;
                    double a = 0.0;
                    for (int64_t c = 0; c < d; ++c) a += doi[c] * v[c];
                    dP[j] = a;
                    dot += P[j] * a;
                }
                double* dq = dqkv + (b * T + i) * 3 * C + h * d;
                for (int64_t j = 0; j <= i; ++j) {
                    double dS = P[j] * (dP[j] - dot);
                    const double* k = qkv + (b * T + j) * 3 * C + C + h * d;
                    double* dk = dqkv + (b * T + j) * 3 * C + C + h * d;
                    double* dv = dqkv + (b * T + j) * 3 * C + 2 * C + h * d;
                    for (int64_t c = 0; c < d; ++c) {
                        dq[c] += dS * k[c] * scale;
                        dk[c] += dS * q[c] * scale;
                        dv[c] += P[j] * doi[c];
                    }
                }
            }
            free(P);
            free(dP);
        }
    }
}

/* ----------------------------------------------------------------------- GELU */

/* Exact form: GELU(x) = x * Phi(x) = 0.5 x (1 + erf(x / sqrt 2)).  The paper asks for
 * mathematically exact kernels ("avoiding lossy approximations"), so this is the
 * default; tanh_form != 0 selects 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))). */
static const double ORC_SQRT_2_OVER_PI = 0.79788456080286535588;
static const double ORC_INV_SQRT_2PI = 0.39894228040143267794;

ORC_API void orc_gelu_fwd(const double* x, int64_t n, int tanh_form, double* y) {
#pragma omp parallel for
    for (int64_t i = 0; i < n; ++i) {
        double v = x[i];
        if (tanh_form) {
            y[i] = 0.5 * v * (1.0 + tanh(ORC_SQRT_2_OVER_PI * (v + 0.044715 * v * v * v)));
        } else {
            y[i] = 0.5 * v * (1.0 + erf(v * M_SQRT1_2));
        }
    }
}

/* dx = dy * GELU'(x);  exact form: GELU'(x) = Phi(x) + x * phi(x). */
ORC_API void orc_gelu_bwd(const double* x, const double* dy, int64_t n, int tanh_form, double* dx) {
#pragma omp parallel for
    for (int64_t i = 0; i < n; ++i) {
        double v = x[i], g;
        if (tanh_form) {
            double u = ORC_SQRT_2_OVER_PI * (v + 0.044715 * v * v * v);
            double t = tanh(u);
            double du = ORC_SQRT_2_OVER_PI * (1.0 + 3.0 * 0.044715 * v * v);
            g = 0.5 * (1.0 + t) + 0.5 * v * (1.0 - t * t) * du;
        } else {
            g = 0.5 * (1.0 + erf(v * M_SQRT1_2)) + v * ORC_INV_SQRT_2PI * exp(-0.5 * v * v);
        }
        dx[i] = dy[i] * g;
    }
}

/* -------------------------------------------------------------- cross-entropy */

/* Per row n over all Vp columns (the softmax runs over the padded vocabulary):
 *   losses[n] = log sum_j exp(logits[n,j]) - logits[n, y_n]
 *   dlogits[n,j] = (softmax(logits[n,:])_j - [j == y_n]) * inv_count
 * where inv_count = 1 / (number of rows the mean runs over).  dlogits may be NULL. */
ORC_API void orc_softmax_xent(const double* logits, const int32_t* targets, int64_t N, int64_t Vp,
                              double inv_count, double* losses, double* dlogits) {
#pragma omp parallel for
    for (int64_t n = 0; n < N; ++n) {
        const double* z = logits + n * Vp;
        double mx = -INFINITY;
        for (int64_t j = 0; j < Vp; ++j)
            if (z[j] > mx) mx = z[j];
        double sum = 0.0;
        for (int64_t j = 0; j < Vp; ++j) sum += exp(z[j] - mx);
        double lse = mx + log(sum);
        losses[n] = lse - z[targets[n]];
        if (dlogits) {
            double* dz = dlogits + n * Vp;
            for (int64_t j = 0; j < Vp; ++j) dz[j] = exp(z[j] - lse) * inv_count;
            dz[targets[n]] -= inv_count;
        }
    }
}

/* ------------------------------------------------------------ clip and AdamW */

/* Sum of squares of one gradient tensor (the caller adds tensors up and takes the root). */
ORC_API double orc_sum_squares(const double* g, int64_t n) {
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) s += g[i] * g[i];
    return s;
}

/* Global-norm clipping factor: min(1, clip / (norm + 1e-6)).  The paper states only
 * "Gradient clip 1.0"; the 1e-6 guard is this build's reading. */
ORC_API double orc_clip_scale(double grad_norm, double clip) {
    double s = clip / (grad_norm + 1e-6);
    return s < 1.0 ? s : 1.0;
}

/* One AdamW update of one tensor at step t >= 1 (hyper-parameter table: AdamW, beta1,
 * beta2, eps, weight decay).  Decoupled decay first, then the bias-corrected Adam step,
 * eps added outside the square root:
 *   g' = scale * g;  p <- p (1 - lr wd decay);  m <- b1 m + (1-b1) g';  v <- b2 v + (1-b2) g'^2
 *   p <- p - lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps). */
ORC_API void orc_adamw(double* p, const double* g, double* m, double* v, int64_t n, double lr, double b1,
                       double b2, double eps, double wd, int decay, int64_t t, double scale) {
    const double c1 = 1.0 - pow(b1, (double)t);
    const double c2 = 1.0 - pow(b2, (double)t);
#pragma omp parallel for
    for (int64_t i = 0; i < n; ++i) {
        double gi = scale * g[i];
        double pi = p[i];
        if (decay) pi *= (1.0 - lr * wd);
        m[i] = b1 * m[i] + (1.0 - b1) * gi;
        v[i] = b2 * v[i] + (1.0 - b2) * gi * gi;
        double mh = m[i] / c1;
        double vh = v[i] / c2;
        p[i] = pi - lr * mh / (sqrt(vh) + eps);
    }
}

/* ---------------------------------------------------------------------- model */

typedef struct {
    char name[48];
    int64_t numel;
    int decay;
    double *p, *g, *m, *v;
} orc_tensor;

typedef struct {
    double *x, *mean1, *rstd1, *a, *qkv, *o, *x1, *mean2, *rstd2, *mm, *h, *gl;
} orc_layer_act;

typedef struct orc_model {
    int64_t L, C, H, T, V, Vp, F;
    int gelu_tanh;
    double ln_eps;
    int n_tensors;
    orc_tensor* t;
    int64_t step;
    /* activations of the chunk last run through the model */
    int64_t cap_rows;
    orc_layer_act* act;
    double *xL, *meanf, *rstdf, *xf, *logits, *dlogits, *losses;
    /* backward temporaries */
    double *dres, *dtmpC, *dtmpC2, *dqkv, *dh, *dgl;
    double last_grad_norm, last_scale;
} orc_model;

static double* dalloc(int64_t n) {
    double* p = (double*)calloc((size_t)(n > 0 ? n : 1), sizeof(double));
    if (!p) {
        fprintf(stderr, "oracle: out of host memory (%lld doubles)\n", (long long)n);
        abort();
    }
    return p;
}

static void add_tensor(orc_model* m, int* idx, const char* name, int64_t numel, int decay) {
    orc_tensor* t = &m->t[(*idx)++];
    snprintf(t->name, sizeof(t->name), "%s", name);
    t->numel = numel;
    t->decay = decay;
    t->p = dalloc(numel);
    t->g = dalloc(numel);
    t->m = dalloc(numel);
    t->v = dalloc(numel);
}

/* Registry order: wte, wpe, then per block ln1.g, ln1.b, attn.qkv.w, attn.qkv.b, attn.proj.w,
 * attn.proj.b, ln2.g, ln2.b, mlp.fc.w, mlp.fc.b, mlp.proj.w, mlp.proj.b, then lnf.g, lnf.b.
 * Weight decay applies to the tensors with two dimensions. */
ORC_API orc_model* orc_model_create(int64_t L, int64_t C, int64_t H, int64_t T, int64_t V, int64_t Vp,
                                    int gelu_tanh) {
    if (L < 1 || C < 1 || H < 1 || C % H || T < 1 || V < 1 || Vp < V) return NULL;
    orc_model* m = (orc_model*)calloc(1, sizeof(orc_model));
    m->L = L; m->C = C; m->H = H; m->T = T; m->V = V; m->Vp = Vp; m->F = 4 * C;
    m->gelu_tanh = gelu_tanh;
    m->ln_eps = 1e-5;
    m->n_tensors = (int)(2 + 12 * L + 2);
    m->t = (orc_tensor*)calloc((size_t)m->n_tensors, sizeof(orc_tensor));
    int k = 0;
    char nm[48];
    add_tensor(m, &k, "wte", Vp * C, 1);
    add_tensor(m, &k, "wpe", T * C, 1);
    for (int64_t l = 0; l < L; ++l) {
#define NM(s) (snprintf(nm, sizeof(nm), "h%lld." s, (long long)l), nm)
        add_tensor(m, &k, NM("ln1.g"), C, 0);
        add_tensor(m, &k, NM("ln1.b"), C, 0);
        add_tensor(m, &k, NM("attn.qkv.w"), 3 * C * C, 1);
        add_tensor(m, &k, NM("attn.qkv.b"), 3 * C, 0);
        add_tensor(m, &k, NM("attn.proj.w"), C * C, 1);
        add_tensor(m, &k, NM("attn.proj.b"), C, 0);
        add_tensor(m, &k, NM("ln2.g"), C, 0);
        add_tensor(m, &k, NM("ln2.b"), C, 0);
        add_tensor(m, &k, NM("mlp.fc.w"), 4 * C * C, 1);
        add_tensor(m, &k, NM("mlp.fc.b"), 4 * C, 0);
        add_tensor(m, &k, NM("mlp.proj.w"), 4 * C * C, 1);
        add_tensor(m, &k, NM("mlp.proj.b"), C, 0);
#undef NM
    }
    add_tensor(m, &k, "lnf.g", C, 0);
    add_tensor(m, &k, "lnf.b", C, 0);
    m->act = (orc_layer_act*)calloc((size_t)L, sizeof(orc_layer_act));
    return m;
}

static void free_acts(orc_model* m) {
    if (!m->cap_rows) return;
    for (int64_t l = 0; l < m->L; ++l) {
        orc_layer_act* a = &m->act[l];
        free(a->x); free(a->mean1); free(a->rstd1); free(a->a); free(a->qkv); free(a->o);
        free(a->x1); free(a->mean2); free(a->rstd2); free(a->mm); free(a->h); free(a->gl);
    }
    free(m->xL); free(m->meanf); free(m->rstdf); free(m->xf); free(m->logits); free(m->dlogits);
    free(m->losses); free(m->dres); free(m->dtmpC); free(m->dtmpC2); free(m->dqkv); free(m->dh);
    free(m->dgl);
    m->cap_rows = 0;
}

ORC_API void orc_model_destroy(orc_model* m) {
    if (!m) return;
    free_acts(m);
    for (int i = 0; i < m->n_tensors; ++i) {
        free(m->t[i].p); free(m->t[i].g); free(m->t[i].m); free(m->t[i].v);
    }
    free(m->t);
    free(m->act);
    free(m);
}

static void ensure_acts(orc_model* m, int64_t rows) {
    if (rows <= m->cap_rows) return;
    free_acts(m);
    const int64_t C = m->C, F = m->F;
    for (int64_t l = 0; l < m->L; ++l) {
        orc_layer_act* a = &m->act[l];
        a->x = dalloc(rows * C); a->mean1 = dalloc(rows); a->rstd1 = dalloc(rows);
        a->a = dalloc(rows * C); a->qkv = dalloc(rows * 3 * C); a->o = dalloc(rows * C);
        a->x1 = dalloc(rows * C); a->mean2 = dalloc(rows); a->rstd2 = dalloc(rows);
        a->mm = dalloc(rows * C); a->h = dalloc(rows * F); a->gl = dalloc(rows * F);
    }
    m->xL = dalloc(rows * C); m->meanf = dalloc(rows); m->rstdf = dalloc(rows);
    m->xf = dalloc(rows * C); m->logits = dalloc(rows * m->Vp); m->dlogits = dalloc(rows * m->Vp);
    m->losses = dalloc(rows);
    m->dres = dalloc(rows * C); m->dtmpC = dalloc(rows * C); m->dtmpC2 = dalloc(rows * C);
    m->dqkv = dalloc(rows * 3 * C); m->dh = dalloc(rows * F); m->dgl = dalloc(rows * F);
    m->cap_rows = rows;
}

ORC_API int orc_model_num_tensors(const orc_model* m) { return m->n_tensors; }

ORC_API int orc_model_tensor_info(const orc_model* m, int i, const char** name, int64_t* numel,
                                  int* decay) {
    if (i < 0 || i >= m->n_tensors) return 1;
    if (name) *name = m->t[i].name;
    if (numel) *numel = m->t[i].numel;
    if (decay) *decay = m->t[i].decay;
    return 0;
}

/* kind: 0 parameter, 1 gradient, 2 first moment, 3 second moment. */
ORC_API double* orc_model_tensor_ptr(orc_model* m, int i, int kind) {
    if (i < 0 || i >= m->n_tensors) return NULL;
    orc_tensor* t = &m->t[i];
    return kind == 0 ? t->p : kind == 1 ? t->g : kind == 2 ? t->m : kind == 3 ? t->v : NULL;
}

ORC_API void orc_model_zero_grad(orc_model* m) {
    for (int i = 0; i < m->n_tensors; ++i) memset(m->t[i].g, 0, (size_t)m->t[i].numel * sizeof(double));
}

ORC_API void orc_model_set_step(orc_model* m, int64_t step) { m->step = step; }

/* per-block tensor offsets inside the registry */
enum { LN1G = 0, LN1B, QKVW, QKVB, PROJW, PROJB, LN2G, LN2B, FCW, FCB, PRW, PRB };
#define LT(m, l, k) (&(m)->t[2 + 12 * (l) + (k)])

static void forward_rows(orc_model* m, const int32_t* tok, int64_t Bc) {
    const int64_t T = m->T, C = m->C, F = m->F, H = m->H, L = m->L, n = Bc * T;
    orc_embedding_fwd(tok, m->t[0].p, m->t[1].p, n, T, C, 0, m->act[0].x);
    for (int64_t l = 0; l < L; ++l) {
        orc_layer_act* a = &m->act[l];
        double* xout = (l + 1 < L) ? m->act[l + 1].x : m->xL;
        orc_layernorm_fwd(a->x, LT(m, l, LN1G)->p, LT(m, l, LN1B)->p, n, C, m->ln_eps, a->a, a->mean1,
                          a->rstd1);
        orc_linear_fwd(a->a, LT(m, l, QKVW)->p, LT(m, l, QKVB)->p, n, C, 3 * C, a->qkv);
        orc_attention_fwd(a->qkv, Bc, T, C, H, a->o, NULL, NULL);
        orc_linear_fwd(a->o, LT(m, l, PROJW)->p, LT(m, l, PROJB)->p, n, C, C, a->x1);
        for (int64_t i = 0; i < n * C; ++i) a->x1[i] += a->x[i];           /* residual */
        orc_layernorm_fwd(a->x1, LT(m, l, LN2G)->p, LT(m, l, LN2B)->p, n, C, m->ln_eps, a->mm, a->mean2,
                          a->rstd2);
        orc_linear_fwd(a->mm, LT(m, l, FCW)->p, LT(m, l, FCB)->p, n, C, F, a->h);
        orc_gelu_fwd(a->h, n * F, m->gelu_tanh, a->gl);
        orc_linear_fwd(a->gl, LT(m, l, PRW)->p, LT(m, l, PRB)->p, n, F, C, xout);
        for (int64_t i = 0; i < n * C; ++i) xout[i] += a->x1[i];           /* residual */
    }
    const int nt = m->n_tensors;
    orc_layernorm_fwd(m->xL, m->t[nt - 2].p, m->t[nt - 1].p, n, C, m->ln_eps, m->xf, m->meanf, m->rstdf);
    orc_linear_fwd(m->xf, m->t[0].p, NULL, n, C, m->Vp, m->logits);      /* tied LM head */
}

static void backward_rows(orc_model* m, const int32_t* tok, int64_t Bc) {
    const int64_t T = m->T, C = m->C, F = m->F, H = m->H, L = m->L, n = Bc * T;
    const int nt = m->n_tensors;
    /* LM head: dxf = dlogits . wte ; dwte += dlogits^T . xf */
    orc_linear_bwd(m->dlogits, m->xf, m->t[0].p, n, C, m->Vp, m->dtmpC, m->t[0].g, NULL);
    orc_layernorm_bwd(m->dtmpC, m->xL, m->t[nt - 2].p, m->meanf, m->rstdf, n, C, m->dres, m->t[nt - 2].g,
                      m->t[nt - 1].g);
    /* m->dres now holds d loss / d (residual stream leaving the last block) */
    for (int64_t l = L - 1; l >= 0; --l) {
        orc_layer_act* a = &m->act[l];
        /* x_out = x1 + gl . Wpr^T + bpr */
        orc_linear_bwd(m->dres, a->gl, LT(m, l, PRW)->p, n, F, C, m->dgl, LT(m, l, PRW)->g,
                       LT(m, l, PRB)->g);
        orc_gelu_bwd(a->h, m->dgl, n * F, m->gelu_tanh, m->dh);
        orc_linear_bwd(m->dh, a->mm, LT(m, l, FCW)->p, n, C, F, m->dtmpC, LT(m, l, FCW)->g,
                       LT(m, l, FCB)->g);
        orc_layernorm_bwd(m->dtmpC, a->x1, LT(m, l, LN2G)->p, a->mean2, a->rstd2, n, C, m->dtmpC2,
                          LT(m, l, LN2G)->g, LT(m, l, LN2B)->g);
        for (int64_t i = 0; i < n * C; ++i) m->dres[i] += m->dtmpC2[i];     /* d/d x1 */
        /* x1 = x + o . Wo^T + bo */
        orc_linear_bwd(m->dres, a->o, LT(m, l, PROJW)->p, n, C, C, m->dtmpC, LT(m, l, PROJW)->g,
                       LT(m, l, PROJB)->g);
        orc_attention_bwd(a->qkv, m->dtmpC, Bc, T, C, H, m->dqkv);
        orc_linear_bwd(m->dqkv, a->a, LT(m, l, QKVW)->p, n, C, 3 * C, m->dtmpC, LT(m, l, QKVW)->g,
                       LT(m, l, QKVB)->g);
        orc_layernorm_bwd(m->dtmpC, a->x, LT(m, l, LN1G)->p, a->mean1, a->rstd1, n, C, m->dtmpC2,
                          LT(m, l, LN1G)->g, LT(m, l, LN1B)->g);
        for (int64_t i = 0; i < n * C; ++i) m->dres[i] += m->dtmpC2[i];     /* d/d x */
    }
    orc_embedding_bwd(tok, m->dres, n, T, C, m->t[0].g, m->t[1].g);
}

/* Mean cross-entropy of B sequences of T tokens, and (if do_backward) its gradient
 * ACCUMULATED into the gradient tensors (call orc_model_zero_grad first for a fresh
 * gradient).  Sequences are independent given the parameters and the mean is linear, so
 * the batch is processed `chunk` sequences at a time; activations of the last chunk stay
 * available through orc_model_activation. */
ORC_API double orc_model_forward_backward(orc_model* m, const int32_t* tok, const int32_t* tgt, int64_t B,
                                          int64_t chunk, int do_backward) {
    if (chunk < 1 || chunk > B) chunk = B;
    ensure_acts(m, chunk * m->T);
    const double inv_count = 1.0 / (double)(B * m->T);
    double total = 0.0;
    for (int64_t b0 = 0; b0 < B; b0 += chunk) {
        int64_t Bc = (B - b0 < chunk) ? (B - b0) : chunk;
        int64_t n = Bc * m->T;
        forward_rows(m, tok + b0 * m->T, Bc);
        orc_softmax_xent(m->logits, tgt + b0 * m->T, n, m->Vp, inv_count, m->losses,
                         do_backward ? m->dlogits : NULL);
        for (int64_t i = 0; i < n; ++i) total += m->losses[i];
        if (do_backward) backward_rows(m, tok + b0 * m->T, Bc);
    }
    return total * inv_count;
}

/* Global gradient norm over every tensor (the tied embedding counted once). */
ORC_API double orc_model_grad_norm(const orc_model* m) {
    double s = 0.0;
    for (int i = 0; i < m->n_tensors; ++i) s += orc_sum_squares(m->t[i].g, m->t[i].numel);
    return sqrt(s);
}

/* Clip by global norm, then one AdamW update of every tensor; the step counter starts
 * at 1 on the first call.  Returns the (unclipped) gradient norm. */
ORC_API double orc_model_adamw_step(orc_model* m, double lr, double b1, double b2, double eps, double wd,
                                    double clip) {
    double gn = orc_model_grad_norm(m);
    double s = (clip > 0.0) ? orc_clip_scale(gn, clip) : 1.0;
    m->step += 1;
    for (int i = 0; i < m->n_tensors; ++i) {
        orc_tensor* t = &m->t[i];
        orc_adamw(t->p, t->g, t->m, t->v, t->numel, lr, b1, b2, eps, wd, t->decay, m->step, s);
    }
    m->last_grad_norm = gn;
    m->last_scale = s;
    return gn;
}

ORC_API double orc_model_last_scale(const orc_model* m) { return m->last_scale; }

/* Activations of the chunk last processed.  Names: x, ln1.mean, ln1.rstd, a, qkv, o, x1,
 * ln2.mean, ln2.rstd, m, h, g (per layer) and xL, xf, logits, dlogits, losses (layer
 * ignored).  Returns NULL for an unknown name. */
ORC_API double* orc_model_activation(orc_model* m, const char* name, int64_t layer) {
    if (!m->cap_rows) return NULL;
    if (!strcmp(name, "xL")) return m->xL;
    if (!strcmp(name, "xf")) return m->xf;
    if (!strcmp(name, "logits")) return m->logits;
    if (!strcmp(name, "dlogits")) return m->dlogits;
    if (!strcmp(name, "losses")) return m->losses;
    if (layer < 0 || layer >= m->L) return NULL;
    orc_layer_act* a = &m->act[layer];
    if (!strcmp(name, "x")) return a->x;
    if (!strcmp(name, "ln1.mean")) return a->mean1;
    if (!strcmp(name, "ln1.rstd")) return a->rstd1;
    if (!strcmp(name, "a")) return a->a;
    if (!strcmp(name, "qkv")) return a->qkv;
    if (!strcmp(name, "o")) return a->o;
    if (!strcmp(name, "x1")) return a->x1;
    if (!strcmp(name, "ln2.mean")) return a->mean2;
    if (!strcmp(name, "ln2.rstd")) return a->rstd2;
    if (!strcmp(name, "m")) return a->mm;
    if (!strcmp(name, "h")) return a->h;
    if (!strcmp(name, "g")) return a->gl;
    return NULL;
}
