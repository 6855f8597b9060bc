/*
 * CPU oracle for the SSD-SGD update path (arXiv 2012.05396).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, single-threaded
 * statement of what the update path computes.  It shares no code with the CUDA
 * library and must never be linked into, imported by or called from it.
 *
 * Every function follows the paper's steps in the paper's order; there is no
 * blocking, fusion or reordering.  Each arithmetic operator below is one
 * separately rounded IEEE-754 operation in the type `real` (compile with
 * -ffp-contract=off so that no multiply-add is fused):
 *   real = float   the reference the GPU results are compared with;
 *   real = double  (-DORACLE_DOUBLE) a shadow used for closed-form pins and to
 *                  report how far fp32 drifts.
 *
 * Readings taken where the paper leaves a choice (each is pinned by a CPU test):
 *  - descent sign everywhere: the momentum rule of Section 3.2.1 is printed with
 *    "-lr", and grad_sync = (older - newer)*(1-m)/(lr*k) points along the
 *    gradient, so the GLU rule subtracts lr_loc*(...) although it is printed "+";
 *  - a worker's gradient already holds the 1/B mini-batch mean; the server sums the
 *    K gradients left to right and multiplies by `rescale` (1/K = average);
 *  - W counts the SSGD iterations (Algorithm 1 loops while num <= wp: W = wp+1);
 *  - pull / pre_weight-refresh tests use the delay-stage index d = n - W, which
 *    equals the printed `num % k == k-1` / `loc_update % k == 0` tests whenever
 *    the paper's own constraint (1+wp) % k == 0 holds;
 *  - grad_sync is recomputed at every GLU call from the current pre_weight and
 *    the current local weight (Algorithm 2 computes it unconditionally).
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#ifdef ORACLE_DOUBLE
typedef double real;
#else
typedef float real;
#endif

typedef struct {
    int32_t K;            /* number of workers                                   */
    int32_t grad_bf16;    /* 0: gradients are float32, 1: bfloat16 bit patterns  */
    int64_t W;            /* SSGD warm-up iterations (paper's wp + 1)            */
    int64_t k;            /* delay steps; 0 = never leave SSGD                   */
    float lr, m, wd;      /* server: learning rate, momentum, weight decay       */
    float lr_loc, alpha, beta;   /* GLU: local lr and the two mixing coefficients */
    float rescale;        /* factor applied to the K-sum (1/K = average)         */
    /* Optional per-tensor multipliers (the paper uses one lr and one wd for the whole
     * model; per-tensor values are the usual refinement, e.g. no decay on BN and bias).
     * T == 0: uniform.  Tensor t covers arena positions [tensor_end[t-1], tensor_end[t]). */
    int32_t T;
    const int64_t *tensor_end;   /* T increasing exclusive end positions             */
    const float *lr_mult;        /* multiplies lr and lr_loc of tensor t             */
    const float *wd_mult;        /* multiplies wd of tensor t                        */
    const int64_t *arena_index;  /* optional: arena position of local element j (for
                                    runs on a gathered sample of the arena)          */
    /* Local updater of the workers (Section 4.4 compares them): 0 = GLU, 1 = plain SGD,
     * i.e. Eq. 5 with the descent sign, w' = w' - lr_loc*(grad' + wd*w'): no grad_sync,
     * pre_weight is neither read nor written, alpha and beta are not used. */
    int32_t local_sgd;
} oracle_hp;

typedef struct {
    int64_t N;            /* elements per buffer                                 */
    real *w, *mom;        /* server state                                        */
    real **w_loc;         /* K local weights  w'_{t,i}                           */
    real **pre;           /* K pre_weight buffers                                */
    real **w_dev;         /* K device-weight buffers, written on pull iterations */
    int64_t iter;         /* iterations done so far (Algorithm 1's num)          */
    int64_t loc_update;   /* GLU calls done so far (Algorithm 2's counter)       */
} oracle_state;

enum { STAGE_WARMUP = 0, STAGE_DELAY = 1 };
enum { F_FIRST = 1, F_REFRESH = 2, F_PULL = 4, F_COPY = 8 };
enum { VIEW_GLOBAL = 0, VIEW_LOCAL = 1, VIEW_DEVICE = 2 };

static real grad_at(const void *g, int bf16, int64_t j)
{
    if (bf16) {
        uint32_t bits = (uint32_t)((const uint16_t *)g)[j] << 16;   /* exact widening */
        float f;
        memcpy(&f, &bits, sizeof f);
        return (real)f;
    }
    return (real)((const float *)g)[j];
}

/* grad_sync scale (1-m)/(lr*k) of Section 3.3, from the float-typed
 * hyper-parameters, evaluated in double and rounded once to `real`. */
static real sync_scale_for(float lr, float m, int64_t k)
{
    if (k <= 0) return (real)0;
    return (real)((1.0 - (double)m) / ((double)lr * (double)k));
}

real oracle_sync_scale(const oracle_hp *hp) { return sync_scale_for(hp->lr, hp->m, hp->k); }

/* The four scalars that may differ per tensor, for local element j.  With
 * multipliers, tensor t uses lr*lr_mult[t], lr_loc*lr_mult[t], wd*wd_mult[t]
 * (each one float multiplication) and the grad_sync scale of its own lr. */
typedef struct { real lr, wd, lr_loc, c; } tensor_scalars;

static tensor_scalars scalars_at(const oracle_hp *hp, int64_t j)
{
    tensor_scalars s;
    if (hp->T == 0) {
        s.lr = (real)hp->lr; s.wd = (real)hp->wd; s.lr_loc = (real)hp->lr_loc;
        s.c = sync_scale_for(hp->lr, hp->m, hp->k);
        return s;
    }
    int64_t pos = hp->arena_index ? hp->arena_index[j] : j;
    int32_t t = 0;
    while (t < hp->T - 1 && pos >= hp->tensor_end[t]) ++t;
    float lr_t = hp->lr * hp->lr_mult[t];
    float wd_t = hp->wd * hp->wd_mult[t];
    float lr_loc_t = hp->lr_loc * hp->lr_mult[t];
    s.lr = (real)lr_t; s.wd = (real)wd_t; s.lr_loc = (real)lr_loc_t;
    s.c = sync_scale_for(lr_t, hp->m, hp->k);
    return s;
}

/* Stage and event flags of 0-based iteration n (Algorithm 1 and Algorithm 2).
 * Warm-up: n < W or k == 0; F_COPY marks the last warm-up iteration, on which
 * the pulled weight is kept as the local weight.  Delay stage, d = n - W:
 * F_FIRST (d == 0: pre_weight initialised from the local weight), F_REFRESH
 * (d > 0 and d % k == 0), F_PULL (d % k == k-1). */
void oracle_schedule(int64_t n, int64_t W, int64_t k, int32_t *stage, int32_t *flags)
{
    if (k == 0 || n < W) {
        *stage = STAGE_WARMUP;
        *flags = (k != 0 && n == W - 1) ? F_COPY : 0;
        return;
    }
    int64_t d = n - W;
    int32_t f = 0;
    if (d == 0) f |= F_FIRST;
    if (d > 0 && d % k == 0) f |= F_REFRESH;
    if (d % k == k - 1) f |= F_PULL;
    *stage = STAGE_DELAY;
    *flags = f;
}

/* Server: aggregate the K pushed gradients (Table 1 "averaged gradient", Eq. 6),
 * then the momentum rule of Section 3.2.1:
 *   mom = -lr*(grad + wd*w) + m*mom ;  w = w + mom. */
void oracle_server_update(int64_t N, const oracle_hp *hp, const void *const *g,
                          real *w, real *mom)
{
    const real m = (real)hp->m;
    const real rescale = (real)hp->rescale;
    const tensor_scalars uniform = scalars_at(hp, 0);
    for (int64_t j = 0; j < N; ++j) {
        const tensor_scalars ts = hp->T ? scalars_at(hp, j) : uniform;
        const real lr = ts.lr, wd = ts.wd;
        real s = grad_at(g[0], hp->grad_bf16, j);
        for (int32_t i = 1; i < hp->K; ++i)
            s = s + grad_at(g[i], hp->grad_bf16, j);
        real grad = s * rescale;
        real decay = wd * w[j];
        real full = grad + decay;
        real step = lr * full;
        real keep = m * mom[j];
        mom[j] = keep - step;
        w[j] = w[j] + mom[j];
    }
}

/* Worker i, one GLU call (Algorithm 2) plus the pull of Algorithm 1.
 *   grad_sync = (pre_weight - w') * (1-m)/(lr*k)                    Section 3.3
 *   if refresh: pre_weight = w'   (the value before the update)     Algorithm 2
 *   w' = w' - lr_loc*(alpha*grad' + wd*w' + beta*grad_sync)         GLU rule
 *   if pull: device weights keep the GLU result, w' = global w      Algorithm 1
 * On the first call pre_weight is initialised with w', so grad_sync is 0.
 * `w_server` is read only when pull is set and must already hold this
 * iteration's server result (the pull waits behind all K pushes). */
void oracle_glu_update(int64_t N, const oracle_hp *hp, const void *g,
                       real *w_loc, real *pre, real *w_dev, const real *w_server,
                       int32_t flags)
{
    const real alpha = (real)hp->alpha, beta = (real)hp->beta;
    const tensor_scalars uniform = scalars_at(hp, 0);
    for (int64_t j = 0; j < N; ++j) {
        const tensor_scalars ts = hp->T ? scalars_at(hp, j) : uniform;
        const real lr_loc = ts.lr_loc, wd = ts.wd, c = ts.c;
        if (hp->local_sgd) {
            real decay_l = wd * w_loc[j];
            real full_l = grad_at(g, hp->grad_bf16, j) + decay_l;
            real step_l = lr_loc * full_l;
            w_loc[j] = w_loc[j] - step_l;
            if (flags & F_PULL) {
                w_dev[j] = w_loc[j];
                w_loc[j] = w_server[j];
            }
            continue;
        }
        if (flags & F_FIRST) pre[j] = w_loc[j];
        real diff = pre[j] - w_loc[j];
        real grad_sync = diff * c;
        if (flags & F_REFRESH) pre[j] = w_loc[j];
        real local = alpha * grad_at(g, hp->grad_bf16, j);
        real decay = wd * w_loc[j];
        real mix = local + decay;
        real global = beta * grad_sync;
        mix = mix + global;
        real step = lr_loc * mix;
        w_loc[j] = w_loc[j] - step;
        if (flags & F_PULL) {
            w_dev[j] = w_loc[j];
            w_loc[j] = w_server[j];
        }
    }
}

/* One whole iteration for all K workers: push -> server update -> each worker's
 * local step.  Returns the flags of the iteration; *view tells which buffer the
 * workers compute their next gradient on (global w during warm-up, w_loc after a
 * plain GLU step, w_dev after a pull iteration). */
int32_t oracle_step(oracle_state *st, const oracle_hp *hp, const void *const *g,
                    int32_t *stage_out, int32_t *view)
{
    int32_t stage, flags;
    oracle_schedule(st->iter, hp->W, hp->k, &stage, &flags);
    oracle_server_update(st->N, hp, g, st->w, st->mom);
    if (stage == STAGE_WARMUP) {
        if (flags & F_COPY)
            for (int32_t i = 0; i < hp->K; ++i)
                for (int64_t j = 0; j < st->N; ++j)
                    st->w_loc[i][j] = st->w[j];
        *view = (flags & F_COPY) ? VIEW_LOCAL : VIEW_GLOBAL;
    } else {
        for (int32_t i = 0; i < hp->K; ++i)
            oracle_glu_update(st->N, hp, g[i], st->w_loc[i], st->pre[i], st->w_dev[i],
                              st->w, flags);
        st->loc_update += 1;
        *view = (flags & F_PULL) ? VIEW_DEVICE : VIEW_LOCAL;
    }
    st->iter += 1;
    *stage_out = stage;
    return flags;
}

int32_t oracle_real_bytes(void) { return (int32_t)sizeof(real); }
