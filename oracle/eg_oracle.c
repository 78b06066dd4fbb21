/*
 * CPU oracle for the EventGraD per-iteration communication step.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, step-by-step restatement of the method of
 * "EventGraD: Event-Triggered Communication in Parallel Machine Learning"
 * (Algorithm B, the trigger condition of Section 4, Eq. (dist_sgd_event), Eq. (thres),
 * the history-averaged slope of Section 7 and the Top-K paragraph of Section 7).
 * It shares no code with the CUDA library and must never be reachable from it.
 *
 * State is stored in fp32 exactly as the method stores it; every arithmetic step is
 * fp64 unless stated.  Build with -ffp-contract=off so that no multiply-add is fused
 * except where fma() is written out.
 *
 * Data layout: packed, x[i*N + off[t] + e] is element e of tensor t of replica (PE) i,
 * off[t] = numel[0] + ... + numel[t-1], N = sum of numel.
 *
 * Pins (tests/test_oracle_pins.py): threshold 0 == regular D-PSGD X W - gamma G
 * (Section 5 remark after Corollary 1; Eq. (dist_sgd_neigh)); infinite threshold == no
 * messages and independent SGD; doubly-stochastic W preserves the replica mean and the
 * ring's circulant eigen-modes decay as ((1+2cos(2 pi m/P))/3)^s (Section 3, Assumption
 * 2.2); error bound ||x_hat - x|| < delta (Section 5); forced event at k = 0 (Section 4);
 * a hand-worked threshold sequence from Eq. (thres) with and without history
 * (tests/golden/threshold_sequence.txt); Top-K against a brute-force sort, K = n == dense,
 * payload = 2K percent (Section 7).
 * Every function here has at least one such pin.  What the pins cannot settle is the choice
 * between two readings of an ambiguous passage: the paper prints no worked numeric trigger
 * sequence, so the pins fix the arithmetic of the readings listed below, not which reading
 * the authors meant.
 *
 * Readings where the paper is silent (kept in one place so they can be checked by eye):
 *  - the tested quantity is the L2 norm of the element-wise difference x - x_hat
 *    (the displayed trigger condition), not the difference of norms;
 *  - inside one iteration: test current x, then communicate, then average + SGD, and a
 *    message is visible to the neighbours in the same iteration (the only order for
 *    which threshold 0 gives exactly Eq. (dist_sgd_neigh));
 *  - the replica's own term in the average is its current x; neighbours contribute the
 *    last value they sent;
 *  - the first event of a tensor has no previous event, hence no slope: the threshold
 *    stays at delta_init until the second event;
 *  - history of H slopes: slope of an event = its norm / iterations since the previous
 *    event; threshold = horizon * mean of the slopes kept (H = 1 is Eq. (thres));
 *  - a mailbox that never received anything is left out of the average and the weight is
 *    1/(1 + number of neighbours heard from); with the forced first event this never
 *    happens and the weight is 1/3 on a ring;
 *  - two further readings of the text are available as variants (ego_set_variant), both off
 *    by default: the own term taken literally from Eq. (dist_sgd_event) (x_hat_i instead of
 *    x_i; with it a replica that never communicated averages with x_hat_i = X_0 = 0), and the
 *    tested quantity taken as the change of the norm, | ||x|| - ||x at the last event|| |;
 *  - Top-K ranks by |x - x_hat| (fp32 difference), sends the parameter values x[e] with
 *    their indices, ties go to the lower index, the message is in ascending index order,
 *    K_t = max(1, ceil(n_t * k_num / k_den)); the first message of a tensor is dense;
 *  - another training algorithm (the Introduction names extensions to other optimizers without
 *    giving one): heavy-ball momentum (ego_set_momentum), off by default.  Every replica keeps
 *    a velocity v of its own, never communicated, v <- mu * v + g, and the gradient term of
 *    Eq. (dist_sgd_event) becomes gamma * v.  Pinned against torch.optim.SGD(momentum=mu), a
 *    closed-form geometric series, mu = 0 == the plain update, and the dense X W - gamma V;
 *  - a second compression on top of the events (Section 7 says quantization can be applied on
 *    top of event-triggered communication and gives no scheme): uniform b-bit quantisation of
 *    the CHANGE since the last message (ego_set_quantisation), off by default.  On an event of
 *    a tensor that has been sent before, with d[e] = x[e] - x_hat[e] (fp32) and L = 2^(b-1) - 1:
 *    the scale is the power of two 2^E with the smallest integer E such that L 2^E >= max|d|,
 *    the codes are q[e] = d[e] / 2^E rounded to the nearest integer (ties to even; |q| <= L by
 *    the choice of E), the message is E and the n codes (4 + ceil(n b / 8) bytes), and sender and
 *    receivers alike set x_hat[e] <- fp32(fp64(x_hat[e]) + q[e] 2^E).  What was not sent,
 *    x - x_hat, stays in the difference and enters the next test and the next message.  The
 *    first message of a tensor is sent in full (as with Top-K), a change that is not finite
 *    too, and b = 32 means no quantisation.  Together with Top-K messages ("quantization and
 *    sparsification on top"): the K_t entries are selected as before, E comes from the largest
 *    change (which is among them), and the message holds E, the K_t indices and the K_t codes
 *    (4 + 4 K_t + ceil(K_t b / 8) bytes); x_hat is updated at the selected entries only.  Pinned against exact rational arithmetic on small
 *    inputs, the round-trip bound |x - x_hat| <= 2^E / 2 (+ rounding), changes that lie on the
 *    grid (reproduced exactly, E as constructed), b = 32 == dense, and the payload count.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#if FLT_EVAL_METHOD != 0
#error "the oracle needs float expressions evaluated in float (FLT_EVAL_METHOD == 0)"
#endif

#define EGO_MAX_HOPS 8
#define EGO_ADAPTIVE 0
#define EGO_FIXED 1

typedef struct {
    uint32_t key;
    int32_t idx;
} ego_keyidx;

typedef struct ego_ctx {
    int P, T;
    int64_t N;
    int64_t *numel, *off;
    int mode;
    double horizon;
    int H;
    double delta_init, delta_fixed;
    int force_first;
    int topk;
    uint32_t k_num, k_den;
    int64_t *Kt;      /* [T] */
    int64_t *out_off; /* [T+1] prefix of Kt */
    int64_t k;        /* iteration counter */
    float *xhat;      /* [P][N] last communicated values */
    double *delta;    /* [P*T] current threshold */
    int64_t *khat;    /* [P*T] iteration of the last event */
    double *hist;     /* [P*T][H] slopes, oldest first */
    int *hist_len;    /* [P*T] */
    uint8_t *valid;   /* [P*T] something has been sent */
    uint8_t *flag;    /* [P*T] decisions of the last step */
    double *norm;     /* [P*T] ||x - x_hat|| seen by the last step */
    double *thr_used; /* [P*T] threshold the last step compared against */
    int32_t *out_idx; /* [P][sum Kt] */
    float *out_val;
    int32_t *out_count; /* [P*T] entries of the last step's sparse message, 0 if none */
    uint64_t *seg_events;
    uint64_t *seg_payload; /* scratch: payload bytes of this step's event, 0 if none */
    uint64_t messages, bytes, events;
    int threads;
    /* variants the paper's text also admits (both off by default) */
    int own_last_sent;    /* 1: the replica's own term of the average is x_hat_i, i.e.
                             Eq. (dist_sgd_event) read literally (X_hat W) */
    int change_of_norm;   /* 1: the tested quantity is | ||x|| - ||x|| at the last event |
                             (the change-of-norm reading of the prose of Section 4) */
    double *sent_norm;    /* [P*T] ||x|| at the last event (0 before the first) */
    int hops;             /* ring neighbours on each side (1 = the paper's ring) */
    /* intermittent delivery (Section 7 remarks on the "stochastic nature of the MPI one-sided
     * implementation"): x_hat is what a replica has SENT, mailbox what its neighbours have
     * RECEIVED; they differ while a message is in flight.  NULL until a delivery mask is used. */
    float *mailbox;       /* [P][N] */
    uint8_t *pending;     /* [P*T] something sent has not arrived yet */
    uint8_t *recv_valid;  /* [P*T] the neighbours have received this tensor at least once */
    uint64_t arrivals;
    double cap_alpha, cap_beta; /* bound g(k) = alpha * beta^k on the squared threshold
                                   (Assumption 1, Corollary 2); alpha <= 0: no bound */
    double cap_g;               /* g(k) of the current iteration, carried as the geometric
                                   sequence it is: g(0) = alpha, g(k+1) = beta * g(k) */
    /* heavy-ball momentum (an extension to another training algorithm, Introduction) */
    float *vel;           /* [P][N] velocity of every replica, fp32 like the parameters; NULL: off */
    double mu;            /* momentum coefficient */
    /* quantised messages (a second compression on top of the events, Section 7) */
    int quant_bits;       /* 0: off; 2..16: bits per code */
    int32_t *qexp;        /* [P*T] scale exponent E of the last step's quantised message */
    uint8_t *quantised;   /* [P*T] the last step's message of this segment was quantised */
} ego_ctx;

void ego_destroy(ego_ctx *c) {
    if (!c) return;
    free(c->numel); free(c->off); free(c->Kt); free(c->out_off); free(c->xhat);
    free(c->delta); free(c->khat); free(c->hist); free(c->hist_len); free(c->valid);
    free(c->flag); free(c->norm); free(c->thr_used); free(c->out_idx); free(c->out_val);
    free(c->out_count); free(c->seg_events); free(c->seg_payload); free(c->sent_norm);
    free(c->mailbox); free(c->pending); free(c->recv_valid); free(c->vel);
    free(c->qexp); free(c->quantised);
    free(c);
}

void ego_reset(ego_ctx *c) {
    int64_t S = (int64_t)c->P * c->T;
    c->k = 0;
    c->cap_g = c->cap_alpha;
    c->messages = c->bytes = c->events = 0;
    c->arrivals = 0;
    if (c->mailbox) {
        memset(c->mailbox, 0, sizeof(float) * (size_t)c->P * (size_t)c->N);
        memset(c->pending, 0, (size_t)S);
        memset(c->recv_valid, 0, (size_t)S);
    }
    memset(c->xhat, 0, sizeof(float) * (size_t)c->P * (size_t)c->N); /* X_0 = 0, Assumption 2.4 */
    if (c->vel) memset(c->vel, 0, sizeof(float) * (size_t)c->P * (size_t)c->N);
    for (int64_t s = 0; s < S; ++s) {
        c->delta[s] = (c->mode == EGO_FIXED) ? c->delta_fixed : c->delta_init;
        c->khat[s] = 0;
        c->hist_len[s] = 0;
        c->valid[s] = 0;
        c->flag[s] = 0;
        c->norm[s] = 0.0;
        c->thr_used[s] = c->delta[s];
        c->out_count[s] = 0;
        c->seg_events[s] = 0;
        c->sent_norm[s] = 0.0;
    }
    memset(c->hist, 0, sizeof(double) * (size_t)S * (size_t)c->H);
}

/* Number of elements of the sparse message of a tensor with n elements. */
static int64_t topk_count(int64_t n, uint32_t k_num, uint32_t k_den) {
    /* ceil(n*k_num/k_den) in integers, at least 1, at most n */
    uint64_t prod = (uint64_t)n * (uint64_t)k_num;
    uint64_t q = (prod + (uint64_t)k_den - 1u) / (uint64_t)k_den;
    if (q < 1) q = 1;
    if (q > (uint64_t)n) q = (uint64_t)n;
    return (int64_t)q;
}

ego_ctx *ego_create(int P, int T, const int64_t *numel, int mode, double horizon, int H,
                    double delta_init, double delta_fixed, int force_first, int topk,
                    uint32_t k_num, uint32_t k_den) {
    if (P < 1 || T < 1 || H < 1 || (topk && (k_den == 0 || k_num == 0))) return NULL;
    ego_ctx *c = (ego_ctx *)calloc(1, sizeof(ego_ctx));
    if (!c) return NULL;
    c->P = P; c->T = T; c->mode = mode; c->horizon = horizon; c->H = H;
    c->delta_init = delta_init; c->delta_fixed = delta_fixed; c->force_first = force_first;
    c->topk = topk; c->k_num = k_num; c->k_den = k_den; c->threads = 1; c->hops = 1;
    c->numel = (int64_t *)malloc(sizeof(int64_t) * T);
    c->off = (int64_t *)malloc(sizeof(int64_t) * T);
    c->Kt = (int64_t *)malloc(sizeof(int64_t) * T);
    c->out_off = (int64_t *)malloc(sizeof(int64_t) * (T + 1));
    int64_t N = 0, KS = 0;
    for (int t = 0; t < T; ++t) {
        if (numel[t] < 1) { ego_destroy(c); return NULL; }
        c->numel[t] = numel[t];
        c->off[t] = N;
        N += numel[t];
        c->Kt[t] = topk ? topk_count(numel[t], k_num, k_den) : 0;
        c->out_off[t] = KS;
        KS += c->Kt[t];
    }
    c->out_off[T] = KS;
    c->N = N;
    int64_t S = (int64_t)P * T;
    c->xhat = (float *)malloc(sizeof(float) * (size_t)P * (size_t)N);
    c->delta = (double *)malloc(sizeof(double) * S);
    c->khat = (int64_t *)malloc(sizeof(int64_t) * S);
    c->hist = (double *)malloc(sizeof(double) * S * H);
    c->hist_len = (int *)malloc(sizeof(int) * S);
    c->valid = (uint8_t *)malloc(S);
    c->flag = (uint8_t *)malloc(S);
    c->norm = (double *)malloc(sizeof(double) * S);
    c->thr_used = (double *)malloc(sizeof(double) * S);
    c->out_idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(P * (KS > 0 ? KS : 1)));
    c->out_val = (float *)malloc(sizeof(float) * (size_t)(P * (KS > 0 ? KS : 1)));
    c->out_count = (int32_t *)malloc(sizeof(int32_t) * S);
    c->seg_events = (uint64_t *)malloc(sizeof(uint64_t) * S);
    c->seg_payload = (uint64_t *)malloc(sizeof(uint64_t) * S);
    c->sent_norm = (double *)malloc(sizeof(double) * S);
    ego_reset(c);
    return c;
}

void ego_set_variant(ego_ctx *c, int own_last_sent, int change_of_norm) {
    c->own_last_sent = own_last_sent != 0;
    c->change_of_norm = change_of_norm != 0;
}

/* Bound sqrt(g(k)) on the thresholds, g the geometric sequence of Corollary 2 with first term
 * alpha and ratio beta.  The sequence is evaluated term by term (one multiplication per
 * iteration); set in the middle of a run it starts from the term of the current iteration. */
void ego_set_threshold_cap(ego_ctx *c, double alpha, double beta) {
    c->cap_alpha = alpha;
    c->cap_beta = beta;
    c->cap_g = alpha;
    for (int64_t q = 0; q < c->k; ++q) c->cap_g = c->cap_g * beta;
}

int ego_set_hops(ego_ctx *c, int hops) {
    if (hops < 1 || hops > EGO_MAX_HOPS) return 1;
    c->hops = hops;
    return 0;
}

/* Heavy-ball momentum with coefficient mu (0 <= mu < 1); the velocities start at zero.
 * Returns non-zero when mu is out of range or memory is short. */
int ego_set_momentum(ego_ctx *c, double mu) {
    if (!(mu >= 0.0 && mu < 1.0)) return 1;
    if (!c->vel) {
        c->vel = (float *)calloc((size_t)c->P * (size_t)c->N, sizeof(float));
        if (!c->vel) return 1;
    }
    c->mu = mu;
    return 0;
}
float *ego_velocity(ego_ctx *c) { return c->vel; }

/* bits per code of a quantised message: 2..16; 0 or 32: messages in full precision. */
int ego_set_quantisation(ego_ctx *c, int bits) {
    if (bits == 32) bits = 0;
    if (bits != 0 && (bits < 2 || bits > 16)) return -1;
    if (bits != 0 && !c->qexp) {
        c->qexp = (int32_t *)calloc((size_t)c->P * c->T, sizeof(int32_t));
        c->quantised = (uint8_t *)calloc((size_t)c->P * c->T, 1);
        if (!c->qexp || !c->quantised) return -1;
    }
    c->quant_bits = bits;
    return 0;
}
const int32_t *ego_quant_exponents(const ego_ctx *c) { return c->qexp; }
const uint8_t *ego_quantised(const ego_ctx *c) { return c->quantised; }

void ego_set_threads(ego_ctx *c, int threads) { c->threads = threads < 1 ? 1 : threads; }

int ego_threads_available(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static uint32_t f32_bits(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    return u;
}

/* order of the Top-K ranking: larger |delta| first, then lower index */
static int cmp_rank(const void *a, const void *b) {
    const ego_keyidx *p = (const ego_keyidx *)a, *q = (const ego_keyidx *)b;
    if (p->key != q->key) return (p->key > q->key) ? -1 : 1;
    if (p->idx != q->idx) return (p->idx < q->idx) ? -1 : 1;
    return 0;
}

static int cmp_idx(const void *a, const void *b) {
    const ego_keyidx *p = (const ego_keyidx *)a, *q = (const ego_keyidx *)b;
    return (p->idx < q->idx) ? -1 : (p->idx > q->idx);
}

/* Distinct neighbours of replica i on a ring where every PE talks to the `hops` nearest PEs on
 * each side (hops = 1: the paper's ring; more: "if the number of neighbors of each PE is
 * increased, information can flow sooner", Section 7).  Order: distance 1 left, distance 1
 * right, distance 2 left, ...; a PE reached twice on a small ring is listed once and the PE
 * itself never. Returns their number. */
static int ring_neighbours(int P, int hops, int i, int nbr[2 * EGO_MAX_HOPS]) {
    int n = 0;
    for (int d = 1; d <= hops; ++d) {
        const int cand[2] = {((i - d) % P + P) % P, (i + d) % P};
        for (int side = 0; side < 2; ++side) {
            int seen = cand[side] == i;
            for (int q = 0; q < n && !seen; ++q) seen = nbr[q] == cand[side];
            if (!seen) nbr[n++] = cand[side];
        }
    }
    return n;
}

/* Phase A for one (replica i, tensor t): norm of the change, trigger test, threshold
 * update, communication into the mailbox x_hat (Algorithm B inner loop; trigger
 * condition of Section 4; Eq. (thres); history paragraph and Top-K paragraph of
 * Section 7). */
static void phase_a_segment(ego_ctx *c, const float *x, int i, int t) {
    const int64_t s = (int64_t)i * c->T + t;
    const int64_t n = c->numel[t];
    const float *xs = x + (int64_t)i * c->N + c->off[t];
    float *hs = c->xhat + (int64_t)i * c->N + c->off[t];

    /* 1-2: d = || x - x_hat ||_2 with fp32 differences, exact fp64 squares, fp64 sum;
     * variant: d = | ||x||_2 - ||x at the last event||_2 | */
    double acc = 0.0;
    double d;
    if (!c->change_of_norm) {
        for (int64_t e = 0; e < n; ++e) {
            const float d32 = xs[e] - hs[e]; /* one fp32 subtraction (FLT_EVAL_METHOD 0) */
            double dd = (double)d32;
            acc = acc + dd * dd;
        }
        d = sqrt(acc);
    } else {
        for (int64_t e = 0; e < n; ++e) {
            double dd = (double)xs[e];
            acc = acc + dd * dd;
        }
        d = fabs(sqrt(acc) - c->sent_norm[s]);
    }
    /* the threshold in force, bounded by sqrt(g(k)) when a bound is set (Assumption 1 with
     * g(k) = alpha * beta^k of Corollary 2) */
    double thr = c->delta[s];
    if (c->cap_alpha > 0.0) {
        const double cap = sqrt(c->cap_g);
        if (cap < thr) thr = cap;
    }
    c->norm[s] = d;
    c->thr_used[s] = thr;

    /* 3: the event test; the first event is forced at k = 0 (Section 4) */
    const int fire = (c->force_first && c->k == 0) || (d >= thr);
    c->flag[s] = (uint8_t)fire;
    c->out_count[s] = 0;
    c->seg_payload[s] = 0;
    if (c->qexp) { c->qexp[s] = 0; c->quantised[s] = 0; }
    if (!fire) return;

    /* 4a: new threshold from the slope between this event and the previous one */
    if (c->mode == EGO_ADAPTIVE && c->valid[s]) {
        const double slope = d / (double)(c->k - c->khat[s]);
        double *h = c->hist + s * c->H;
        if (c->hist_len[s] == c->H) {
            for (int q = 1; q < c->H; ++q) h[q - 1] = h[q];
            c->hist_len[s] = c->H - 1;
        }
        h[c->hist_len[s]++] = slope;
        double sum = 0.0;
        for (int q = 0; q < c->hist_len[s]; ++q) sum = sum + h[q];
        c->delta[s] = c->horizon * (sum / (double)c->hist_len[s]);
    }

    /* 4b: the message */
    uint64_t payload;
    int quantise = c->quant_bits != 0 && c->valid[s];
    const int sparse_route = c->topk && c->valid[s];
    float dmax = 0.0f;
    if (quantise) { /* the largest change; a change that is not finite is sent in full */
        for (int64_t e = 0; e < n; ++e) {
            const float a = fabsf(xs[e] - hs[e]);
            if (!(a <= FLT_MAX)) quantise = 0;
            if (a > dmax) dmax = a;
        }
    }
    if (c->qexp) { c->qexp[s] = 0; c->quantised[s] = (uint8_t)quantise; }
    int E = 0;
    const double L = c->quant_bits ? (double)((1 << (c->quant_bits - 1)) - 1) : 0.0;
    if (quantise) {
        if (dmax > 0.0f) { /* the smallest E with L 2^E >= max|d| */
            E = -400;
            while (ldexp(L, E) < (double)dmax) ++E;
        }
        c->qexp[s] = E;
    }
    if (quantise && !sparse_route) {
        const int b = c->quant_bits;
        for (int64_t e = 0; e < n; ++e) {
            const float d32 = xs[e] - hs[e];
            double q = rint((double)d32 * ldexp(1.0, -E)); /* exact scaling, ties to even */
            if (q > L) q = L;
            if (q < -L) q = -L;
            const double r = (double)hs[e] + q * ldexp(1.0, E);
            hs[e] = (float)r;
        }
        payload = 4u + ((uint64_t)n * (uint64_t)b + 7u) / 8u;
    } else if (!c->topk || !c->valid[s]) {
        for (int64_t e = 0; e < n; ++e) hs[e] = xs[e];
        payload = 4u * (uint64_t)n;
    } else {
        const int64_t K = c->Kt[t];
        ego_keyidx *r = (ego_keyidx *)malloc(sizeof(ego_keyidx) * (size_t)n);
        for (int64_t e = 0; e < n; ++e) {
            const float d32 = xs[e] - hs[e];
            r[e].key = f32_bits(d32) & 0x7FFFFFFFu; /* bits of |delta| order like |delta| */
            r[e].idx = (int32_t)e;
        }
        qsort(r, (size_t)n, sizeof(ego_keyidx), cmp_rank);
        qsort(r, (size_t)K, sizeof(ego_keyidx), cmp_idx);
        int32_t *oi = c->out_idx + (int64_t)i * c->out_off[c->T] + c->out_off[t];
        float *ov = c->out_val + (int64_t)i * c->out_off[c->T] + c->out_off[t];
        for (int64_t q = 0; q < K; ++q) { /* pack (index, value) */
            oi[q] = r[q].idx;
            ov[q] = xs[r[q].idx];
        }
        if (quantise) { /* the values go out as codes of the change: what arrives is x_hat + q 2^E */
            for (int64_t q = 0; q < K; ++q) {
                const float d32 = xs[oi[q]] - hs[oi[q]];
                double code = rint((double)d32 * ldexp(1.0, -E));
                if (code > L) code = L;
                if (code < -L) code = -L;
                ov[q] = (float)((double)hs[oi[q]] + code * ldexp(1.0, E));
            }
        }
        for (int64_t q = 0; q < K; ++q) hs[oi[q]] = ov[q]; /* scatter on receipt */
        c->out_count[s] = (int32_t)K;
        payload = quantise ? 4u + 4u * (uint64_t)K + ((uint64_t)K * (uint64_t)c->quant_bits + 7u) / 8u
                           : 8u * (uint64_t)K;
        free(r);
    }
    c->seg_payload[s] = payload;

    /* 4c: bookkeeping */
    if (c->change_of_norm) c->sent_norm[s] = sqrt(acc);
    c->khat[s] = c->k;
    c->valid[s] = 1;
    c->seg_events[s] += 1;
}

/* Phase B for one (replica i, tensor t): average with the neighbours' last received
 * values and apply the gradient (Eq. (dist_sgd_event) with W_ij = 1/(N_i + 1)). */
static void phase_b_segment(ego_ctx *c, float *x, const float *g, float lr, int i, int t) {
    int nbr[2 * EGO_MAX_HOPS];
    const int deg = ring_neighbours(c->P, c->hops, i, nbr);
    const float *hn[2 * EGO_MAX_HOPS];
    int cnt = 0;
    const float *box = c->mailbox ? c->mailbox : c->xhat;          /* what neighbours hold */
    const uint8_t *heard = c->mailbox ? c->recv_valid : c->valid;
    for (int q = 0; q < deg; ++q)
        if (heard[(int64_t)nbr[q] * c->T + t])
            hn[cnt++] = box + (int64_t)nbr[q] * c->N + c->off[t];
    const double w = 1.0 / (double)(1 + cnt);
    float *xs = x + (int64_t)i * c->N + c->off[t];
    const float *gs = g + (int64_t)i * c->N + c->off[t];
    const double neg_lr = -(double)lr;
    const float *own = c->own_last_sent ? c->xhat + (int64_t)i * c->N + c->off[t] : xs;
    float *vs = c->vel ? c->vel + (int64_t)i * c->N + c->off[t] : NULL;
    for (int64_t e = 0; e < c->numel[t]; ++e) {
        double sum = (double)own[e];
        for (int q = 0; q < cnt; ++q) sum = sum + (double)hn[q][e];
        const double avg = sum * w;
        double step = (double)gs[e];
        if (vs) {
            /* v <- mu * v + g, stored in fp32 like every other state; the update uses the
             * stored value */
            vs[e] = (float)fma(c->mu, (double)vs[e], (double)gs[e]);
            step = (double)vs[e];
        }
        const double r = fma(neg_lr, step, avg);
        xs[e] = (float)r;
    }
}

/* Switches to the two-copy model (sent / received).  Everything sent so far has arrived. */
int ego_enable_delivery_masks(ego_ctx *c) {
    if (c->mailbox) return 0;
    const int64_t S = (int64_t)c->P * c->T;
    const size_t bytes = sizeof(float) * (size_t)c->P * (size_t)c->N;
    c->mailbox = (float *)malloc(bytes);
    c->pending = (uint8_t *)calloc((size_t)S, 1);
    c->recv_valid = (uint8_t *)malloc((size_t)S);
    if (!c->mailbox || !c->pending || !c->recv_valid) return 1;
    memcpy(c->mailbox, c->xhat, bytes);
    memcpy(c->recv_valid, c->valid, (size_t)S);
    return 0;
}

/* One iteration of Algorithm B for all replicas.  x is updated in place.
 * deliver (may be NULL = everything arrives at once): deliver[i*T+t] != 0 means that whatever
 * replica i has sent of tensor t and has not arrived yet -- this iteration's message
 * included -- arrives at its neighbours now, before they average; 0 keeps it in flight.
 * A later message overwrites an earlier one in flight, as a later put into the same window
 * location does. */
void ego_step_masked(ego_ctx *c, float *x, const float *g, float lr, const uint8_t *deliver) {
    const int64_t S = (int64_t)c->P * c->T;
    if (deliver && !c->mailbox) ego_enable_delivery_masks(c);
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(c->threads)
#endif
    for (int64_t s = 0; s < S; ++s) phase_a_segment(c, x, (int)(s / c->T), (int)(s % c->T));

    /* message accounting: one message per (event, neighbour) */
    for (int64_t s = 0; s < S; ++s) {
        if (!c->flag[s]) continue;
        int nbr[2 * EGO_MAX_HOPS];
        const uint64_t deg = (uint64_t)ring_neighbours(c->P, c->hops, (int)(s / c->T), nbr);
        c->events += 1;
        c->messages += deg;
        c->bytes += deg * c->seg_payload[s];
    }

    /* arrivals */
    if (c->mailbox) {
        for (int64_t s = 0; s < S; ++s) {
            if (c->flag[s]) c->pending[s] = 1;
            if (c->pending[s] && (!deliver || deliver[s])) {
                const int i = (int)(s / c->T), t = (int)(s % c->T);
                const int64_t o = (int64_t)i * c->N + c->off[t];
                memcpy(c->mailbox + o, c->xhat + o, sizeof(float) * (size_t)c->numel[t]);
                c->pending[s] = 0;
                c->recv_valid[s] = 1;
                c->arrivals += 1;
            }
        }
    }

    /* every mailbox is final before anybody averages */
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(c->threads)
#endif
    for (int64_t s = 0; s < S; ++s)
        phase_b_segment(c, x, g, lr, (int)(s / c->T), (int)(s % c->T));

    c->k += 1;
    if (c->cap_alpha > 0.0) c->cap_g = c->cap_g * c->cap_beta; /* g(k+1) = beta * g(k) */
}

void ego_step(ego_ctx *c, float *x, const float *g, float lr) { ego_step_masked(c, x, g, lr, NULL); }

/* ---- readers ---------------------------------------------------------------------- */
void ego_stats(const ego_ctx *c, uint64_t *messages, uint64_t *bytes, uint64_t *events) {
    if (messages) *messages = c->messages;
    if (bytes) *bytes = c->bytes;
    if (events) *events = c->events;
}
int64_t ego_iteration(const ego_ctx *c) { return c->k; }
int64_t ego_total_numel(const ego_ctx *c) { return c->N; }
const uint8_t *ego_flags(const ego_ctx *c) { return c->flag; }
const double *ego_norms(const ego_ctx *c) { return c->norm; }
const double *ego_thresholds_used(const ego_ctx *c) { return c->thr_used; }
const double *ego_thresholds(const ego_ctx *c) { return c->delta; }
const uint8_t *ego_valid(const ego_ctx *c) { return c->valid; }
const int64_t *ego_last_event_iteration(const ego_ctx *c) { return c->khat; }
const uint64_t *ego_segment_events(const ego_ctx *c) { return c->seg_events; }
const double *ego_sent_norms(const ego_ctx *c) { return c->sent_norm; }
const double *ego_history(const ego_ctx *c) { return c->hist; }
const int *ego_history_len(const ego_ctx *c) { return c->hist_len; }
float *ego_xhat(ego_ctx *c) { return c->xhat; }
float *ego_received(ego_ctx *c) { return c->mailbox ? c->mailbox : c->xhat; }
const uint8_t *ego_pending(const ego_ctx *c) { return c->pending; }
const uint8_t *ego_received_once(const ego_ctx *c) { return c->mailbox ? c->recv_valid : c->valid; }
uint64_t ego_arrivals(const ego_ctx *c) { return c->arrivals; }
int64_t ego_topk_count(const ego_ctx *c, int t) { return c->Kt[t]; }
int32_t ego_outbox(const ego_ctx *c, int i, int t, const int32_t **idx, const float **val) {
    const int64_t o = (int64_t)i * c->out_off[c->T] + c->out_off[t];
    *idx = c->out_idx + o;
    *val = c->out_val + o;
    return c->out_count[(int64_t)i * c->T + t];
}

/* Model obtained after training by averaging all replicas (last line of Algorithms A and
 * B): out[e] = (1/P) sum_i x_i[e], fp64 sum in ascending i, rounded once to fp32. */
void ego_average_model(const ego_ctx *c, const float *x, float *out) {
    for (int64_t e = 0; e < c->N; ++e) {
        double s = 0.0;
        for (int i = 0; i < c->P; ++i) s = s + (double)x[(int64_t)i * c->N + e];
        out[e] = (float)(s / (double)c->P);
    }
}

/* Consensus distance sum_i || x_i - mean ||^2 (the quantity bounded by Lemma 2 of the
 * appendix), fp64 throughout, mean unrounded. */
double ego_consensus_distance(const ego_ctx *c, const float *x) {
    double total = 0.0;
    for (int64_t e = 0; e < c->N; ++e) {
        double s = 0.0;
        for (int i = 0; i < c->P; ++i) s = s + (double)x[(int64_t)i * c->N + e];
        const double m = s / (double)c->P;
        for (int i = 0; i < c->P; ++i) {
            const double d = (double)x[(int64_t)i * c->N + e] - m;
            total = total + d * d;
        }
    }
    return total;
}
