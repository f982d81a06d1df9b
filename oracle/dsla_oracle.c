/*
 * CPU checker for the dual-state linear attention (DSLA) layer.  TEST INFRASTRUCTURE ONLY:
 * it is slow on purpose, written straight from the definition, in fp64, and shares no code
 * with the CUDA library.  Only tests, the smoke check and the benchmark's cpu_baseline /
 * reference arm may call it.
 *
 * Definition followed (Sec. 4.1, the dual-state recurrence and the blended readout):
 *     S^i_t = G^i_t (.) S^i_{t-1} + k_t^T v_t          i = 1 (history), 2 (recency)
 *     o_t   = q_t ( gamma S^1_t + (1 - gamma) S^2_t )
 * Readings taken where the text is silent or garbled:
 *   - the printed update shows S_{t-1} without a state index; each state recurs on itself,
 *     which is what the unrolled score form (products of G^1 only in sigma^1, of G^2 only in
 *     sigma^2) requires;
 *   - G^i_t is consumed already activated, either a scalar per (token, head) [G = g 11^T] or a
 *     vector over key channels [G = alpha^T 1, the gated-linear-attention form of Sec. 2];
 *   - the current token enters undecayed (the sums run to t = T inclusive and o_t uses S_t);
 *   - identity feature map, no normaliser; an optional scalar `scale` multiplies the output;
 *   - the initial state is whatever the caller passes (zeros for a fresh prompt).
 * No blocking, fusion or reordering: one token at a time, one (sequence, head) at a time.
 * Threads only split independent (sequence, head) units.
 *
 * Pins (tests/test_oracle_pins.py): quadratic masked form built from explicit gate products,
 * unrolled score form, single-state (GLA) reduction, g = 1 cumulative-sum form, g = 0 form,
 * geometric-series closed form, composition, chunked restatement, linearity, permutation.
 *
 * dsla_oracle_run_n is the same loop for n states with one blend weight per state (the generalisation
 * to more than two states of Sec. 4.2, run with 1, 2, 4 and 8 states in the number-of-states ablation
 * of Sec. 5.5):   S^i_t = G^i_t (.) S^i_{t-1} + k_t^T v_t,   o_t = q_t sum_i w_i S^i_t.
 * Pins (tests/test_oracle_nstate.py): unrolled score form with explicit gate products for 1, 3, 4 states;
 * two states with w = (gamma, 1 - gamma) reproduce dsla_oracle_run bit for bit; one state is the plain
 * gated-linear-attention loop of Sec. 3.
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    const double *q, *k, *v;      /* [T_total, H, dk], [T_total, H, dk], [T_total, H, dv] */
    const double *g[2];           /* [T_total, H] or [T_total, H, dk] when per_channel */
    const double *gamma;          /* [H] */
    const int32_t *cu;            /* [N + 1] */
    const int32_t *slots;         /* [N] or NULL (slot = sequence index) */
    int N, H, dk, dv, per_channel;
    double scale;
    double *S;                    /* [num_slots, 2, H, dk, dv] in/out */
    double *o;                    /* [T_total, H, dv] */
    int next_unit;                /* work counter, guarded by mu */
    pthread_mutex_t mu;
} job_t;

/* One (sequence, head) unit, token by token. */
static void run_unit(const job_t *J, int n, int h)
{
    const int H = J->H, dk = J->dk, dv = J->dv;
    const int slot = J->slots ? J->slots[n] : n;
    if (slot < 0) return;
    double *S1 = J->S + (((size_t)slot * 2 + 0) * H + h) * (size_t)dk * dv;
    double *S2 = J->S + (((size_t)slot * 2 + 1) * H + h) * (size_t)dk * dv;
    double *St[2] = { S1, S2 };
    const double gam = J->gamma[h];
    for (int t = J->cu[n]; t < J->cu[n + 1]; ++t) {
        const double *qt = J->q + ((size_t)t * H + h) * dk;
        const double *kt = J->k + ((size_t)t * H + h) * dk;
        const double *vt = J->v + ((size_t)t * H + h) * dv;
        for (int i = 0; i < 2; ++i) {
            for (int a = 0; a < dk; ++a) {
                const double g = J->per_channel ? J->g[i][((size_t)t * H + h) * dk + a]
                                                : J->g[i][(size_t)t * H + h];
                double *row = St[i] + (size_t)a * dv;
                for (int b = 0; b < dv; ++b)
                    row[b] = g * row[b] + kt[a] * vt[b];      /* S^i_t = G^i_t (.) S^i_{t-1} + k_t^T v_t */
            }
        }
        double *ot = J->o + ((size_t)t * H + h) * dv;
        for (int b = 0; b < dv; ++b) {
            double acc = 0.0;
            for (int a = 0; a < dk; ++a)
                acc += qt[a] * (gam * S1[(size_t)a * dv + b] + (1.0 - gam) * S2[(size_t)a * dv + b]);
            ot[b] = J->scale * acc;                           /* o_t = q_t (gamma S^1_t + (1-gamma) S^2_t) */
        }
    }
}

static void *worker(void *p)
{
    job_t *J = (job_t *)p;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        int u = J->next_unit++;
        pthread_mutex_unlock(&J->mu);
        if (u >= J->N * J->H) break;
        run_unit(J, u / J->H, u % J->H);
    }
    return NULL;
}

/* Runs every sequence of a packed batch from the state found in its slot; overwrites the slot
 * with the final state.  Two sequences must not share a slot.  Returns 0, or -1 on bad sizes. */
int dsla_oracle_run(const double *q, const double *k, const double *v,
                    const double *g_hist, const double *g_rec, int per_channel,
                    const double *gamma, const int32_t *cu_seqlens, const int32_t *slots,
                    int N, int H, int dk, int dv, double scale,
                    double *S, double *o, int nthreads)
{
    if (N < 0 || H <= 0 || dk <= 0 || dv <= 0 || !cu_seqlens) return -1;
    job_t J;
    memset(&J, 0, sizeof J);
    J.q = q; J.k = k; J.v = v; J.g[0] = g_hist; J.g[1] = g_rec; J.gamma = gamma;
    J.cu = cu_seqlens; J.slots = slots; J.N = N; J.H = H; J.dk = dk; J.dv = dv;
    J.per_channel = per_channel; J.scale = scale; J.S = S; J.o = o; J.next_unit = 0;
    pthread_mutex_init(&J.mu, NULL);
    if (nthreads < 1) nthreads = 1;
    if (nthreads > N * H) nthreads = N * H > 0 ? N * H : 1;
    if (nthreads == 1) {
        worker(&J);
    } else {
        pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
        for (int i = 0; i < nthreads; ++i) pthread_create(&th[i], NULL, worker, &J);
        for (int i = 0; i < nthreads; ++i) pthread_join(th[i], NULL);
        free(th);
    }
    pthread_mutex_destroy(&J.mu);
    return 0;
}


/* ---- n states ------------------------------------------------------------------------------- */
typedef struct {
    const double *q, *k, *v;
    const double *const *g;       /* n pointers: [T_total, H] or [T_total, H, dk] when per_channel */
    const double *w;              /* [H, n] blend weight of every state */
    const int32_t *cu, *slots;
    int N, H, dk, dv, n, per_channel;
    double scale;
    double *S;                    /* [num_slots, n, H, dk, dv] in/out */
    double *o;
    int next_unit;
    pthread_mutex_t mu;
} jobn_t;

static void run_unit_n(const jobn_t *J, int s, int h)
{
    const int H = J->H, dk = J->dk, dv = J->dv, n = J->n;
    const int slot = J->slots ? J->slots[s] : s;
    if (slot < 0) return;
    for (int t = J->cu[s]; t < J->cu[s + 1]; ++t) {
        const double *qt = J->q + ((size_t)t * H + h) * dk;
        const double *kt = J->k + ((size_t)t * H + h) * dk;
        const double *vt = J->v + ((size_t)t * H + h) * dv;
        double *ot = J->o + ((size_t)t * H + h) * dv;
        for (int b = 0; b < dv; ++b) ot[b] = 0.0;
        for (int i = 0; i < n; ++i) {
            double *Si = J->S + (((size_t)slot * n + i) * H + h) * (size_t)dk * dv;
            const double wi = J->w[(size_t)h * n + i];
            for (int a = 0; a < dk; ++a) {
                const double g = J->per_channel ? J->g[i][((size_t)t * H + h) * dk + a] : J->g[i][(size_t)t * H + h];
                double *row = Si + (size_t)a * dv;
                for (int b = 0; b < dv; ++b) {
                    row[b] = g * row[b] + kt[a] * vt[b];          /* S^i_t = G^i_t (.) S^i_{t-1} + k_t^T v_t */
                    ot[b] += qt[a] * wi * row[b];                 /* o_t = q_t sum_i w_i S^i_t */
                }
            }
        }
        for (int b = 0; b < dv; ++b) ot[b] *= J->scale;
    }
}

static void *worker_n(void *p)
{
    jobn_t *J = (jobn_t *)p;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        int u = J->next_unit++;
        pthread_mutex_unlock(&J->mu);
        if (u >= J->N * J->H) break;
        run_unit_n(J, u / J->H, u % J->H);
    }
    return NULL;
}

int dsla_oracle_run_n(const double *q, const double *k, const double *v, const double *const *gates, int n_states,
                      int per_channel, const double *weights, const int32_t *cu_seqlens, const int32_t *slots,
                      int N, int H, int dk, int dv, double scale, double *S, double *o, int nthreads)
{
    if (N < 0 || H <= 0 || dk <= 0 || dv <= 0 || n_states <= 0 || !cu_seqlens) return -1;
    jobn_t J;
    memset(&J, 0, sizeof J);
    J.q = q; J.k = k; J.v = v; J.g = gates; J.w = weights; J.cu = cu_seqlens; J.slots = slots;
    J.N = N; J.H = H; J.dk = dk; J.dv = dv; J.n = n_states; J.per_channel = per_channel; J.scale = scale; J.S = S; J.o = o;
    pthread_mutex_init(&J.mu, NULL);
    if (nthreads < 1) nthreads = 1;
    if (nthreads > N * H) nthreads = N * H > 0 ? N * H : 1;
    if (nthreads == 1) {
        worker_n(&J);
    } else {
        pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
        for (int i = 0; i < nthreads; ++i) pthread_create(&th[i], NULL, worker_n, &J);
        for (int i = 0; i < nthreads; ++i) pthread_join(th[i], NULL);
        free(th);
    }
    pthread_mutex_destroy(&J.mu);
    return 0;
}
