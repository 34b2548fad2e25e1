/*
 * CPU oracle for the Gated DeltaNet (GDN) tail-replay path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, token-by-token evaluation of the GDN recurrence in fp64.  It exists to grade
 * the CUDA kernels and is called only from the tests, the smoke check and the benchmark's
 * cpu_baseline / reference legs.  It shares no code with the CUDA path: no chunking, no
 * WY transform, no reordering.  Everything here is pinned by the CPU tests (closed forms,
 * hand-worked examples, brute-force chunked form, contraction bound); nothing is
 * "parity unpinned".
 *
 * The recurrence (paper Eq. 1, restricted to the replayed tail with a zero start by Eq. 2):
 *
 *     S_t = S_{t-1} * alpha_t * (I - beta_t k_t k_t^T) + beta_t v_t k_t^T,     S in R^{dv x dk}
 *     o_t = S_t q_t
 *
 * Eq. 1 prints the transition on the left of the state; with S stored dv x dk that product
 * only type-checks on the right (the transition is symmetric), which is the form above.
 * alpha_t = exp(g_t) with g_t = log alpha_t <= 0 given as input.  v-head h reads q/k head
 * h / (Hv/Hq).  The output o_t uses the state after token t's update.
 *
 * Layouts: q,k [T,Hq,dk]; v [T,Hv,dv]; g,beta [T,Hv]; cu [N+1]; out_o [T,Hv,dv];
 * init_state / out_state [N,Hv,dk,dv] with out_state[n,h,a,b] = S[b][a] (the transpose).
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    const float *q, *k, *v, *g, *beta;
    const double *qd, *kd, *vd, *gd, *betad;   /* the same five inputs given in fp64 (then the float ones are NULL) */
    const int32_t *cu;
    int32_t num_seqs, Hq, Hv, dk, dv;
    const double *init_state;
    double *out_o, *out_state;
    int64_t next_item;          /* guarded by lock */
    pthread_mutex_t lock;
} oracle_job;

/* One chain: request n, v-head h.  Eq. 1 / Eq. 2 applied token by token. */
static void run_chain(const oracle_job *J, int32_t n, int32_t h)
{
    const int32_t dk = J->dk, dv = J->dv, Hq = J->Hq, Hv = J->Hv;
    const int32_t hq = h / (Hv / Hq);
    double *S = (double *)calloc((size_t)dv * dk, sizeof(double));   /* S[i*dk + j], i<dv, j<dk */
    double *Sk = (double *)malloc((size_t)dv * sizeof(double));
    double *kk = (double *)malloc((size_t)dk * sizeof(double));
    double *qq = (double *)malloc((size_t)dk * sizeof(double));
    double *vv = (double *)malloc((size_t)dv * sizeof(double));

    if (J->init_state) {
        const double *H0 = J->init_state + ((size_t)n * Hv + h) * dk * dv;
        for (int32_t i = 0; i < dv; ++i)
            for (int32_t j = 0; j < dk; ++j)
                S[(size_t)i * dk + j] = H0[(size_t)j * dv + i];
    }

    for (int64_t t = J->cu[n]; t < J->cu[n + 1]; ++t) {
        const double alpha = exp(J->gd ? J->gd[t * Hv + h] : (double)J->g[t * Hv + h]);
        const double beta = J->betad ? J->betad[t * Hv + h] : (double)J->beta[t * Hv + h];
        for (int32_t j = 0; j < dk; ++j) {
            kk[j] = J->kd ? J->kd[(t * Hq + hq) * dk + j] : (double)J->k[(t * Hq + hq) * dk + j];
            qq[j] = J->qd ? J->qd[(t * Hq + hq) * dk + j] : (double)J->q[(t * Hq + hq) * dk + j];
        }
        for (int32_t i = 0; i < dv; ++i)
            vv[i] = J->vd ? J->vd[(t * Hv + h) * dv + i] : (double)J->v[(t * Hv + h) * dv + i];

        /* S k  (what the old state recalls for this key) */
        for (int32_t i = 0; i < dv; ++i) {
            double acc = 0.0;
            for (int32_t j = 0; j < dk; ++j) acc += S[(size_t)i * dk + j] * kk[j];
            Sk[i] = acc;
        }
        /* S <- alpha * (S - beta (S k) k^T) + beta v k^T */
        for (int32_t i = 0; i < dv; ++i)
            for (int32_t j = 0; j < dk; ++j)
                S[(size_t)i * dk + j] =
                    alpha * (S[(size_t)i * dk + j] - beta * Sk[i] * kk[j]) + beta * vv[i] * kk[j];
        /* o_t = S_t q_t */
        if (J->out_o) {
            double *o = J->out_o + (t * Hv + h) * dv;
            for (int32_t i = 0; i < dv; ++i) {
                double acc = 0.0;
                for (int32_t j = 0; j < dk; ++j) acc += S[(size_t)i * dk + j] * qq[j];
                o[i] = acc;
            }
        }
    }

    if (J->out_state) {
        double *H = J->out_state + ((size_t)n * Hv + h) * dk * dv;
        for (int32_t j = 0; j < dk; ++j)
            for (int32_t i = 0; i < dv; ++i)
                H[(size_t)j * dv + i] = S[(size_t)i * dk + j];
    }
    free(S); free(Sk); free(kk); free(qq); free(vv);
}

static void *worker(void *arg)
{
    oracle_job *J = (oracle_job *)arg;
    const int64_t items = (int64_t)J->num_seqs * J->Hv;
    for (;;) {
        pthread_mutex_lock(&J->lock);
        int64_t it = J->next_item++;
        pthread_mutex_unlock(&J->lock);
        if (it >= items) break;
        run_chain(J, (int32_t)(it / J->Hv), (int32_t)(it % J->Hv));
    }
    return NULL;
}

static int run_job(oracle_job *Jp, int32_t num_threads);

/*
 * Returns 0 on success, -1 on bad arguments.  init_state may be NULL (zero start, Eq. 2);
 * out_o or out_state may be NULL to skip that output.  num_threads <= 1 runs inline.
 */
int gdn_oracle_forward(const float *q, const float *k, const float *v, const float *g,
                       const float *beta, const int32_t *cu, int32_t num_seqs, int32_t Hq,
                       int32_t Hv, int32_t dk, int32_t dv, const double *init_state,
                       double *out_o, double *out_state, int32_t num_threads)
{
    if (!q || !k || !v || !g || !beta || !cu) return -1;
    if (num_seqs < 0 || Hq <= 0 || Hv <= 0 || Hv % Hq != 0 || dk <= 0 || dv <= 0) return -1;
    for (int32_t n = 0; n < num_seqs; ++n)
        if (cu[n + 1] < cu[n]) return -1;

    oracle_job J;
    memset(&J, 0, sizeof J);
    J.q = q; J.k = k; J.v = v; J.g = g; J.beta = beta; J.cu = cu;
    J.num_seqs = num_seqs; J.Hq = Hq; J.Hv = Hv; J.dk = dk; J.dv = dv;
    J.init_state = init_state; J.out_o = out_o; J.out_state = out_state;
    return run_job(&J, num_threads);
}

/* The same recurrence on inputs that are already fp64 (what the fp64 input pipeline in front of it produces). */
int gdn_oracle_forward_f64(const double *q, const double *k, const double *v, const double *g,
                           const double *beta, const int32_t *cu, int32_t num_seqs, int32_t Hq,
                           int32_t Hv, int32_t dk, int32_t dv, const double *init_state,
                           double *out_o, double *out_state, int32_t num_threads)
{
    if (!q || !k || !v || !g || !beta || !cu) return -1;
    if (num_seqs < 0 || Hq <= 0 || Hv <= 0 || Hv % Hq != 0 || dk <= 0 || dv <= 0) return -1;
    for (int32_t n = 0; n < num_seqs; ++n)
        if (cu[n + 1] < cu[n]) return -1;

    oracle_job J;
    memset(&J, 0, sizeof J);
    J.qd = q; J.kd = k; J.vd = v; J.gd = g; J.betad = beta; J.cu = cu;
    J.num_seqs = num_seqs; J.Hq = Hq; J.Hv = Hv; J.dk = dk; J.dv = dv;
    J.init_state = init_state; J.out_o = out_o; J.out_state = out_state;
    return run_job(&J, num_threads);
}

static int run_job(oracle_job *Jp, int32_t num_threads)
{
    oracle_job J = *Jp;
    J.next_item = 0;
    pthread_mutex_init(&J.lock, NULL);

    if (num_threads <= 1) {
        worker(&J);
    } else {
        if (num_threads > 1024) num_threads = 1024;
        pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)num_threads);
        int started = 0;
        for (int i = 0; i < num_threads; ++i)
            if (pthread_create(&th[started], NULL, worker, &J) == 0) ++started;
        if (started == 0) worker(&J);
        for (int i = 0; i < started; ++i) pthread_join(th[i], NULL);
        free(th);
    }
    pthread_mutex_destroy(&J.lock);
    return 0;
}
