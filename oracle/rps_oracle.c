/*
 * CPU oracle for the RPS synchronisation step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, single-threaded
 * restatement of Algorithm 1 ("RPS") of "Distributed Learning over Unreliable
 * Networks" with all floating-point work in double precision.  It shares no
 * code, header, table or constant generator with the CUDA library and must
 * never be called from the product path: only the tests, the smoke check and
 * the benchmark's CPU-baseline leg use it.
 *
 * Notation follows the paper: n workers, model size d, drop probability p,
 * learning rate gamma, x_t^(i) the model of worker i, v_t^(i) the model after
 * the local SGD step, block j of the model is served by worker b_t^(j).
 *
 * Pins (see tests/test_oracle_*.py):
 *   philox4x32_10        published known-answer vectors (Salmon et al., SC'11)
 *   masks                p=0 / p=1 exact, drop rate, 1+Binomial(n-1,1-p) counts
 *   step                 X_{t+1} = V_t W_t (Eq. 3) for every drop pattern on tiny
 *                        n, with W checked against the exact sums printed in the
 *                        proofs of Lemmas 7 and 8; closed forms at p=0 and p=1
 *   noise                distribution tests against a library normal CDF; the
 *                        paper fixes only zero mean and bounded variance
 *                        (Assumption 1), so its exact values are a convention of
 *                        this implementation: parity unpinned by the paper for that part
 *   run, run_gradavg     equal to repeated single steps with step indices t0, t0+1, ... bit for
 *                        bit (a late, repeated or skipped index fails), cut points, closed form
 *   bf16 rounding        library conversion on random inputs
 *   alpha_mc             exact alpha_1, alpha_2 from all drop patterns on tiny n (within the
 *                        sampling error), 0 and 1 at p = 0 and p = 1, a second route to the
 *                        same per-sample value through counts of arrivals and receivers
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define RPS_ORACLE_F32 0
#define RPS_ORACLE_BF16 1

#define RPS_ORACLE_ASSIGN_FIXED 0 /* Section 4.1: worker i averages block i       */
#define RPS_ORACLE_ASSIGN_PERM 1  /* Algorithm 1: servers drawn without replacement */

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as    */
/* easy as 1, 2, 3", SC'11).  One round multiplies counter words 0 and 2 by    */
/* two fixed odd constants, and mixes the high halves with the other counter   */
/* words and the round key; the key grows by a Weyl constant between rounds.   */
/* ------------------------------------------------------------------------- */
void rps_oracle_philox4x32(const uint32_t ctr[4], const uint32_t key[2], int rounds, uint32_t out[4])
{
    const uint64_t mult_a = 0xD2511F53u;
    const uint64_t mult_b = 0xCD9E8D57u;
    const uint32_t weyl_a = 0x9E3779B9u;
    const uint32_t weyl_b = 0xBB67AE85u;
    uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int round = 0; round < rounds; ++round) {
        uint64_t prod_a = mult_a * (uint64_t)c[0];
        uint64_t prod_b = mult_b * (uint64_t)c[2];
        uint32_t next[4];
        next[0] = (uint32_t)(prod_b >> 32) ^ c[1] ^ k[0];
        next[1] = (uint32_t)prod_b;
        next[2] = (uint32_t)(prod_a >> 32) ^ c[3] ^ k[1];
        next[3] = (uint32_t)prod_a;
        memcpy(c, next, sizeof c);
        k[0] += weyl_a;
        k[1] += weyl_b;
    }
    memcpy(out, c, sizeof c);
}

void rps_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    rps_oracle_philox4x32(ctr, key, 10, out);
}

/* Counter layout shared by convention with the CUDA library (each side has its
 * own code for it): words 0,1 = step t; word 3's low byte tags the stream.     */
enum { STREAM_UP = 0, STREAM_DOWN = 1, STREAM_NOISE = 2, STREAM_PERM = 3 };

static void philox_draw_rounds(uint64_t seed, uint64_t t, uint32_t w2, uint32_t w3, int rounds, uint32_t out[4])
{
    uint32_t ctr[4] = {(uint32_t)t, (uint32_t)(t >> 32), w2, w3};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    rps_oracle_philox4x32(ctr, key, rounds, out);
}

/* Drop masks and the server draw use the standard ten rounds. */
static void philox_draw(uint64_t seed, uint64_t t, uint32_t w2, uint32_t w3, uint32_t out[4])
{
    philox_draw_rounds(seed, t, w2, w3, 10, out);
}

/* The gradient noise uses Philox4x32 with seven rounds, the fewest with which the generator's authors
 * report it passing their statistical test batteries (ten is their default, with a safety margin).
 * The paper asks of the noise only zero mean and bounded variance (Assumption 1). */
#define RPS_ORACLE_NOISE_ROUNDS 7

/* ------------------------------------------------------------------------- */
/* Unreliable channel (Section 3): every message is lost independently with    */
/* probability p.  A message is lost iff a fresh 32-bit draw is below          */
/* floor(p * 2^32); an integer compare, so p = 0 never drops and p = 1 always. */
/* ------------------------------------------------------------------------- */
static int message_lost(uint64_t seed, uint64_t t, int j, int i, int direction, double p)
{
    uint32_t r[4];
    philox_draw(seed, t, ((uint32_t)j << 16) | (uint32_t)i, (uint32_t)direction, r);
    uint64_t threshold = (uint64_t)floor(p * 4294967296.0);
    return (uint64_t)r[0] < threshold;
}

/* Which worker averages block j at step t (b_t^(j) of Algorithm 1). */
static void assign_servers(int n, uint64_t seed, uint64_t t, int assign, int32_t* server)
{
    for (int j = 0; j < n; ++j) server[j] = j;
    if (assign != RPS_ORACLE_ASSIGN_PERM) return;
    /* Fisher-Yates shuffle: every assignment of servers to blocks equally likely, no worker twice. */
    for (int k = n - 1; k >= 1; --k) {
        uint32_t r[4];
        philox_draw(seed, t, (uint32_t)k, STREAM_PERM, r);
        int pick = (int)(((uint64_t)r[0] * (uint64_t)(k + 1)) >> 32);
        int32_t tmp = server[k];
        server[k] = server[pick];
        server[pick] = tmp;
    }
}

/*
 * Drop masks of step t.  Bit i of up[j]   = worker i's block j reached its server.
 *                        Bit i of down[j] = worker i received the averaged block j.
 * With self_delivery the server's own copy never crosses the network, so its
 * two bits are always 1 (proof of Lemma 7: a server always holds its own copy of
 * the block; proof of Lemma 8, Case 2: a node's own block needs no message to
 * reach it).  Without it
 * all 2n messages of a block can be lost; if nothing arrives there is no
 * average to send, so nobody receives one (down = 0) and every worker keeps v.
 * cnt[j] = |N_t^(j)|.
 */
int rps_oracle_masks(int n, double p, uint64_t seed, uint64_t t, int self_delivery, int assign,
                     uint64_t* up, uint64_t* down, int32_t* cnt, int32_t* server)
{
    if (n < 1 || n > 64 || !(p >= 0.0 && p <= 1.0)) return -1;
    int32_t srv[64];
    assign_servers(n, seed, t, assign, srv);
    for (int j = 0; j < n; ++j) {
        uint64_t u = 0, dn = 0;
        for (int i = 0; i < n; ++i) {
            int arrived_up = !message_lost(seed, t, j, i, STREAM_UP, p);
            int arrived_down = !message_lost(seed, t, j, i, STREAM_DOWN, p);
            if (self_delivery && i == srv[j]) {
                arrived_up = 1;
                arrived_down = 1;
            }
            if (arrived_up) u |= (uint64_t)1 << i;
            if (arrived_down) dn |= (uint64_t)1 << i;
        }
        int c = 0;
        for (int i = 0; i < n; ++i) c += (int)((u >> i) & 1);
        if (c == 0) dn = 0;
        up[j] = u;
        down[j] = dn;
        cnt[j] = c;
        if (server) server[j] = srv[j];
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Gradient noise xi(t, i, c): a standard normal per (step, worker, column).   */
/* One 7-round Philox draw (four 32-bit words) serves a pair of workers (2k,     */
/* 2k+1) on                                                                     */
/* four consecutive columns 4q..4q+3.  Each word gives one Box-Muller pair:     */
/* its low 16 bits are the radius uniform, its high 16 bits the angle uniform,  */
/* both taken at bin centres (k + 1/2) / 2^16 so that neither is 0 or 1.       */
/* Words 0,1 -> worker 2k (columns 0,1 and 2,3); words 2,3 -> worker 2k+1.      */
/* ------------------------------------------------------------------------- */
double rps_oracle_noise(uint64_t seed, uint64_t t, int i, int64_t c)
{
    uint32_t r[4];
    int64_t q = c / 4;
    int e = (int)(c % 4);
    philox_draw_rounds(seed, t, (uint32_t)q, (uint32_t)STREAM_NOISE | ((uint32_t)(i / 2) << 8),
                       RPS_ORACLE_NOISE_ROUNDS, r);
    uint32_t word = r[(i % 2) * 2 + e / 2];
    double u_radius = ((double)(word & 0xFFFFu) + 0.5) / 65536.0;
    double u_angle = ((double)(word >> 16) + 0.5) / 65536.0;
    double radius = sqrt(-2.0 * log(u_radius));
    double angle = 2.0 * M_PI * u_angle;
    return (e % 2 == 0) ? radius * cos(angle) : radius * sin(angle);
}

/* ------------------------------------------------------------------------- */
/* Replica storage: float32, or bfloat16 bit patterns in uint16.               */
/* ------------------------------------------------------------------------- */
double rps_oracle_bf16_to_double(uint16_t bits)
{
    uint32_t wide = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &wide, sizeof f);
    return (double)f;
}

/* Round a double to the nearest bfloat16 (8 significant bits), ties to even,
 * in a single rounding.  Values here are far from overflow; tiny values round
 * on the subnormal grid 2^-133.                                                */
uint16_t rps_oracle_double_to_bf16(double v)
{
    if (v == 0.0 || v != v) {
        float f = (float)v;
        uint32_t w;
        memcpy(&w, &f, sizeof w);
        return (uint16_t)(w >> 16);
    }
    int exponent = ilogb(v);
    if (exponent < -126) exponent = -126;
    double scaled = ldexp(v, 7 - exponent); /* |scaled| in [128, 256) for normal results */
    double rounded = nearbyint(scaled);     /* default rounding mode: ties to even      */
    float f = (float)ldexp(rounded, exponent - 7);
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    return (uint16_t)(w >> 16);
}

static double load_elem(int dtype, const void* base, int64_t idx)
{
    if (dtype == RPS_ORACLE_BF16) return rps_oracle_bf16_to_double(((const uint16_t*)base)[idx]);
    return (double)((const float*)base)[idx];
}

static void store_elem(int dtype, void* base, int64_t idx, double v)
{
    if (dtype == RPS_ORACLE_BF16)
        ((uint16_t*)base)[idx] = rps_oracle_double_to_bf16(v);
    else
        ((float*)base)[idx] = (float)v; /* one rounding, to nearest even */
}

/* Step 0, model partitioning: n blocks of ceil(d/n) columns; the last
 * non-empty block is short and trailing blocks may be empty when n does not
 * divide d (the paper only treats equal blocks).                              */
int64_t rps_oracle_block_size(int n, int64_t d) { return (d + n - 1) / n; }

/*
 * One iteration of Algorithm 1 on dense [n][d] arrays x (updated in place) and
 * b (targets of the quadratic objective f_i(x) = 0.5 ||x - b_i||^2, so that
 * grad F_i(x; xi) = (x - b_i) + sigma * xi).
 *
 *   v^(i)      = x^(i) - gamma * grad F_i(x^(i); xi)                (local SGD)
 *   vtilde^(j) = 1/|N^(j)| * sum_{k in N^(j)} v^(k,j)               (RS step)
 *   x^(i,j)    = vtilde^(j) if worker i received it, else v^(i,j)    (AG step)
 *
 * gamma and sigma are first rounded to float, as the C ABI of the library does,
 * so that both sides use the same scalars.  forced_up/forced_down (both or
 * neither) replace the sampled masks; they are used as given.
 */
int rps_oracle_step(int n, int64_t d, int dtype, void* x, const void* b, double gamma, double sigma,
                    double p, uint64_t seed, uint64_t t, int self_delivery, int assign,
                    const uint64_t* forced_up, const uint64_t* forced_down)
{
    if (n < 1 || n > 64 || d < 1) return -1;
    uint64_t up[64], down[64];
    int32_t cnt[64];
    if (forced_up && forced_down) {
        for (int j = 0; j < n; ++j) {
            up[j] = forced_up[j];
            down[j] = forced_down[j];
            cnt[j] = 0;
            for (int i = 0; i < n; ++i) cnt[j] += (int)((up[j] >> i) & 1);
            if (cnt[j] == 0) down[j] = 0;
        }
    } else if (rps_oracle_masks(n, p, seed, t, self_delivery, assign, up, down, cnt, NULL) != 0) {
        return -1;
    }
    const double g = (double)(float)gamma;
    const double s = (double)(float)sigma;
    const int64_t block = rps_oracle_block_size(n, d);
    double v[64];
    for (int64_t c = 0; c < d; ++c) {
        const int j = (int)(c / block);
        for (int i = 0; i < n; ++i) {
            double xi = load_elem(dtype, x, (int64_t)i * d + c);
            double bi = load_elem(dtype, b, (int64_t)i * d + c);
            double grad = (xi - bi);
            if (s != 0.0) grad += s * rps_oracle_noise(seed, t, i, c);
            v[i] = xi - g * grad;
        }
        double vtilde = 0.0;
        if (cnt[j] > 0) {
            double sum = 0.0;
            for (int k = 0; k < n; ++k)
                if ((up[j] >> k) & 1) sum += v[k];
            vtilde = sum / (double)cnt[j];
        }
        for (int i = 0; i < n; ++i) {
            double out = ((down[j] >> i) & 1) ? vtilde : v[i];
            store_elem(dtype, x, (int64_t)i * d + c, out);
        }
    }
    return 0;
}

/* T iterations starting at step t0. */
int rps_oracle_run(int n, int64_t d, int dtype, void* x, const void* b, double gamma, double sigma,
                   double p, uint64_t seed, uint64_t t0, int64_t steps, int self_delivery, int assign)
{
    for (int64_t k = 0; k < steps; ++k) {
        int rc = rps_oracle_step(n, d, dtype, x, b, gamma, sigma, p, seed, t0 + (uint64_t)k,
                                 self_delivery, assign, NULL, NULL);
        if (rc != 0) return rc;
    }
    return 0;
}

/*
 * The step restricted to chosen columns, for spot checks at full size: cols[m]
 * lists column indices; x_cols / b_cols are dense [n][ncols] gathers of those
 * columns (x_cols updated in place).  Same arithmetic as rps_oracle_step, column
 * by column, with the block and the noise taken from the true column index.
 */
int rps_oracle_step_columns(int n, int64_t d, int dtype, int64_t ncols, const int64_t* cols,
                            void* x_cols, const void* b_cols, double gamma, double sigma, double p,
                            uint64_t seed, uint64_t t, int self_delivery, int assign)
{
    if (n < 1 || n > 64 || d < 1) return -1;
    uint64_t up[64], down[64];
    int32_t cnt[64];
    if (rps_oracle_masks(n, p, seed, t, self_delivery, assign, up, down, cnt, NULL) != 0) return -1;
    const double g = (double)(float)gamma;
    const double s = (double)(float)sigma;
    const int64_t block = rps_oracle_block_size(n, d);
    double v[64];
    for (int64_t m = 0; m < ncols; ++m) {
        const int64_t c = cols[m];
        if (c < 0 || c >= d) return -1;
        const int j = (int)(c / block);
        for (int i = 0; i < n; ++i) {
            double xi = load_elem(dtype, x_cols, (int64_t)i * ncols + m);
            double bi = load_elem(dtype, b_cols, (int64_t)i * ncols + m);
            double grad = (xi - bi);
            if (s != 0.0) grad += s * rps_oracle_noise(seed, t, i, c);
            v[i] = xi - g * grad;
        }
        double vtilde = 0.0;
        if (cnt[j] > 0) {
            double sum = 0.0;
            for (int k = 0; k < n; ++k)
                if ((up[j] >> k) & 1) sum += v[k];
            vtilde = sum / (double)cnt[j];
        }
        for (int i = 0; i < n; ++i) {
            double out = ((down[j] >> i) & 1) ? vtilde : v[i];
            store_elem(dtype, x_cols, (int64_t)i * ncols + m, out);
        }
    }
    return 0;
}

/*
 * Diagnostics used when tracking convergence: squared distance of the mean
 * model xbar to the optimum mean_i(b_i) of the quadratic objective, and the
 * consensus error sum_i ||x^(i) - xbar||^2 (the quantity bounded in Lemma 3).
 */
int rps_oracle_diag(int n, int64_t d, int dtype, const void* x, const void* b, double* dist2_to_opt,
                    double* consensus)
{
    double dist2 = 0.0, cons = 0.0;
    for (int64_t c = 0; c < d; ++c) {
        double xbar = 0.0, bbar = 0.0;
        for (int i = 0; i < n; ++i) {
            xbar += load_elem(dtype, x, (int64_t)i * d + c);
            bbar += load_elem(dtype, b, (int64_t)i * d + c);
        }
        xbar /= n;
        bbar /= n;
        dist2 += (xbar - bbar) * (xbar - bbar);
        for (int i = 0; i < n; ++i) {
            double dev = load_elem(dtype, x, (int64_t)i * d + c) - xbar;
            cons += dev * dev;
        }
    }
    *dist2_to_opt = dist2;
    *consensus = cons;
    return 0;
}

/*
 * The comparison method of Section 5 ("Comparison with Gradient Averaging"): the same unreliable
 * Reduce-Scatter / All-Gather, but what travels is the stochastic gradient instead of the model.
 *
 *   g^(i)      = grad F_i(x^(i); xi)
 *   gtilde^(j) = 1/|N^(j)| * sum_{k in N^(j)} g^(k,j)
 *   x^(i,j)    = x^(i,j) - gamma * gtilde^(j)   if worker i received it,
 *                x^(i,j) - gamma * g^(i,j)      otherwise (it applies its own gradient).
 *
 * The paper gives no formulas for it; this is the reading in which a worker that misses the average
 * still takes an SGD step.  Its point: a drop leaves a difference between replicas that nothing ever
 * removes, because the model is the sum of all earlier gradients.  Masks, noise and rounding are those
 * of rps_oracle_step.
 */
int rps_oracle_step_gradavg(int n, int64_t d, int dtype, void* x, const void* b, double gamma, double sigma,
                            double p, uint64_t seed, uint64_t t, int self_delivery, int assign,
                            const uint64_t* forced_up, const uint64_t* forced_down)
{
    if (n < 1 || n > 64 || d < 1) return -1;
    uint64_t up[64], down[64];
    int32_t cnt[64];
    if (forced_up && forced_down) {
        for (int j = 0; j < n; ++j) {
            up[j] = forced_up[j];
            down[j] = forced_down[j];
            cnt[j] = 0;
            for (int i = 0; i < n; ++i) cnt[j] += (int)((up[j] >> i) & 1);
            if (cnt[j] == 0) down[j] = 0;
        }
    } else if (rps_oracle_masks(n, p, seed, t, self_delivery, assign, up, down, cnt, NULL) != 0) {
        return -1;
    }
    const double lr = (double)(float)gamma;
    const double s = (double)(float)sigma;
    const int64_t block = rps_oracle_block_size(n, d);
    double xs[64], grad[64];
    for (int64_t c = 0; c < d; ++c) {
        const int j = (int)(c / block);
        for (int i = 0; i < n; ++i) {
            xs[i] = load_elem(dtype, x, (int64_t)i * d + c);
            grad[i] = xs[i] - load_elem(dtype, b, (int64_t)i * d + c);
            if (s != 0.0) grad[i] += s * rps_oracle_noise(seed, t, i, c);
        }
        double gtilde = 0.0;
        if (cnt[j] > 0) {
            double sum = 0.0;
            for (int k = 0; k < n; ++k)
                if ((up[j] >> k) & 1) sum += grad[k];
            gtilde = sum / (double)cnt[j];
        }
        for (int i = 0; i < n; ++i) {
            double applied = ((down[j] >> i) & 1) ? gtilde : grad[i];
            store_elem(dtype, x, (int64_t)i * d + c, xs[i] - lr * applied);
        }
    }
    return 0;
}

int rps_oracle_run_gradavg(int n, int64_t d, int dtype, void* x, const void* b, double gamma, double sigma,
                           double p, uint64_t seed, uint64_t t0, int64_t steps, int self_delivery, int assign)
{
    for (int64_t k = 0; k < steps; ++k) {
        int rc = rps_oracle_step_gradavg(n, d, dtype, x, b, gamma, sigma, p, seed, t0 + (uint64_t)k,
                                         self_delivery, assign, NULL, NULL);
        if (rc != 0) return rc;
    }
    return 0;
}

/*
 * Monte-Carlo estimate of the constants alpha_1 and alpha_2 of Eqs. (4) and (5),
 *   E[W W^T]     = alpha_1 I + (1 - alpha_1) A_n,     E[W A_n W^T] = alpha_2 I + (1 - alpha_2) A_n,
 * with A_n = 1 1^T / n and W = W_t^(j) the matrix of Eq. (3): X_{t+1}^(j) = V_t^(j) W_t^(j), column k
 * of W holding the weights with which worker k's new block j mixes the workers' v.  A matrix of
 * the form a I + (1 - a) A_n has a = (its diagonal entry) - (its off-diagonal entry), so each
 * sampled W contributes mean(diag M) - mean(offdiag M) for M = W W^T and M = W A_n W^T, and the
 * estimate is the mean over the n blocks of `steps` consecutive steps from t0.  Every matrix is
 * formed entry by entry and multiplied out with plain loops.  Needs n >= 2.
 */
int rps_oracle_alpha_mc(int n, double p, uint64_t seed, uint64_t t0, int64_t steps, int self_delivery, int assign,
                        double* alpha1, double* alpha2)
{
    if (n < 2 || n > 64 || steps < 1) return -1;
    uint64_t up[64], down[64];
    int32_t cnt[64], server[64];
    double* w = (double*)malloc(sizeof(double) * n * n * 4);
    if (!w) return -2;
    double* wa = w + n * n;   /* W A_n        */
    double* m1 = wa + n * n;  /* W W^T        */
    double* m2 = m1 + n * n;  /* W A_n W^T    */
    double sum1 = 0.0, sum2 = 0.0;
    for (int64_t s = 0; s < steps; ++s) {
        if (rps_oracle_masks(n, p, seed, t0 + (uint64_t)s, self_delivery, assign, up, down, cnt, server) != 0) {
            free(w);
            return -1;
        }
        for (int j = 0; j < n; ++j) {
            /* W[m][k]: weight of v^(m) in x_{t+1}^(k) for block j */
            for (int m = 0; m < n; ++m)
                for (int k = 0; k < n; ++k) {
                    const int received = (int)((down[j] >> k) & 1u);
                    const int arrived = (int)((up[j] >> m) & 1u);
                    w[m * n + k] = received ? (arrived ? 1.0 / cnt[j] : 0.0) : (m == k ? 1.0 : 0.0);
                }
            for (int m = 0; m < n; ++m)
                for (int k = 0; k < n; ++k) {
                    double acc = 0.0;
                    for (int l = 0; l < n; ++l) acc += w[m * n + l] * (1.0 / n);
                    wa[m * n + k] = acc;
                }
            for (int m = 0; m < n; ++m)
                for (int k = 0; k < n; ++k) {
                    double a1 = 0.0, a2 = 0.0;
                    for (int l = 0; l < n; ++l) {
                        a1 += w[m * n + l] * w[k * n + l];
                        a2 += wa[m * n + l] * w[k * n + l];
                    }
                    m1[m * n + k] = a1;
                    m2[m * n + k] = a2;
                }
            double d1 = 0.0, o1 = 0.0, d2 = 0.0, o2 = 0.0;
            for (int m = 0; m < n; ++m)
                for (int k = 0; k < n; ++k) {
                    if (m == k) {
                        d1 += m1[m * n + k];
                        d2 += m2[m * n + k];
                    } else {
                        o1 += m1[m * n + k];
                        o2 += m2[m * n + k];
                    }
                }
            sum1 += d1 / n - o1 / ((double)n * (n - 1));
            sum2 += d2 / n - o2 / ((double)n * (n - 1));
        }
    }
    free(w);
    *alpha1 = sum1 / ((double)steps * n);
    *alpha2 = sum2 / ((double)steps * n);
    return 0;
}
