/*
 * TEST INFRASTRUCTURE ONLY -- the fp64 CPU oracle for the multi-step Mamba
 * verification step.  Nothing on the product path may call into this file; it
 * exists so that the CUDA kernels can be compared, element by element, with a
 * slow and obviously correct statement of what the paper's method computes.
 * It shares no code, header, table or helper with the CUDA library.
 *
 * What is computed (paper sections in brackets):
 *
 *   linear RNN               h_t = Abar_t h_{t-1} + Bbar_t x_t ,  y_t = C_t^T h_t      [Eq. 1]
 *   on-the-fly discretising  Abar_t = exp(dt_t * A_h) ,  Bbar_t x_t = dt_t * B_t * x_t [Sec. 2.2,
 *                            "Discretize"; the zero-order-hold / Euler reading]
 *   MultiStep                from the cached state h_i run tokens i+1..k, return every
 *                            output and the state at the verified position j     [Sec. 4.2]
 *   fused verifier           i) replay of the tokens accepted last round, ii) the new
 *                            draft tokens, iii) caching of the state at j        [Sec. 4.3]
 *   rolling causal conv      the depthwise convolution in front of the SSM keeps a
 *                            window of the last W-1 inputs so that replayed tokens see
 *                            the right history                    [Sec. 4.3, footnote]
 *
 * The method is a re-scheduling of the plain recurrence, not an approximation,
 * so the oracle IS the plain recurrence: sequential over tokens, plain loops
 * over (sequence, head, row p, column n), double precision throughout, no
 * blocking and no re-association.  Threads (OpenMP) are only ever spread over
 * independent (sequence, head) pairs.
 *
 * Readings of points the paper leaves open (all of them are also listed in the
 * design document): scalar A per head and scalar dt per (token, head); the state
 * tile of a head is P x N with x,y carrying P and B,C carrying N; B and C are
 * shared by groups of heads (head h uses group h / (H/G)); dt arrives already
 * positive; the conv is depthwise over the H*P channels of x with a bias, tap
 * W-1 multiplies the current token, SiLU follows when enabled; the skip term
 * is D_h times the POST-conv x; the optional gate multiplies y by SiLU(z).
 *
 * A second parameterisation, "Mamba-1" (Algorithm 1, Sec. 2.2: a sampling interval
 * per channel and a dynamic A per (channel, state column), which is the form of
 * the pure-Mamba verifiers of Table 1), has its own functions at the end of the
 * file: oracle_verify_m1 / oracle_step_m1.  Reading taken there: the "N'" axis of
 * Algorithm 1 is the channel axis of a head (P here), so dt is [.. H*P], A is
 * [H*P][N] and the skip weight D is per channel.
 *
 * Pins: multi-step == repeated oracle_step; multi-round accept/replay ==
 * oracle_sequential; dt=0, B=0, A->0 closed forms; causal linear attention as
 * a matmul; explicit unrolled sums on tiny inputs; numpy full convolution.
 * Parity unpinned by the paper (pinned only by the readings above): tap order
 * of the conv, SiLU placement, the gate, the head->group mapping.
 *
 * Layouts (row-major, last index fastest):
 *   state       [Bt][H][P][N]           conv_state  [Bt][W-1][H*P]  (oldest row first)
 *   x, z, y     [Bt][Tmax][H][P]        dt          [Bt][Tmax][H]
 *   Bm          [Bt][Tmax][GB][N]       Cm          [Bt][Tmax][GC][N]
 *   A, D        [H]                     conv_w      [H*P][W]      conv_b [H*P]
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_FLAG_GATE 1      /* y <- y * SiLU(z)             */
#define ORACLE_FLAG_CONV_SILU 2 /* xc <- SiLU(conv(x) + bias)   */

typedef struct {
    int32_t Bt, Tmax, H, P, N, GB, GC, W, flags;
} oracle_dims;

static double silu(double v) { return v / (1.0 + exp(-v)); }

/* One token of one (sequence, head): the conv tap sum, the window shift, the
 * discretised recurrence on the P x N tile and the output row.  [Eq. 1, Sec. 2.2]
 *   win : [W-1][P] window of this head's channels, oldest first (updated)
 *   hh  : [P][N] state tile (updated)
 *   yrow: [P] output                                                      */
static void token_update(const oracle_dims *d, int h, double *win, double *hh,
                         const double *xin, double dt, const double *Brow, const double *Crow,
                         const double *zrow, double A_h, double D_h,
                         const double *conv_w, const double *conv_b, double *yrow, double *xc_scratch)
{
    const int P = d->P, N = d->N, W = d->W;
    for (int p = 0; p < P; ++p) {
        const int c = h * P + p;
        double acc = conv_b[c];
        for (int w = 0; w < W - 1; ++w) acc += conv_w[c * W + w] * win[w * P + p];
        acc += conv_w[c * W + (W - 1)] * xin[p];
        xc_scratch[p] = (d->flags & ORACLE_FLAG_CONV_SILU) ? silu(acc) : acc;
    }
    /* drop the oldest input, append the current one */
    for (int w = 0; w + 1 < W - 1; ++w)
        for (int p = 0; p < P; ++p) win[w * P + p] = win[(w + 1) * P + p];
    if (W > 1)
        for (int p = 0; p < P; ++p) win[(W - 2) * P + p] = xin[p];

    const double a = exp(dt * A_h);
    for (int p = 0; p < P; ++p)
        for (int n = 0; n < N; ++n)
            hh[p * N + n] = a * hh[p * N + n] + (dt * xc_scratch[p]) * Brow[n];
    for (int p = 0; p < P; ++p) {
        double s = 0.0;
        for (int n = 0; n < N; ++n) s += Crow[n] * hh[p * N + n];
        s += D_h * xc_scratch[p];
        if ((d->flags & ORACLE_FLAG_GATE) && zrow) s *= silu(zrow[p]);
        yrow[p] = s;
    }
}

/*
 * The verification call [Sec. 4.2 MultiStep, Sec. 4.3 i)-iii)].
 * For sequence b: T_b = n_prev[b] + k tokens are run from the cached state;
 * the state and the conv window as they stand after token n_prev[b]-1 go to
 * state_out / conv_state_out (copies of the inputs when n_prev[b] == 0); y gets
 * rows 0..T_b-1 of sequence b and is not touched beyond them.
 * Returns 0, or -1 if some n_prev[b] < 0 or n_prev[b] + k > Tmax.
 */
int oracle_verify(const oracle_dims *d, int32_t k, const int32_t *n_prev,
                  const double *state, const double *conv_state,
                  const double *x, const double *dt, const double *Bm, const double *Cm,
                  const double *A, const double *D,
                  const double *conv_w, const double *conv_b, const double *z,
                  double *y, double *state_out, double *conv_state_out, int32_t nthreads)
{
    const int Bt = d->Bt, Tmax = d->Tmax, H = d->H, P = d->P, N = d->N, W = d->W;
    const int C = H * P;
    for (int b = 0; b < Bt; ++b)
        if (n_prev[b] < 0 || n_prev[b] + k > Tmax) return -1;
    if (nthreads < 1) nthreads = 1;

#pragma omp parallel for collapse(2) num_threads(nthreads) schedule(dynamic, 1)
    for (int b = 0; b < Bt; ++b) {
        for (int h = 0; h < H; ++h) {
            const int j = n_prev[b], T = j + k;
            const int gB = h / (H / d->GB), gC = h / (H / d->GC);
            double *hh = (double *)malloc(sizeof(double) * P * N);
            double *win = (double *)malloc(sizeof(double) * (W > 1 ? (W - 1) : 1) * P);
            double *xc = (double *)malloc(sizeof(double) * P);
            const double *st_in = state + ((size_t)b * H + h) * P * N;
            double *st_out = state_out + ((size_t)b * H + h) * P * N;
            memcpy(hh, st_in, sizeof(double) * P * N);
            for (int w = 0; w < W - 1; ++w)
                for (int p = 0; p < P; ++p)
                    win[w * P + p] = conv_state[((size_t)b * (W - 1) + w) * C + h * P + p];
            if (j == 0) { /* nothing newly accepted: the cache is carried over as it is */
                memcpy(st_out, st_in, sizeof(double) * P * N);
                for (int w = 0; w < W - 1; ++w)
                    for (int p = 0; p < P; ++p)
                        conv_state_out[((size_t)b * (W - 1) + w) * C + h * P + p] = win[w * P + p];
            }
            for (int t = 0; t < T; ++t) {
                const size_t bt = (size_t)b * Tmax + t;
                token_update(d, h, win, hh, x + (bt * H + h) * P, dt[bt * H + h],
                             Bm + (bt * d->GB + gB) * N, Cm + (bt * d->GC + gC) * N,
                             z ? z + (bt * H + h) * P : NULL, A[h], D[h], conv_w, conv_b,
                             y + (bt * H + h) * P, xc);
                if (t == j - 1) { /* snapshot at the newly verified position */
                    memcpy(st_out, hh, sizeof(double) * P * N);
                    for (int w = 0; w < W - 1; ++w)
                        for (int p = 0; p < P; ++p)
                            conv_state_out[((size_t)b * (W - 1) + w) * C + h * P + p] = win[w * P + p];
                }
            }
            free(hh); free(win); free(xc);
        }
    }
    return 0;
}

/*
 * Single-token decoding step, written on its own (it does not call
 * token_update): every sequence advances by exactly one token, in place.
 * The conv is done for all channels first, then the recurrence.  [Eq. 1]
 *   x1,z1,y1 : [Bt][H][P]   dt1 : [Bt][H]   B1 : [Bt][GB][N]   C1 : [Bt][GC][N]
 *   active   : [Bt] (nullable) -- sequences with active[b]==0 are left alone.
 */
int oracle_step(const oracle_dims *d, double *state, double *conv_state,
                const double *x1, const double *dt1, const double *B1, const double *C1,
                const double *A, const double *D, const double *conv_w, const double *conv_b,
                const double *z1, double *y1, const int32_t *active)
{
    const int Bt = d->Bt, H = d->H, P = d->P, N = d->N, W = d->W, C = H * P;
    double *u = (double *)malloc(sizeof(double) * C); /* post-conv x of one sequence */
    for (int b = 0; b < Bt; ++b) {
        if (active && !active[b]) continue;
        double *cs = conv_state + (size_t)b * (W - 1) * C;
        for (int c = 0; c < C; ++c) {
            double s = conv_w[c * W + W - 1] * x1[(size_t)b * C + c] + conv_b[c];
            for (int w = 0; w < W - 1; ++w) s += conv_w[c * W + w] * cs[(size_t)w * C + c];
            u[c] = (d->flags & ORACLE_FLAG_CONV_SILU) ? s / (1.0 + exp(-s)) : s;
        }
        for (int w = 0; w < W - 2; ++w)
            memcpy(cs + (size_t)w * C, cs + (size_t)(w + 1) * C, sizeof(double) * C);
        if (W > 1) memcpy(cs + (size_t)(W - 2) * C, x1 + (size_t)b * C, sizeof(double) * C);

        for (int h = 0; h < H; ++h) {
            const double delta = dt1[(size_t)b * H + h];
            const double decay = exp(delta * A[h]);
            const double *Bv = B1 + ((size_t)b * d->GB + h / (H / d->GB)) * N;
            const double *Cv = C1 + ((size_t)b * d->GC + h / (H / d->GC)) * N;
            double *S = state + ((size_t)b * H + h) * P * N;
            for (int p = 0; p < P; ++p) {
                const double xin = u[h * P + p];
                double out = D[h] * xin;
                for (int n = 0; n < N; ++n) {
                    S[p * N + n] = decay * S[p * N + n] + delta * Bv[n] * xin;
                    out += S[p * N + n] * Cv[n];
                }
                if ((d->flags & ORACLE_FLAG_GATE) && z1) {
                    const double g = z1[((size_t)b * H + h) * P + p];
                    out *= g / (1.0 + exp(-g));
                }
                y1[((size_t)b * H + h) * P + p] = out;
            }
        }
    }
    free(u);
    return 0;
}

/*
 * Direct sequential run over a stream of tokens with no speculation at all:
 * sequence b consumes its first len[b] tokens one oracle_step at a time, in
 * place.  This is what accept-then-advance must reproduce.  [Sec. 4.2, Alg. 2]
 *   x,z,y : [Bt][L][H][P]   dt : [Bt][L][H]   Bm : [Bt][L][GB][N]   Cm : [Bt][L][GC][N]
 * Threads are spread over sequences only.
 */
int oracle_sequential(const oracle_dims *d, int32_t L, const int32_t *len,
                      double *state, double *conv_state,
                      const double *x, const double *dt, const double *Bm, const double *Cm,
                      const double *A, const double *D, const double *conv_w, const double *conv_b,
                      const double *z, double *y, int32_t nthreads)
{
    const int Bt = d->Bt, H = d->H, P = d->P, N = d->N, W = d->W, C = H * P;
    for (int b = 0; b < Bt; ++b)
        if (len[b] < 0 || len[b] > L) return -1;
    if (nthreads < 1) nthreads = 1;
    oracle_dims one = *d;
    one.Bt = 1;
#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
    for (int b = 0; b < Bt; ++b) {
        for (int t = 0; t < len[b]; ++t) {
            const size_t bt = (size_t)b * L + t;
            oracle_step(&one, state + (size_t)b * H * P * N, conv_state + (size_t)b * (W - 1) * C,
                        x + bt * C, dt + bt * H, Bm + bt * d->GB * N, Cm + bt * d->GC * N,
                        A, D, conv_w, conv_b, z ? z + bt * C : NULL, y + bt * C, NULL);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Mamba-1 parameterisation [Algorithm 1, Sec. 2.2]: the sampling interval is per channel and the
 * dynamic A per (channel, state column):
 *     h_t[p][n] = exp(dt_t[c] * A[c][n]) * h_{t-1}[p][n] + dt_t[c] * xc_t[p] * B_t[n],   c = h*P + p
 *     y_t[p]    = sum_n C_t[n] * h_t[p][n] + D[c] * xc_t[p]        ( * SiLU(z_t[p]) when gated )
 * Everything else (conv, groups, snapshot at the verified position) is as in oracle_verify.
 * Layouts that differ:  dt [Bt][Tmax][H*P]   A [H*P][N]   D [H*P]
 */
int oracle_verify_m1(const oracle_dims *d, int32_t k, const int32_t *n_prev,
                     const double *state, const double *conv_state,
                     const double *x, const double *dt, const double *Bm, const double *Cm,
                     const double *A, const double *D,
                     const double *conv_w, const double *conv_b, const double *z,
                     double *y, double *state_out, double *conv_state_out, int32_t nthreads)
{
    const int Bt = d->Bt, Tmax = d->Tmax, H = d->H, P = d->P, N = d->N, W = d->W;
    const int C = H * P;
    for (int b = 0; b < Bt; ++b)
        if (n_prev[b] < 0 || n_prev[b] + k > Tmax) return -1;
    if (nthreads < 1) nthreads = 1;

#pragma omp parallel for collapse(2) num_threads(nthreads) schedule(dynamic, 1)
    for (int b = 0; b < Bt; ++b) {
        for (int c = 0; c < C; ++c) { /* every channel is its own recurrence */
            const int h = c / P, j = n_prev[b], T = j + k;
            const int gB = h / (H / d->GB), gC = h / (H / d->GC);
            double hrow[1024]; /* N <= 1024 checked by the caller */
            double win[16];
            const double *st_in = state + ((size_t)b * C + c) * N;
            double *st_out = state_out + ((size_t)b * C + c) * N;
            for (int n = 0; n < N; ++n) hrow[n] = st_in[n];
            for (int w = 0; w < W - 1; ++w) win[w] = conv_state[((size_t)b * (W - 1) + w) * C + c];
            if (j == 0) {
                for (int n = 0; n < N; ++n) st_out[n] = hrow[n];
                for (int w = 0; w < W - 1; ++w) conv_state_out[((size_t)b * (W - 1) + w) * C + c] = win[w];
            }
            for (int t = 0; t < T; ++t) {
                const size_t bt = (size_t)b * Tmax + t;
                const double xin = x[bt * C + c];
                double u = conv_b[c] + conv_w[c * W + (W - 1)] * xin;
                for (int w = 0; w < W - 1; ++w) u += conv_w[c * W + w] * win[w];
                if (d->flags & ORACLE_FLAG_CONV_SILU) u = silu(u);
                for (int w = 0; w + 1 < W - 1; ++w) win[w] = win[w + 1];
                if (W > 1) win[W - 2] = xin;
                const double delta = dt[bt * C + c];
                const double *Brow = Bm + (bt * d->GB + gB) * N, *Crow = Cm + (bt * d->GC + gC) * N;
                double out = 0.0;
                for (int n = 0; n < N; ++n) {
                    hrow[n] = exp(delta * A[(size_t)c * N + n]) * hrow[n] + delta * u * Brow[n];
                    out += Crow[n] * hrow[n];
                }
                out += D[c] * u;
                if ((d->flags & ORACLE_FLAG_GATE) && z) out *= silu(z[bt * C + c]);
                y[bt * C + c] = out;
                if (t == j - 1) {
                    for (int n = 0; n < N; ++n) st_out[n] = hrow[n];
                    for (int w = 0; w < W - 1; ++w) conv_state_out[((size_t)b * (W - 1) + w) * C + c] = win[w];
                }
            }
        }
    }
    return 0;
}

/*
 * One decoding step in the Mamba-1 parameterisation, written on its own: the whole batch goes through
 * the conv first, then through the decay, then through the input term, then through the read-out, each
 * as a separate sweep (another order of the same arithmetic than oracle_verify_m1's).  In place.
 *   x1,z1,y1,dt1 : [Bt][H*P]   B1 : [Bt][GB][N]   C1 : [Bt][GC][N]
 */
int oracle_step_m1(const oracle_dims *d, double *state, double *conv_state,
                   const double *x1, const double *dt1, const double *B1, const double *C1,
                   const double *A, const double *D, const double *conv_w, const double *conv_b,
                   const double *z1, double *y1)
{
    const int Bt = d->Bt, H = d->H, P = d->P, N = d->N, W = d->W, C = H * P;
    double *u = (double *)malloc(sizeof(double) * (size_t)Bt * C);
    for (int b = 0; b < Bt; ++b)
        for (int c = 0; c < C; ++c) {
            double s = conv_b[c];
            for (int w = 0; w < W; ++w)
                s += conv_w[c * W + w] * (w < W - 1 ? conv_state[((size_t)b * (W - 1) + w) * C + c] : x1[(size_t)b * C + c]);
            u[(size_t)b * C + c] = (d->flags & ORACLE_FLAG_CONV_SILU) ? s / (1.0 + exp(-s)) : s;
        }
    for (int b = 0; b < Bt; ++b) {
        double *cs = conv_state + (size_t)b * (W - 1) * C;
        for (int w = 0; w < W - 2; ++w) memcpy(cs + (size_t)w * C, cs + (size_t)(w + 1) * C, sizeof(double) * C);
        if (W > 1) memcpy(cs + (size_t)(W - 2) * C, x1 + (size_t)b * C, sizeof(double) * C);
    }
    for (int b = 0; b < Bt; ++b)        /* decay */
        for (int c = 0; c < C; ++c)
            for (int n = 0; n < N; ++n)
                state[((size_t)b * C + c) * N + n] *= exp(A[(size_t)c * N + n] * dt1[(size_t)b * C + c]);
    for (int b = 0; b < Bt; ++b)        /* input term */
        for (int c = 0; c < C; ++c) {
            const double *Bv = B1 + ((size_t)b * d->GB + (c / P) / (H / d->GB)) * N;
            const double scale = dt1[(size_t)b * C + c] * u[(size_t)b * C + c];
            for (int n = 0; n < N; ++n) state[((size_t)b * C + c) * N + n] += Bv[n] * scale;
        }
    for (int b = 0; b < Bt; ++b)        /* read-out */
        for (int c = 0; c < C; ++c) {
            const double *Cv = C1 + ((size_t)b * d->GC + (c / P) / (H / d->GC)) * N;
            double out = D[c] * u[(size_t)b * C + c];
            for (int n = 0; n < N; ++n) out += Cv[n] * state[((size_t)b * C + c) * N + n];
            if ((d->flags & ORACLE_FLAG_GATE) && z1) {
                const double g = z1[(size_t)b * C + c];
                out *= g / (1.0 + exp(-g));
            }
            y1[(size_t)b * C + c] = out;
        }
    free(u);
    return 0;
}
