/*
 * CPU oracle for the Mamba drafter's conv1d + selective-SSM (S6) + gate path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, sequential, fp64 statement
 * of what the path computes.  It shares no code with the CUDA library and is
 * never called from the product path; only the tests, the smoke check and the
 * benchmark's CPU-baseline leg use it.
 *
 * What it follows.  The paper uses Mamba as its drafter by citation (Section
 * 3.1) and adds tree-structured drafting in which a child node needs nothing
 * but its parent's recurrent state (Section 4.1).  The recurrence itself is the
 * selective SSM in its standard form, per channel d and state index n:
 *
 *     u_t      = SiLU( b_d + sum_{k=0..W-1} w[d][k] * x[t-(W-1)+k] )      (causal depthwise conv, tap W-1 = current token)
 *     Delta_t  = softplus( dt_t + dt_bias[d] )                            (or dt_t + dt_bias[d] as given, when the flag is off)
 *     h_t[n]   = exp(Delta_t * A[d][n]) * h_{t-1}[n] + Delta_t * B_t[n] * u_t
 *     y_t      = sum_n C_t[n] * h_t[n] + D[d] * u_t
 *     out_t    = y_t * SiLU(z_t)
 *
 * State carried between calls: h (D x N) and the last W-1 raw inputs x of each
 * channel (the conv window), oldest first.
 *
 * Every loop below is the definition written out: one token after another, no
 * chunking, no reordering.  Threads (OpenMP) split the independent channels
 * only; the arithmetic of a channel is untouched by the thread count.
 *
 * Parity pins (tests/test_oracle_pins.py): geometric-series closed form,
 * A = 0 cumulative sum, Delta = 0 frozen state, O(T^2) explicit products on
 * tiny inputs, scipy.signal.lfilter for the time-invariant case, numpy.convolve
 * and an impulse response for the conv, scalar identities for SiLU/softplus,
 * prefill hand-off, prefill == chain of steps, tree node == its root-to-node
 * path run as one short sequence, packed == each sequence alone; for the tree
 * with the block's projections: equality with the plain tree fed by numpy's
 * matmul of the conv outputs, one-hot weights that turn both projections into
 * gathers, zero weights (closed-form decay).  The paper prints no numeric value
 * for this path, so no pin comes from a printed table.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum {
    MDO_DT_SOFTPLUS = 1, /* Delta = softplus(dt + dt_bias), else Delta = dt + dt_bias */
    MDO_PRECONV     = 2, /* x already is u: no conv, conv window untouched            */
    MDO_CONV_ONLY   = 4  /* out = u; the recurrence is not run                        */
};

typedef struct {
    int32_t d_inner, d_state, d_conv;
    uint32_t flags;
    const double *A;       /* (D, N) */
    const double *Dskip;   /* (D) or NULL = 0 */
    const double *conv_w;  /* (D, W) */
    const double *conv_b;  /* (D) or NULL = 0 */
    const double *dt_bias; /* (D) or NULL = 0 */
} mdo_layer;

double mdo_silu(double v) { return v / (1.0 + exp(-v)); }

double mdo_softplus(double v) { return log1p(exp(v)); }

int mdo_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
    return omp_get_max_threads();
#else
    (void)n;
    return 1;
#endif
}

/*
 * One token of one channel.  win[0..W-2] holds the previous W-1 raw inputs
 * (oldest first), h[0..N-1] the state; both are advanced in place.
 */
static double channel_token(const mdo_layer *L, int d, double *win, double *h,
                            double x, double z, double dt, const double *Bt, const double *Ct)
{
    const int N = L->d_state, W = L->d_conv;
    double u;
    if (L->flags & MDO_PRECONV) {
        u = x;
    } else {
        double acc = L->conv_b ? L->conv_b[d] : 0.0;
        for (int k = 0; k < W - 1; ++k) acc += L->conv_w[(size_t)d * W + k] * win[k];
        acc += L->conv_w[(size_t)d * W + (W - 1)] * x;
        for (int k = 0; k + 1 < W - 1; ++k) win[k] = win[k + 1];
        if (W > 1) win[W - 2] = x;
        u = mdo_silu(acc);
    }
    if (L->flags & MDO_CONV_ONLY) return u;

    double v = dt + (L->dt_bias ? L->dt_bias[d] : 0.0);
    double delta = (L->flags & MDO_DT_SOFTPLUS) ? mdo_softplus(v) : v;
    double y = 0.0;
    for (int n = 0; n < N; ++n) {
        h[n] = exp(delta * L->A[(size_t)d * N + n]) * h[n] + delta * Bt[n] * u;
        y += Ct[n] * h[n];
    }
    y += (L->Dskip ? L->Dskip[d] : 0.0) * u;
    return y * mdo_silu(z);
}

/*
 * Context encode.  Sequences are packed: tokens of sequence s are rows
 * cu_seqlens[s] .. cu_seqlens[s+1]-1 of x, z, dt (T x D) and B, C (T x N).
 * conv_init: (n_seq, W-1, D) or NULL (zeros); h_init: (n_seq, D, N) or NULL.
 * out: (T, D).  conv_final (n_seq, W-1, D) and h_final (n_seq, D, N) may be NULL.
 */
void mdo_prefill(const mdo_layer *L, int n_seq, const int32_t *cu_seqlens,
                 const double *x, const double *z, const double *dt,
                 const double *B, const double *C,
                 const double *conv_init, const double *h_init,
                 double *out, double *conv_final, double *h_final)
{
    const int D = L->d_inner, N = L->d_state, W = L->d_conv;
    for (int s = 0; s < n_seq; ++s) {
        const int t0 = cu_seqlens[s], t1 = cu_seqlens[s + 1];
#pragma omp parallel for schedule(static)
        for (int d = 0; d < D; ++d) {
            double win[16], h[256];
            for (int k = 0; k < W - 1; ++k)
                win[k] = conv_init ? conv_init[((size_t)s * (W - 1) + k) * D + d] : 0.0;
            for (int n = 0; n < N; ++n)
                h[n] = h_init ? h_init[((size_t)s * D + d) * N + n] : 0.0;
            for (int t = t0; t < t1; ++t)
                out[(size_t)t * D + d] = channel_token(L, d, win, h, x[(size_t)t * D + d], z[(size_t)t * D + d],
                                                       dt[(size_t)t * D + d], B + (size_t)t * N, C + (size_t)t * N);
            if (conv_final)
                for (int k = 0; k < W - 1; ++k) conv_final[((size_t)s * (W - 1) + k) * D + d] = win[k];
            if (h_final)
                for (int n = 0; n < N; ++n) h_final[((size_t)s * D + d) * N + n] = h[n];
        }
    }
}

/*
 * Tree drafting for one sequence, path by path.  parent[i] is the tree-local
 * parent of node i (-1: the committed state conv0 / h0).  For EVERY node v the
 * root-to-v path is rebuilt and run token by token from the committed state;
 * out[v] and the state after v are what that run leaves.  Deliberately
 * redundant (cost ~ nodes x depth): no node's result depends on another node's
 * stored result.
 * x, z, dt: (M, D); B, C: (M, N); conv0: (W-1, D) or NULL; h0: (D, N) or NULL.
 * out: (M, D); conv_nodes: (M, W-1, D) or NULL; h_nodes: (M, D, N) or NULL.
 * Returns 0, or -1 if a parent index is not an earlier node.
 */
int mdo_tree(const mdo_layer *L, int M, const int32_t *parent,
             const double *x, const double *z, const double *dt,
             const double *B, const double *C,
             const double *conv0, const double *h0,
             double *out, double *conv_nodes, double *h_nodes)
{
    const int D = L->d_inner, N = L->d_state, W = L->d_conv;
    for (int v = 0; v < M; ++v)
        if (parent[v] >= v || parent[v] < -1) return -1;
    int *path = (int *)malloc(sizeof(int) * (size_t)(M > 0 ? M : 1));
    for (int v = 0; v < M; ++v) {
        int len = 0;
        for (int a = v; a >= 0; a = parent[a]) path[len++] = a; /* v, parent(v), ..., root */
#pragma omp parallel for schedule(static)
        for (int d = 0; d < D; ++d) {
            double win[16], h[256], o = 0.0;
            for (int k = 0; k < W - 1; ++k) win[k] = conv0 ? conv0[(size_t)k * D + d] : 0.0;
            for (int n = 0; n < N; ++n) h[n] = h0 ? h0[(size_t)d * N + n] : 0.0;
            for (int j = len - 1; j >= 0; --j) {
                const size_t a = (size_t)path[j];
                o = channel_token(L, d, win, h, x[a * D + d], z[a * D + d], dt[a * D + d], B + a * N, C + a * N);
            }
            out[(size_t)v * D + d] = o;
            if (conv_nodes)
                for (int k = 0; k < W - 1; ++k) conv_nodes[((size_t)v * (W - 1) + k) * D + d] = win[k];
            if (h_nodes)
                for (int n = 0; n < N; ++n) h_nodes[((size_t)v * D + d) * N + n] = h[n];
        }
    }
    free(path);
    return 0;
}

/*
 * Tree drafting with the block's own selection projections.  The drafter is a
 * Mamba model (paper Section 3.1, by citation), and in that block the step
 * size, B and C of a token are not inputs: they are linear functions of the
 * token's conv output u (all D channels of it),
 *
 *     s        = Wx * u                      Wx: (R + 2N, D)
 *     dt[d]    = sum_{r<R} Wdt[d][r] * s[r]   Wdt: (D, R)     (dt_bias and softplus are applied as above)
 *     B[n]     = s[R + n]
 *     C[n]     = s[R + N + n]
 *
 * so a node is: conv step on every channel, the two projections, then the
 * recurrence and the gate on every channel.  As in mdo_tree every node is
 * rebuilt along its root-to-node path from the committed state (Section 4.1:
 * a child needs only its parent's state).
 *
 * x, z: (M, D); out: (M, D); conv_nodes (M, W-1, D), h_nodes (M, D, N),
 * dt_nodes (M, D), B_nodes (M, N), C_nodes (M, N) may each be NULL.
 * Returns 0, or -1 if a parent index is not an earlier node.
 */
int mdo_tree_proj(const mdo_layer *L, int R, const double *Wx, const double *Wdt,
                  int M, const int32_t *parent, const double *x, const double *z,
                  const double *conv0, const double *h0,
                  double *out, double *conv_nodes, double *h_nodes,
                  double *dt_nodes, double *B_nodes, double *C_nodes)
{
    const int D = L->d_inner, N = L->d_state, W = L->d_conv;
    for (int v = 0; v < M; ++v)
        if (parent[v] >= v || parent[v] < -1) return -1;
    mdo_layer conv_part = *L, scan_part = *L;
    conv_part.flags = (L->flags & ~(uint32_t)MDO_PRECONV) | MDO_CONV_ONLY;
    scan_part.flags = (L->flags & ~(uint32_t)MDO_CONV_ONLY) | MDO_PRECONV;
    int *path = (int *)malloc(sizeof(int) * (size_t)(M > 0 ? M : 1));
    double *win = (double *)malloc(sizeof(double) * (size_t)(W > 1 ? W - 1 : 1) * D);
    double *h = (double *)malloc(sizeof(double) * (size_t)D * N);
    double *u = (double *)malloc(sizeof(double) * (size_t)D);
    double *dt = (double *)malloc(sizeof(double) * (size_t)D);
    double *s = (double *)malloc(sizeof(double) * (size_t)(R + 2 * N));
    for (int v = 0; v < M; ++v) {
        int len = 0;
        for (int a = v; a >= 0; a = parent[a]) path[len++] = a;
        for (int d = 0; d < D; ++d) {
            for (int k = 0; k < W - 1; ++k) win[(size_t)d * (W - 1) + k] = conv0 ? conv0[(size_t)k * D + d] : 0.0;
            for (int n = 0; n < N; ++n) h[(size_t)d * N + n] = h0 ? h0[(size_t)d * N + n] : 0.0;
        }
        for (int j = len - 1; j >= 0; --j) {
            const size_t a = (size_t)path[j];
            for (int d = 0; d < D; ++d)
                u[d] = channel_token(&conv_part, d, win + (size_t)d * (W - 1), NULL, x[a * D + d], 0.0, 0.0, NULL, NULL);
            for (int r = 0; r < R + 2 * N; ++r) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += Wx[(size_t)r * D + d] * u[d];
                s[r] = acc;
            }
            for (int d = 0; d < D; ++d) {
                double acc = 0.0;
                for (int r = 0; r < R; ++r) acc += Wdt[(size_t)d * R + r] * s[r];
                dt[d] = acc;
            }
            for (int d = 0; d < D; ++d)
                out[(size_t)v * D + d] = channel_token(&scan_part, d, NULL, h + (size_t)d * N, u[d], z[a * D + d], dt[d], s + R, s + R + N);
        }
        for (int d = 0; d < D; ++d) {
            if (conv_nodes)
                for (int k = 0; k < W - 1; ++k) conv_nodes[((size_t)v * (W - 1) + k) * D + d] = win[(size_t)d * (W - 1) + k];
            if (h_nodes)
                for (int n = 0; n < N; ++n) h_nodes[((size_t)v * D + d) * N + n] = h[(size_t)d * N + n];
            if (dt_nodes) dt_nodes[(size_t)v * D + d] = dt[d];
        }
        for (int n = 0; n < N; ++n) {
            if (B_nodes) B_nodes[(size_t)v * N + n] = s[R + n];
            if (C_nodes) C_nodes[(size_t)v * N + n] = s[R + N + n];
        }
    }
    free(path); free(win); free(h); free(u); free(dt); free(s);
    return 0;
}

/*
 * ---------------------------------------------------------------------------------------------------------
 * Mamba-2 (SSD) drafter: the same path with ONE scalar A per head.
 *
 * The paper names Mamba-2 as the drop-in that "directly benefits" the approach (Section 1, the paragraph before
 * Related Work) and defines nothing about it; the recurrence below is the state-space-duality form of the cited
 * model, kept as close to the S6 statement above as it goes.  The D channels are split into H = D / P heads of P
 * channels (d = j * P + p); the step size and A are per HEAD, B and C are shared by all heads (one group):
 *
 *     u_t[d]     = SiLU( b_d + sum_k w[d][k] * x[t-(W-1)+k][d] )              (as above, per channel)
 *     Delta_t[j] = softplus( dt_t[j] + dt_bias[j] )                           (or as given, when the flag is off)
 *     h_t[d][n]  = exp(Delta_t[j] * A[j]) * h_{t-1}[d][n] + Delta_t[j] * B_t[n] * u_t[d]
 *     y_t[d]     = sum_n C_t[n] * h_t[d][n] + D[d] * u_t[d]
 *     out_t[d]   = y_t[d] * SiLU(z_t[d])
 *
 * Written out token by token, channel by channel: no chunking, no matrix form.  Pins (tests/pins.py): with every
 * head's A copied to all N states of its P channels and dt copied to the head's channels this IS mdo_prefill /
 * mdo_tree (which have their own pins); geometric series and cumulative sum in closed form; head indexing by an
 * input that differs in one head only.
 */
typedef struct {
    int32_t d_inner, headdim, d_state, d_conv;
    uint32_t flags;
    const double *A;       /* (H)  one scalar per head, <= 0 */
    const double *Dskip;   /* (D) or NULL = 0 */
    const double *conv_w;  /* (D, W) */
    const double *conv_b;  /* (D) or NULL = 0 */
    const double *dt_bias; /* (H) or NULL = 0 */
} mdo_ssd_layer;

/* One token of one channel of head j = d / P.  dt is the head's pre-activation for this token. */
static double ssd_channel_token(const mdo_ssd_layer *L, int d, double *win, double *h,
                                double x, double z, double dt, const double *Bt, const double *Ct)
{
    const int N = L->d_state, W = L->d_conv, j = d / L->headdim;
    double u;
    if (L->flags & MDO_PRECONV) {
        u = x;
    } else {
        double acc = L->conv_b ? L->conv_b[d] : 0.0;
        for (int k = 0; k < W - 1; ++k) acc += L->conv_w[(size_t)d * W + k] * win[k];
        acc += L->conv_w[(size_t)d * W + (W - 1)] * x;
        for (int k = 0; k + 1 < W - 1; ++k) win[k] = win[k + 1];
        if (W > 1) win[W - 2] = x;
        u = mdo_silu(acc);
    }
    if (L->flags & MDO_CONV_ONLY) return u;
    double v = dt + (L->dt_bias ? L->dt_bias[j] : 0.0);
    double delta = (L->flags & MDO_DT_SOFTPLUS) ? mdo_softplus(v) : v;
    double decay = exp(delta * L->A[j]);
    double y = 0.0;
    for (int n = 0; n < N; ++n) {
        h[n] = decay * h[n] + delta * Bt[n] * u;
        y += Ct[n] * h[n];
    }
    y += (L->Dskip ? L->Dskip[d] : 0.0) * u;
    return y * mdo_silu(z);
}

/*
 * Context encode, packed sequences as in mdo_prefill.  x, z: (T, D); dt: (T, H); B, C: (T, N).
 * conv_init (n_seq, W-1, D), h_init (n_seq, D, N) may be NULL; so may conv_final, h_final.
 */
void mdo_ssd_prefill(const mdo_ssd_layer *L, int n_seq, const int32_t *cu_seqlens,
                     const double *x, const double *z, const double *dt,
                     const double *B, const double *C,
                     const double *conv_init, const double *h_init,
                     double *out, double *conv_final, double *h_final)
{
    const int D = L->d_inner, N = L->d_state, W = L->d_conv, H = D / L->headdim;
    for (int s = 0; s < n_seq; ++s) {
        const int t0 = cu_seqlens[s], t1 = cu_seqlens[s + 1];
#pragma omp parallel for schedule(static)
        for (int d = 0; d < D; ++d) {
            double win[16], h[256];
            for (int k = 0; k < W - 1; ++k)
                win[k] = conv_init ? conv_init[((size_t)s * (W - 1) + k) * D + d] : 0.0;
            for (int n = 0; n < N; ++n)
                h[n] = h_init ? h_init[((size_t)s * D + d) * N + n] : 0.0;
            for (int t = t0; t < t1; ++t)
                out[(size_t)t * D + d] = ssd_channel_token(L, d, win, h, x[(size_t)t * D + d], z[(size_t)t * D + d],
                                                           dt[(size_t)t * H + d / L->headdim], B + (size_t)t * N, C + (size_t)t * N);
            if (conv_final)
                for (int k = 0; k < W - 1; ++k) conv_final[((size_t)s * (W - 1) + k) * D + d] = win[k];
            if (h_final)
                for (int n = 0; n < N; ++n) h_final[((size_t)s * D + d) * N + n] = h[n];
        }
    }
}

/*
 * Tree drafting for one sequence, every node rebuilt along its root-to-node path from the committed state, as in
 * mdo_tree.  x, z: (M, D); dt: (M, H); B, C: (M, N).  Returns 0, or -1 if a parent index is not an earlier node.
 */
int mdo_ssd_tree(const mdo_ssd_layer *L, int M, const int32_t *parent,
                 const double *x, const double *z, const double *dt,
                 const double *B, const double *C,
                 const double *conv0, const double *h0,
                 double *out, double *conv_nodes, double *h_nodes)
{
    const int D = L->d_inner, N = L->d_state, W = L->d_conv, H = D / L->headdim;
    for (int v = 0; v < M; ++v)
        if (parent[v] >= v || parent[v] < -1) return -1;
    int *path = (int *)malloc(sizeof(int) * (size_t)(M > 0 ? M : 1));
    for (int v = 0; v < M; ++v) {
        int len = 0;
        for (int a = v; a >= 0; a = parent[a]) path[len++] = a;
#pragma omp parallel for schedule(static)
        for (int d = 0; d < D; ++d) {
            double win[16], h[256], o = 0.0;
            for (int k = 0; k < W - 1; ++k) win[k] = conv0 ? conv0[(size_t)k * D + d] : 0.0;
            for (int n = 0; n < N; ++n) h[n] = h0 ? h0[(size_t)d * N + n] : 0.0;
            for (int jn = len - 1; jn >= 0; --jn) {
                const size_t a = (size_t)path[jn];
                o = ssd_channel_token(L, d, win, h, x[a * D + d], z[a * D + d], dt[a * H + d / L->headdim], B + a * N, C + a * N);
            }
            out[(size_t)v * D + d] = o;
            if (conv_nodes)
                for (int k = 0; k < W - 1; ++k) conv_nodes[((size_t)v * (W - 1) + k) * D + d] = win[k];
            if (h_nodes)
                for (int n = 0; n < N; ++n) h_nodes[((size_t)v * D + d) * N + n] = h[n];
        }
    }
    free(path);
    return 0;
}
