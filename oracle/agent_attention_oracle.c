/*
 * Agent Attention forward pass: plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, dense, obviously-correct statement of
 * what the method computes, written from the paper's equations.  It shares no code,
 * header, table or helper with the CUDA library and must never be called from a product
 * path; only tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Everything is double precision.  Nothing is blocked, fused, split or padded: every
 * softmax row is materialised in full and normalised by its plain definition.
 *
 * Layouts (dense, last index fastest), per slab = one (batch, head) pair:
 *   Q, K, V : [N][d]   token t = y*W + x on an H x W grid (row-major, App. B reshape)
 *   A       : [n][d]   agent a = ay*pw + ax
 *   B1      : [n][N]   per head, shared over the batch          (Eq. 5)
 *   B2      : [N][n]   per head, shared over the batch          (Eq. 5)
 *   Wd      : [d][3][3] per head, one 3x3 filter per channel    (Eq. 6, k = 3 in Eq. 7)
 *
 * Parity pins live in tests/test_oracle_pins.py.  Unpinned: nothing in this file; the
 * paper's trained-model numbers (accuracy, FID) are "parity unpinned" and not attempted.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------------------------
 * Agent tokens by pooling, A = Pooling(Q)  (Sec. 4.2, text under Eq. 6).
 * Average pooling to a ph x pw grid.  Window of pooled cell (ay, ax): rows
 * floor(ay*H/ph) .. ceil((ay+1)*H/ph)-1 and columns likewise; when ph divides H this is
 * plain (H/ph) x (W/pw) block averaging.
 * ------------------------------------------------------------------------------- */
void aa_oracle_pool(const double* Q, int H, int W, int d, int ph, int pw, double* A)
{
    for (int ay = 0; ay < ph; ++ay) {
        int y0 = (ay * H) / ph;
        int y1 = ((ay + 1) * H + ph - 1) / ph;
        for (int ax = 0; ax < pw; ++ax) {
            int x0 = (ax * W) / pw;
            int x1 = ((ax + 1) * W + pw - 1) / pw;
            double* a = A + (size_t)(ay * pw + ax) * d;
            for (int c = 0; c < d; ++c) a[c] = 0.0;
            for (int y = y0; y < y1; ++y)
                for (int x = x0; x < x1; ++x) {
                    const double* q = Q + (size_t)(y * W + x) * d;
                    for (int c = 0; c < d; ++c) a[c] += q[c];
                }
            double cnt = (double)(y1 - y0) * (double)(x1 - x0);
            for (int c = 0; c < d; ++c) a[c] /= cnt;
        }
    }
}

/* ---------------------------------------------------------------------------------
 * Softmax attention, Eq. 1 with Sim(q,k) = exp(q.k * scale) (Sec. 3.2), with the
 * additive bias of Eq. 5 inside the exponent (the bias itself is not scaled):
 *   out[i,:] = sum_j  exp(s_ij) / (sum_j' exp(s_ij'))  *  Vm[j,:],
 *   s_ij = scale * <Qm[i,:], Km[j,:]> + bias[i,j].
 * Qm [rows][d], Km [cols][d], Vm [cols][dv], bias [rows][cols] or NULL, out [rows][dv].
 * If probs != NULL the row-stochastic matrix [rows][cols] is written there too.
 * Both stages of Eq. 3 are calls of this one routine.
 * ------------------------------------------------------------------------------- */
void aa_oracle_softmax_attention(const double* Qm, const double* Km, const double* Vm,
                                 const double* bias, int rows, int cols, int d, int dv,
                                 double scale, double* out, double* probs)
{
    double* s = (double*)malloc(sizeof(double) * (size_t)cols);
    for (int i = 0; i < rows; ++i) {
        const double* q = Qm + (size_t)i * d;
        double mx = -INFINITY;
        for (int j = 0; j < cols; ++j) {
            const double* k = Km + (size_t)j * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += q[c] * k[c];
            double v = dot * scale;
            if (bias) v += bias[(size_t)i * cols + j];
            s[j] = v;
            if (v > mx) mx = v;
        }
        double den = 0.0;
        for (int j = 0; j < cols; ++j) { s[j] = exp(s[j] - mx); den += s[j]; }
        for (int j = 0; j < cols; ++j) s[j] /= den;
        if (probs) memcpy(probs + (size_t)i * cols, s, sizeof(double) * (size_t)cols);
        double* o = out + (size_t)i * dv;
        for (int c = 0; c < dv; ++c) o[c] = 0.0;
        for (int j = 0; j < cols; ++j) {
            const double* v = Vm + (size_t)j * dv;
            double p = s[j];
            for (int c = 0; c < dv; ++c) o[c] += p * v[c];
        }
    }
    free(s);
}

/* ---------------------------------------------------------------------------------
 * Diversity restoration term of Eq. 6: O += DWC(V), a depthwise 3x3 convolution over the
 * token grid, stride 1, zero padding 1, cross-correlation indexing (no filter flip), no
 * additive conv bias:
 *   O[y,x,c] += sum_{u,v in 0..2} Wd[c][u][v] * V[y+u-1, x+v-1, c]   (terms outside the grid dropped)
 * ------------------------------------------------------------------------------- */
void aa_oracle_dwc_add(const double* V, const double* Wd, int H, int W, int d, double* O)
{
    for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x) {
            double* o = O + (size_t)(y * W + x) * d;
            for (int u = 0; u < 3; ++u) {
                int yy = y + u - 1;
                if (yy < 0 || yy >= H) continue;
                for (int v = 0; v < 3; ++v) {
                    int xx = x + v - 1;
                    if (xx < 0 || xx >= W) continue;
                    const double* vin = V + (size_t)(yy * W + xx) * d;
                    for (int c = 0; c < d; ++c) o[c] += Wd[(size_t)c * 9 + u * 3 + v] * vin[c];
                }
            }
        }
}

/* ---------------------------------------------------------------------------------
 * The module of Eq. 6,  O = s(Q A^T + B2) s(A K^T + B1) V + DWC(V),  evaluated as the two
 * Softmax attentions of Eq. 3 (agent aggregation, then agent broadcast).
 *
 *   Q, K, V [B][heads][N][d];  A_in [B][heads][n][d] or NULL (then A = Pooling(Q) with a
 *   ph x pw agent grid, n = ph*pw);  b1 [heads][n][N] / b2 [heads][N][n] or NULL;
 *   wd [heads][d][3][3] or NULL;  O [B][heads][N][d].
 *   A_out, VA_out: optional [B][heads][n][d] copies of the agents and agent features.
 *   threads: slabs are independent and are spread over this many OpenMP threads.
 * Returns the number of threads actually used, or -1 on bad arguments.
 * ------------------------------------------------------------------------------- */
int aa_oracle_forward(const double* Q, const double* K, const double* V, const double* A_in,
                      int B, int heads, int H, int W, int d, int n, int ph, int pw,
                      const double* b1, const double* b2, const double* wd,
                      double scale1, double scale2,
                      double* O, double* A_out, double* VA_out, int threads)
{
    if (!Q || !K || !V || !O || B <= 0 || heads <= 0 || H <= 0 || W <= 0 || d <= 0 || n <= 0)
        return -1;
    if (!A_in && (ph <= 0 || pw <= 0 || ph * pw != n || ph > H || pw > W)) return -1;
    const int N = H * W;
    const int slabs = B * heads;
    int used = 1;
    if (threads < 1) threads = 1;
#ifdef _OPENMP
    if (threads > slabs) threads = slabs;
    used = threads;
    #pragma omp parallel for num_threads(threads) schedule(dynamic, 1)
#endif
    for (int s = 0; s < slabs; ++s) {
        const int head = s % heads;
        const size_t off = (size_t)s * N * d;
        const double* q = Q + off;
        const double* k = K + off;
        const double* v = V + off;
        double* o = O + off;
        double* a  = (double*)malloc(sizeof(double) * (size_t)n * d);
        double* va = (double*)malloc(sizeof(double) * (size_t)n * d);
        if (A_in) memcpy(a, A_in + (size_t)s * n * d, sizeof(double) * (size_t)n * d);
        else      aa_oracle_pool(q, H, W, d, ph, pw, a);
        /* agent aggregation  V_A = Attn^S(A, K, V)  with B1 */
        aa_oracle_softmax_attention(a, k, v, b1 ? b1 + (size_t)head * n * N : NULL,
                                    n, N, d, d, scale1, va, NULL);
        /* agent broadcast  O = Attn^S(Q, A, V_A)  with B2 */
        aa_oracle_softmax_attention(q, a, va, b2 ? b2 + (size_t)head * N * n : NULL,
                                    N, n, d, d, scale2, o, NULL);
        if (wd) aa_oracle_dwc_add(v, wd + (size_t)head * d * 9, H, W, d, o);
        if (A_out)  memcpy(A_out  + (size_t)s * n * d, a,  sizeof(double) * (size_t)n * d);
        if (VA_out) memcpy(VA_out + (size_t)s * n * d, va, sizeof(double) * (size_t)n * d);
        free(a);
        free(va);
    }
    return used;
}

/* ---------------------------------------------------------------------------------
 * Generalized-linear-attention form, Eq. 4 (with the biases of Eq. 5): for one slab form
 * the explicit N x N matrix  M = s(Q A^T + B2) . s(A K^T + B1)  and  O = M V.
 * Tiny inputs only (O(N^2) memory).  M [N][N], O [N][d].
 * ------------------------------------------------------------------------------- */
void aa_oracle_explicit(const double* Q, const double* A, const double* K, const double* V,
                        const double* b1, const double* b2, int N, int n, int d,
                        double scale1, double scale2, double* M, double* O)
{
    double* phiq = (double*)malloc(sizeof(double) * (size_t)N * n);   /* s(Q A^T + B2) */
    double* phik = (double*)malloc(sizeof(double) * (size_t)n * N);   /* s(A K^T + B1) */
    double* dump = (double*)malloc(sizeof(double) * (size_t)(N > n ? N : n) * d);
    aa_oracle_softmax_attention(Q, A, A, b2, N, n, d, d, scale2, dump, phiq);
    aa_oracle_softmax_attention(A, K, K, b1, n, N, d, d, scale1, dump, phik);
    for (int i = 0; i < N; ++i)
        for (int j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int a = 0; a < n; ++a) acc += phiq[(size_t)i * n + a] * phik[(size_t)a * N + j];
            M[(size_t)i * N + j] = acc;
        }
    for (int i = 0; i < N; ++i)
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int j = 0; j < N; ++j) acc += M[(size_t)i * N + j] * V[(size_t)j * d + c];
            O[(size_t)i * d + c] = acc;
        }
    free(phiq); free(phik); free(dump);
}

/* ---------------------------------------------------------------------------------
 * Composition of an agent bias from its three components (App. B):
 *   B = (B'_c + B'_r + B'_b).reshape(n, N),  N = h*w,
 * with the column bias col [n][w] repeated over the h rows, the row bias row [n][h] repeated over
 * the w columns, and the block bias blk [n][h0][w0] resized to h x w.  The paper says "repeating
 * or interpolating"; the reading taken here resizes the block bias by bilinear interpolation with
 * half-pixel centres and edge clamping (source coordinate max(0, (y + 0.5) * h0 / h - 0.5), and
 * likewise in x), which is the identity when h0 = h and w0 = w.  Any component may be NULL (zero).
 * transpose == 0 writes [n][N] (the layout of B1); transpose != 0 writes [N][n] (that of B2).
 * ------------------------------------------------------------------------------- */
void aa_oracle_compose_bias(const double* col, const double* row, const double* blk,
                            int n, int h, int w, int h0, int w0, int transpose, double* out)
{
    const int N = h * w;
    for (int a = 0; a < n; ++a)
        for (int y = 0; y < h; ++y)
            for (int x = 0; x < w; ++x) {
                double v = 0.0;
                if (col) v += col[(size_t)a * w + x];
                if (row) v += row[(size_t)a * h + y];
                if (blk) {
                    double sy = ((double)y + 0.5) * (double)h0 / (double)h - 0.5;
                    double sx = ((double)x + 0.5) * (double)w0 / (double)w - 0.5;
                    if (sy < 0.0) sy = 0.0;
                    if (sx < 0.0) sx = 0.0;
                    int y0 = (int)floor(sy), x0 = (int)floor(sx);
                    if (y0 > h0 - 1) y0 = h0 - 1;
                    if (x0 > w0 - 1) x0 = w0 - 1;
                    int y1 = y0 < h0 - 1 ? y0 + 1 : y0;
                    int x1 = x0 < w0 - 1 ? x0 + 1 : x0;
                    double ly = sy - (double)y0, lx = sx - (double)x0;
                    if (ly > 1.0) ly = 1.0;
                    if (lx > 1.0) lx = 1.0;
                    const double* b = blk + (size_t)a * h0 * w0;
                    v += (1.0 - ly) * ((1.0 - lx) * b[y0 * w0 + x0] + lx * b[y0 * w0 + x1])
                       +        ly  * ((1.0 - lx) * b[y1 * w0 + x0] + lx * b[y1 * w0 + x1]);
                }
                const int t = y * w + x;
                if (transpose) out[(size_t)t * n + a] = v;
                else           out[(size_t)a * N + t] = v;
            }
}

/* ---------------------------------------------------------------------------------
 * Gradients of Eq. 6 (pooled agents).  The paper prints no backward formulas; these are the
 * chain rule applied to the steps of aa_oracle_forward, written out densely per slab:
 *   with P2 = s(scale2 Q A^T + B2), P1 = s(scale1 A K^T + B1), V_A = P1 V, O = P2 V_A + DWC(V)
 *   dV_A = P2^T dO            dP2 = dO V_A^T      dS2 = P2 o (dP2 - rowsum(P2 o dP2))
 *   dQ  = scale2 dS2 A        dA  = scale2 dS2^T Q + scale1 dS1 K
 *   dP1 = dV_A V^T            dS1 = P1 o (dP1 - rowsum(P1 o dP1))
 *   dK  = scale1 dS1^T A      dV  = P1^T dV_A + DWC^T(dO)
 *   dB1 = sum over batch dS1  dB2 = sum over batch dS2   dWd[c][u][v] = sum dO[y,x,c] V[y+u-1,x+v-1,c]
 *   dQ += Pooling^T(dA): every token of agent a's window receives dA[a] / (window size).
 * dO, dQ, dK, dV [B][heads][N][d]; dB1 [heads][n][N], dB2 [heads][N][n], dWd [heads][d][3][3]
 * (each may be NULL when the forward had no such input; they are overwritten, not accumulated into).
 * Serial over slabs (the bias and filter gradients sum over the batch).  Returns 0, or -1 on bad arguments.
 * ------------------------------------------------------------------------------- */
int aa_oracle_backward(const double* Q, const double* K, const double* V, const double* dO,
                       int B, int heads, int H, int W, int d, int n, int ph, int pw,
                       const double* b1, const double* b2, const double* wd,
                       double scale1, double scale2,
                       double* dQ, double* dK, double* dV, double* dB1, double* dB2, double* dWd)
{
    if (!Q || !K || !V || !dO || !dQ || !dK || !dV || B <= 0 || heads <= 0 || H <= 0 || W <= 0 || d <= 0)
        return -1;
    if (ph <= 0 || pw <= 0 || ph * pw != n || ph > H || pw > W) return -1;
    const int N = H * W;
    const size_t nN = (size_t)n * N, nd = (size_t)n * d, Nd = (size_t)N * d;
    if (dB1) memset(dB1, 0, sizeof(double) * heads * nN);
    if (dB2) memset(dB2, 0, sizeof(double) * heads * nN);
    if (dWd) memset(dWd, 0, sizeof(double) * (size_t)heads * d * 9);
    double* a = (double*)malloc(sizeof(double) * nd);
    double* v_a = (double*)malloc(sizeof(double) * nd);
    double* dva = (double*)malloc(sizeof(double) * nd);
    double* da = (double*)malloc(sizeof(double) * nd);
    double* p1 = (double*)malloc(sizeof(double) * nN);      /* [n][N] */
    double* p2 = (double*)malloc(sizeof(double) * nN);      /* [N][n] */
    double* ds = (double*)malloc(sizeof(double) * nN);
    double* oat = (double*)malloc(sizeof(double) * Nd);
    for (int s = 0; s < B * heads; ++s) {
        const int head = s % heads;
        const double *q = Q + s * Nd, *k = K + s * Nd, *v = V + s * Nd, *go = dO + s * Nd;
        double *gq = dQ + s * Nd, *gk = dK + s * Nd, *gv = dV + s * Nd;
        aa_oracle_pool(q, H, W, d, ph, pw, a);
        aa_oracle_softmax_attention(a, k, v, b1 ? b1 + head * nN : NULL, n, N, d, d, scale1, v_a, p1);
        aa_oracle_softmax_attention(q, a, v_a, b2 ? b2 + head * nN : NULL, N, n, d, d, scale2, oat, p2);
        /* broadcast stage */
        for (int r = 0; r < n; ++r)
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int i = 0; i < N; ++i) acc += p2[(size_t)i * n + r] * go[(size_t)i * d + c];
                dva[(size_t)r * d + c] = acc;
            }
        for (int i = 0; i < N; ++i) {
            double dot = 0.0;
            for (int r = 0; r < n; ++r) {
                double dp = 0.0;
                for (int c = 0; c < d; ++c) dp += go[(size_t)i * d + c] * v_a[(size_t)r * d + c];
                ds[(size_t)i * n + r] = dp;
                dot += p2[(size_t)i * n + r] * dp;
            }
            for (int r = 0; r < n; ++r) {
                const double g = p2[(size_t)i * n + r] * (ds[(size_t)i * n + r] - dot);
                ds[(size_t)i * n + r] = g;
                if (dB2) dB2[head * nN + (size_t)i * n + r] += g;
            }
        }
        for (int i = 0; i < N; ++i)
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int r = 0; r < n; ++r) acc += ds[(size_t)i * n + r] * a[(size_t)r * d + c];
                gq[(size_t)i * d + c] = scale2 * acc;
            }
        for (int r = 0; r < n; ++r)
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int i = 0; i < N; ++i) acc += ds[(size_t)i * n + r] * q[(size_t)i * d + c];
                da[(size_t)r * d + c] = scale2 * acc;
            }
        /* aggregation stage */
        for (int r = 0; r < n; ++r) {
            double dot = 0.0;
            for (int j = 0; j < N; ++j) {
                double dp = 0.0;
                for (int c = 0; c < d; ++c) dp += dva[(size_t)r * d + c] * v[(size_t)j * d + c];
                ds[(size_t)r * N + j] = dp;
                dot += p1[(size_t)r * N + j] * dp;
            }
            for (int j = 0; j < N; ++j) {
                const double g = p1[(size_t)r * N + j] * (ds[(size_t)r * N + j] - dot);
                ds[(size_t)r * N + j] = g;
                if (dB1) dB1[head * nN + (size_t)r * N + j] += g;
            }
        }
        for (int j = 0; j < N; ++j)
            for (int c = 0; c < d; ++c) {
                double gk_acc = 0.0, gv_acc = 0.0;
                for (int r = 0; r < n; ++r) {
                    gk_acc += ds[(size_t)r * N + j] * a[(size_t)r * d + c];
                    gv_acc += p1[(size_t)r * N + j] * dva[(size_t)r * d + c];
                }
                gk[(size_t)j * d + c] = scale1 * gk_acc;
                gv[(size_t)j * d + c] = gv_acc;
            }
        for (int r = 0; r < n; ++r)
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int j = 0; j < N; ++j) acc += ds[(size_t)r * N + j] * k[(size_t)j * d + c];
                da[(size_t)r * d + c] += scale1 * acc;
            }
        /* depthwise term */
        if (wd) {
            const double* w = wd + (size_t)9 * d * head;          /* this head's [d][3][3] filter */
            for (int y = 0; y < H; ++y)
                for (int x = 0; x < W; ++x)
                    for (int u = 0; u < 3; ++u)
                        for (int t = 0; t < 3; ++t) {
                            const int yy = y + u - 1, xx = x + t - 1;
                            if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
                            for (int c = 0; c < d; ++c) {
                                const double g = go[((size_t)y * W + x) * d + c];
                                gv[((size_t)yy * W + xx) * d + c] += w[(size_t)c * 9 + u * 3 + t] * g;
                                if (dWd) dWd[((size_t)head * d + c) * 9 + u * 3 + t] += g * v[((size_t)yy * W + xx) * d + c];
                            }
                        }
        }
        /* pooling: the window of agent (ay, ax) as in aa_oracle_pool */
        for (int ay = 0; ay < ph; ++ay)
            for (int ax = 0; ax < pw; ++ax) {
                const int y0 = (ay * H) / ph, y1 = ((ay + 1) * H + ph - 1) / ph;
                const int x0 = (ax * W) / pw, x1 = ((ax + 1) * W + pw - 1) / pw;
                const double inv = 1.0 / (double)((y1 - y0) * (x1 - x0));
                for (int y = y0; y < y1; ++y)
                    for (int x = x0; x < x1; ++x)
                        for (int c = 0; c < d; ++c)
                            gq[((size_t)y * W + x) * d + c] += da[(size_t)(ay * pw + ax) * d + c] * inv;
            }
    }
    free(a); free(v_a); free(dva); free(da); free(p1); free(p2); free(ds); free(oat);
    return 0;
}

/* ---------------------------------------------------------------------------------
 * Module complexity, Eq. 7, in multiply-accumulates for N tokens, C channels (all heads),
 * n agents, DWC kernel size k:
 *   parts = { 4NC^2 (projections), NC (agents), 2nNC (aggregation: logits and weighted
 *   sum), 2NnC (broadcast), k^2 NC (DWC) };  returns their sum.
 * ------------------------------------------------------------------------------- */
long long aa_oracle_macs(long long N, long long C, long long n, long long k, long long* parts)
{
    long long p[5];
    p[0] = 4 * N * C * C;
    p[1] = N * C;
    p[2] = 2 * n * N * C;
    p[3] = 2 * N * n * C;
    p[4] = k * k * N * C;
    if (parts) memcpy(parts, p, sizeof(p));
    return p[0] + p[1] + p[2] + p[3] + p[4];
}

int aa_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
