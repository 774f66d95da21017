/*
 * CPU oracle for the composed attention variant softmax(mask(alibi(rope(Q,K)))) @ V
 * and its gradients.  TEST INFRASTRUCTURE ONLY: the product (the CUDA library) never
 * links, imports or calls this file; only tests, the smoke check and the bench's
 * cpu_baseline / reference arm do.
 *
 * The method is exact attention (the online-softmax recurrence of Section 2 is exact),
 * so this file is the plain definition written out in fp64, with no tiling, no fusion
 * and no reordering: rotate every row, form every score, mask, take a max-shifted
 * softmax, multiply by V.  Tensors are [B, H, S, D] contiguous doubles.
 *
 * Readings where the paper is silent (each is pinned by a CPU test):
 *  - RoPE (Sections 2 and 4.1): NeoX half-swap pairing (i, i+R/2), frequency
 *    theta^(-2i/R), position p0 + row index for Q and K alike; dims >= R pass through.
 *  - GQA: query head h reads kv head h / g (consecutive query heads share one).
 *  - Sliding window with causal: keep 0 <= i-j <= W (W+1 keys); without causal |i-j| <= W.
 *  - ALiBi: slope_h * (j - i) added after the softmax scale is applied.
 *  - Saved statistic (Section 4.4): L_i = m_i + ln(l_i), natural log.
 *  - Block-sparse attention (Section 4.3): the active-block lists only restrict the kept set: a pair
 *    (i, j) is kept iff the element mask keeps it AND block (i / bs, j / bs) is active.  Here the lists
 *    arrive as a dense nb x nb byte matrix (nb = ceil(S / bs)); a row with no kept pair gives O = 0,
 *    L = -inf and zero gradients.
 *  - Backward (Section 4.4, FlashAttention-2 algebra) with the chain rule through the
 *    rotation: gradients w.r.t. rotated rows are rotated back by the transpose.
 *  - additive_bias (Section 3.1 names the combinator only): a dense tensor bias[bb, hh, i, j] added to the
 *    scaled score after the softmax scale, like the ALiBi term; its batch and head extents are 1
 *    (broadcast) or B / Hq.  A bias of -inf drops the pair like a mask.  The bias gets no gradient.
 *  - relu_attention (Section 3.1 names the combinator only): the normaliser softmax is replaced by
 *    P_ij = max(s_ij, 0) / n_i over the kept pairs, n_i = number of kept pairs of row i (the sequence
 *    length when nothing is masked, which is the published ReLU-attention scaling); O_i = sum_j P_ij v_j.
 *    There is no row statistic L for it.  Gradient: dS_ij = [s_ij > 0] <dO_i, v_j> / n_i.
 *  - full (Section 3.1): no mask, i.e. causal = 0 and window < 0.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* Rotate one row x[0..D) at position p into y.  sign=+1 forward, -1 transpose/inverse. */
static void rope_row(const double* x, double* y, int D, int R, double theta, long p, int sign)
{
    int half = R / 2;
    for (int d = R; d < D; ++d) y[d] = x[d];
    for (int i = 0; i < half; ++i) {
        double freq = pow(theta, -2.0 * (double)i / (double)R);
        double ang = (double)p * freq;
        double c = cos(ang), s = sin(ang) * (double)sign;
        double a = x[i], b = x[i + half];
        y[i] = a * c - b * s;
        y[i + half] = b * c + a * s;
    }
}

/* Section 4.1: RoPE applied to every row of x [B,H,S,D]; y may not alias x. */
void af_oracle_rope(const double* x, double* y, int B, int H, int S, int D,
                    double theta, int R, int p0, int inverse)
{
    long rows = (long)B * H * S;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        long s = r % S;
        rope_row(x + r * D, y + r * D, D, R, theta, (long)p0 + s, inverse ? -1 : 1);
    }
}

/* Section 4.3: active-block matrix (NULL = every block active). */
typedef struct { const unsigned char* active; int bs, nb; } block_mask;

static int kept(int i, int j, int causal, int window, const block_mask* bm)
{
    if (bm && bm->active && !bm->active[(long)(i / bm->bs) * bm->nb + j / bm->bs]) return 0;
    if (causal && j > i) return 0;
    if (window >= 0) {
        int d = i - j;
        if (d < 0) d = -d;
        if (d > window) return 0;
    }
    return 1;
}

/*
 * Forward.  rows == NULL: all S query rows, o is [B,Hq,S,D], lse [B,Hq,S].
 * Otherwise only the n_rows listed query rows (same list for every head):
 * o is [B,Hq,n_rows,D], lse [B,Hq,n_rows].  slopes: Hq doubles or NULL.
 */
/* bias[bb, hh, i, j], bb = b or 0, hh = h or 0 (extents 1 broadcast); NULL = none */
static double bias_at(const double* bias, int bias_B, int bias_H, int S, int b, int h, int i, int j)
{
    if (!bias) return 0.0;
    long bb = bias_B == 1 ? 0 : b, hh = bias_H == 1 ? 0 : h;
    return bias[((bb * bias_H + hh) * S + i) * (long)S + j];
}

/* Section 3.1, all combinators: relu != 0 selects the relu_attention normaliser (lse is then not written). */
void af_oracle_fwd_variant(const double* q, const double* k, const double* v,
                           int B, int Hq, int Hkv, int S, int D,
                           double theta, int R, int p0, int causal, int window,
                           const double* slopes, double scale,
                           const unsigned char* blocks, int block_size,
                           const double* bias, int bias_B, int bias_H, int relu,
                           const int* rows, int n_rows, double* o, double* lse)
{
    block_mask bmv = { blocks, block_size, block_size > 0 ? (S + block_size - 1) / block_size : 0 };
    const block_mask* bm = blocks ? &bmv : NULL;
    int g = Hq / Hkv;
    int nr = rows ? n_rows : S;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * Hq; ++bh) {
        int b = bh / Hq, h = bh % Hq, hk = h / g;
        const double* kh = k + ((long)b * Hkv + hk) * S * D;
        const double* vh = v + ((long)b * Hkv + hk) * S * D;
        const double* qh = q + ((long)b * Hq + h) * S * D;
        double* kr = (double*)malloc(sizeof(double) * S * D);
        double* qr = (double*)malloc(sizeof(double) * D);
        double* sc = (double*)malloc(sizeof(double) * S);
        for (int j = 0; j < S; ++j) rope_row(kh + (long)j * D, kr + (long)j * D, D, R, theta, (long)p0 + j, 1);
        for (int t = 0; t < nr; ++t) {
            int i = rows ? rows[t] : t;
            rope_row(qh + (long)i * D, qr, D, R, theta, (long)p0 + i, 1);
            double m = -INFINITY;
            for (int j = 0; j < S; ++j) {
                if (!kept(i, j, causal, window, bm)) { sc[j] = -INFINITY; continue; }
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += qr[d] * kr[(long)j * D + d];
                double s = scale * dot;
                if (slopes) s += slopes[h] * (double)(j - i);
                s += bias_at(bias, bias_B, bias_H, S, b, h, i, j);
                sc[j] = s;
                if (s > m) m = s;
            }
            double* orow = o + (((long)b * Hq + h) * nr + t) * D;
            for (int d = 0; d < D; ++d) orow[d] = 0.0;
            double l = 0.0;
            if (relu) {
                /* relu_attention: P_ij = max(s_ij, 0) / n_i over the kept pairs */
                long n_kept = 0;
                for (int j = 0; j < S; ++j) if (sc[j] != -INFINITY) ++n_kept;
                if (n_kept == 0) continue;
                for (int j = 0; j < S; ++j) {
                    if (sc[j] == -INFINITY || sc[j] <= 0.0) continue;
                    double p = sc[j] / (double)n_kept;
                    for (int d = 0; d < D; ++d) orow[d] += p * vh[(long)j * D + d];
                }
                continue;
            }
            if (m == -INFINITY) { lse[((long)b * Hq + h) * nr + t] = -INFINITY; continue; }
            for (int j = 0; j < S; ++j) {
                if (sc[j] == -INFINITY) continue;
                double p = exp(sc[j] - m);
                l += p;
                for (int d = 0; d < D; ++d) orow[d] += p * vh[(long)j * D + d];
            }
            for (int d = 0; d < D; ++d) orow[d] /= l;
            lse[((long)b * Hq + h) * nr + t] = m + log(l);
        }
        free(kr); free(qr); free(sc);
    }
}

void af_oracle_fwd_blocks(const double* q, const double* k, const double* v,
                          int B, int Hq, int Hkv, int S, int D,
                          double theta, int R, int p0, int causal, int window,
                          const double* slopes, double scale,
                          const unsigned char* blocks, int block_size,
                          const int* rows, int n_rows, double* o, double* lse)
{
    af_oracle_fwd_variant(q, k, v, B, Hq, Hkv, S, D, theta, R, p0, causal, window, slopes, scale, blocks, block_size,
                          NULL, 1, 1, 0, rows, n_rows, o, lse);
}

void af_oracle_fwd(const double* q, const double* k, const double* v,
                   int B, int Hq, int Hkv, int S, int D,
                   double theta, int R, int p0, int causal, int window,
                   const double* slopes, double scale,
                   const int* rows, int n_rows, double* o, double* lse)
{
    af_oracle_fwd_blocks(q, k, v, B, Hq, Hkv, S, D, theta, R, p0, causal, window, slopes, scale, NULL, 0,
                         rows, n_rows, o, lse);
}

/*
 * Backward, given upstream dO [B,Hq,S,D].  Recomputes P from the definition.
 * dq [B,Hq,S,D], dk, dv [B,Hkv,S,D]; dk and dv of a kv head sum over its g query heads.
 */
void af_oracle_bwd_variant(const double* q, const double* k, const double* v, const double* d_o,
                           int B, int Hq, int Hkv, int S, int D,
                           double theta, int R, int p0, int causal, int window,
                           const double* slopes, double scale,
                           const unsigned char* blocks, int block_size,
                           const double* bias, int bias_B, int bias_H, int relu,
                           double* dq, double* dk, double* dv)
{
    block_mask bmv = { blocks, block_size, block_size > 0 ? (S + block_size - 1) / block_size : 0 };
    const block_mask* bm = blocks ? &bmv : NULL;
    int g = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bk = 0; bk < B * Hkv; ++bk) {
        int b = bk / Hkv, hk = bk % Hkv;
        const double* kh = k + ((long)b * Hkv + hk) * S * D;
        const double* vh = v + ((long)b * Hkv + hk) * S * D;
        double* kr = (double*)malloc(sizeof(double) * S * D);
        double* dkr = (double*)calloc((size_t)S * D, sizeof(double)); /* grad w.r.t. rotated K */
        double* dvh = dv + ((long)b * Hkv + hk) * S * D;
        double* qr = (double*)malloc(sizeof(double) * D);
        double* dqr = (double*)malloc(sizeof(double) * D);
        double* orow = (double*)malloc(sizeof(double) * D);
        double* pr = (double*)malloc(sizeof(double) * S);
        memset(dvh, 0, sizeof(double) * S * D);
        for (int j = 0; j < S; ++j) rope_row(kh + (long)j * D, kr + (long)j * D, D, R, theta, (long)p0 + j, 1);
        for (int hh = 0; hh < g; ++hh) {
            int h = hk * g + hh;
            const double* qh = q + ((long)b * Hq + h) * S * D;
            const double* doh = d_o + ((long)b * Hq + h) * S * D;
            double* dqh = dq + ((long)b * Hq + h) * S * D;
            for (int i = 0; i < S; ++i) {
                rope_row(qh + (long)i * D, qr, D, R, theta, (long)p0 + i, 1);
                const double* doi = doh + (long)i * D;
                double m = -INFINITY;
                for (int j = 0; j < S; ++j) {
                    if (!kept(i, j, causal, window, bm)) { pr[j] = -INFINITY; continue; }
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += qr[d] * kr[(long)j * D + d];
                    double s = scale * dot;
                    if (slopes) s += slopes[h] * (double)(j - i);
                    s += bias_at(bias, bias_B, bias_H, S, b, h, i, j);
                    pr[j] = s;
                    if (s > m) m = s;
                }
                for (int d = 0; d < D; ++d) { dqr[d] = 0.0; orow[d] = 0.0; }
                if (m == -INFINITY) { for (int d = 0; d < D; ++d) dqh[(long)i * D + d] = 0.0; continue; }
                if (relu) {
                    /* relu_attention: P_ij = max(s_ij, 0) / n_i; dV_j += P_ij dO_i; dS_ij = [s_ij > 0] <dO_i, v_j> / n_i */
                    long n_kept = 0;
                    for (int j = 0; j < S; ++j) if (pr[j] != -INFINITY) ++n_kept;
                    for (int j = 0; j < S; ++j) {
                        if (pr[j] == -INFINITY || pr[j] <= 0.0) continue;
                        double p = pr[j] / (double)n_kept;
                        double dp = 0.0;
                        for (int d = 0; d < D; ++d) dp += doi[d] * vh[(long)j * D + d];
                        double ds = dp / (double)n_kept;
                        for (int d = 0; d < D; ++d) {
                            dvh[(long)j * D + d] += p * doi[d];
                            dqr[d] += scale * ds * kr[(long)j * D + d];
                            dkr[(long)j * D + d] += scale * ds * qr[d];
                        }
                    }
                    rope_row(dqr, dqh + (long)i * D, D, R, theta, (long)p0 + i, -1);
                    continue;
                }
                double l = 0.0;
                for (int j = 0; j < S; ++j) {
                    if (pr[j] == -INFINITY) { pr[j] = 0.0; continue; }
                    pr[j] = exp(pr[j] - m);
                    l += pr[j];
                }
                for (int j = 0; j < S; ++j) {
                    pr[j] /= l;
                    if (pr[j] != 0.0)
                        for (int d = 0; d < D; ++d) orow[d] += pr[j] * vh[(long)j * D + d];
                }
                double delta = 0.0;
                for (int d = 0; d < D; ++d) delta += doi[d] * orow[d];
                for (int j = 0; j < S; ++j) {
                    double p = pr[j];
                    if (p == 0.0) continue;
                    double dp = 0.0;
                    for (int d = 0; d < D; ++d) dp += doi[d] * vh[(long)j * D + d];
                    double ds = p * (dp - delta);
                    for (int d = 0; d < D; ++d) {
                        dvh[(long)j * D + d] += p * doi[d];
                        dqr[d] += scale * ds * kr[(long)j * D + d];
                        dkr[(long)j * D + d] += scale * ds * qr[d];
                    }
                }
                rope_row(dqr, dqh + (long)i * D, D, R, theta, (long)p0 + i, -1);
            }
        }
        double* dkh = dk + ((long)b * Hkv + hk) * S * D;
        for (int j = 0; j < S; ++j) rope_row(dkr + (long)j * D, dkh + (long)j * D, D, R, theta, (long)p0 + j, -1);
        free(kr); free(dkr); free(qr); free(dqr); free(orow); free(pr);
    }
}

void af_oracle_bwd_blocks(const double* q, const double* k, const double* v, const double* d_o,
                          int B, int Hq, int Hkv, int S, int D,
                          double theta, int R, int p0, int causal, int window,
                          const double* slopes, double scale,
                          const unsigned char* blocks, int block_size,
                          double* dq, double* dk, double* dv)
{
    af_oracle_bwd_variant(q, k, v, d_o, B, Hq, Hkv, S, D, theta, R, p0, causal, window, slopes, scale, blocks,
                          block_size, NULL, 1, 1, 0, dq, dk, dv);
}

void af_oracle_bwd(const double* q, const double* k, const double* v, const double* d_o,
                   int B, int Hq, int Hkv, int S, int D,
                   double theta, int R, int p0, int causal, int window,
                   const double* slopes, double scale,
                   double* dq, double* dk, double* dv)
{
    af_oracle_bwd_blocks(q, k, v, d_o, B, Hq, Hkv, S, D, theta, R, p0, causal, window, slopes, scale, NULL, 0,
                         dq, dk, dv);
}
