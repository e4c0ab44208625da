/*
 * fp64 CPU oracle for the learnable-token-eviction (LTE) sparse-attention layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what the
 * layer computes, written from the paper's Section 3.1 (Eq. 5, Eq. 6, Eq. 7 and
 * the "Inference implementation" paragraphs).  It shares no code with the CUDA
 * library and must never be called from the product path: only the tests, the
 * smoke check and the benchmark's cpu_baseline / reference arm may load it.
 *
 * Conventions (0-based positions; the paper is 1-based):
 *   W      sliding window = W keys including the query itself: i-W < j <= i
 *   R      retain budget (paper: b), cap on out-of-window KVs per head
 *   sink   first `sink` positions are always candidates (paper: s)
 *   half   floor(receptive field / 2) of the scorer CNN
 *   z      pre-sigmoid logit, r = sigmoid(z) the retention score
 *   zthr   logit of the keep threshold tau (0 for tau = 0.5); keep iff z > zthr
 * All tensors are contiguous, last index fastest: q,k,v,o [B,H,T,d];
 * z, lse [B,H,T]; idx [B,H,R] (ascending, unused = -1); cnt [B,H].
 *
 * Total order used wherever a budget forces a choice (paper: "keep those with
 * top-b scores", "evict the lowest-score entry if it scores higher"):
 *   sink positions first (by position), then z descending, then position
 *   ascending.  An equal-score newcomer never displaces an older entry.
 *
 * Parity pins (tests, -m "not gpu"): dense brute force from the set definition,
 * delta-weight closed forms, q=0 / v=const closed forms, streaming == one-shot
 * pool, central finite differences for every gradient.  The conv-stack channel
 * plan at the paper's 1.4B size is "parity unpinned" (the paper's parameter
 * share for that size cannot be reproduced from the text).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define NEG_INF (-INFINITY)

static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

/* ------------------------------------------------------------------------- */
/* Scorer, single grouped conv layer (Section 3.1.1, "LTE module"; the width-K
 * instance: one centred cross-correlation over concat(k, v), 2d -> 1 per head).
 *   z[b,h,j] = bias[h] + sum_{t<K} sum_{c<2d} w[h,t,c] * x[b,h,j+t-half,c],
 * x = [k ; v], x = 0 at negative positions (left zero padding), and no right
 * padding: z is undefined (-inf) for j > T-1-half.                           */
void oracle_scores(int B, int H, int T, int d, int K,
                   const double* k, const double* v,
                   const double* w, const double* bias, double* z)
{
    const int half = K / 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const double* kk = k + ((size_t)b * H + h) * T * d;
            const double* vv = v + ((size_t)b * H + h) * T * d;
            double* zz = z + ((size_t)b * H + h) * T;
            for (int j = 0; j < T; ++j) {
                if (j + half > T - 1) { zz[j] = NEG_INF; continue; }
                double acc = bias ? bias[h] : 0.0;
                for (int t = 0; t < K; ++t) {
                    int p = j + t - half;
                    if (p < 0) continue;
                    const double* wt = w + ((size_t)h * K + t) * 2 * d;
                    for (int c = 0; c < d; ++c) acc += wt[c] * kk[(size_t)p * d + c];
                    for (int c = 0; c < d; ++c) acc += wt[d + c] * vv[(size_t)p * d + c];
                }
                zz[j] = acc;
            }
        }
}

/* Scorer, the paper's stack (Appendix A): L dilated grouped conv layers (kernel
 * ks, dilation dil) each followed by Swish, channels c[0]=2d -> c[1] -> ... ->
 * c[L], then a per-head linear map to one logit.  Written in causal form: every
 * layer's input is zero at negative positions; layer l's output at time t reads
 * its input at t, t-dil, ..., t-(ks-1)*dil.  The logit of token j is the stack's
 * output at time j + half, half = L*(ks-1)*dil/2, which centres the receptive
 * field on j.  Weights: wl[l] is [H, c[l+1], ks, c[l]], bl[l] is [H, c[l+1]],
 * wout [H, c[L]], bout [H].  No dropout (inference semantics).               */
void oracle_scores_stack(int B, int H, int T, int d, int L, int ks, int dil,
                         const int* ch, /* L+1 entries, ch[0] = 2d */
                         const double* const* wl, const double* const* bl,
                         const double* wout, const double* bout,
                         const double* k, const double* v, double* z)
{
    const int half = L * (ks - 1) * dil / 2;
    int cmax = 0;
    for (int l = 0; l <= L; ++l) if (ch[l] > cmax) cmax = ch[l];
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const double* kk = k + ((size_t)b * H + h) * T * d;
            const double* vv = v + ((size_t)b * H + h) * T * d;
            double* zz = z + ((size_t)b * H + h) * T;
            double* cur = (double*)malloc(sizeof(double) * (size_t)T * cmax);
            double* nxt = (double*)malloc(sizeof(double) * (size_t)T * cmax);
            for (int t = 0; t < T; ++t) {
                for (int c = 0; c < d; ++c) cur[(size_t)t * cmax + c] = kk[(size_t)t * d + c];
                for (int c = 0; c < d; ++c) cur[(size_t)t * cmax + d + c] = vv[(size_t)t * d + c];
            }
            for (int l = 0; l < L; ++l) {
                const int cin = ch[l], cout = ch[l + 1];
                const double* Wl = wl[l] + (size_t)h * cout * ks * cin;
                const double* Bl = bl[l] ? bl[l] + (size_t)h * cout : NULL;
                for (int t = 0; t < T; ++t)
                    for (int o = 0; o < cout; ++o) {
                        double acc = Bl ? Bl[o] : 0.0;
                        for (int tau = 0; tau < ks; ++tau) {
                            int p = t - (ks - 1 - tau) * dil;
                            if (p < 0) continue;
                            const double* wv = Wl + ((size_t)o * ks + tau) * cin;
                            for (int c = 0; c < cin; ++c) acc += wv[c] * cur[(size_t)p * cmax + c];
                        }
                        nxt[(size_t)t * cmax + o] = acc * sigmoid(acc); /* Swish */
                    }
                double* tmp = cur; cur = nxt; nxt = tmp;
            }
            for (int j = 0; j < T; ++j) {
                int t = j + half;
                if (t > T - 1) { zz[j] = NEG_INF; continue; }
                double acc = bout ? bout[h] : 0.0;
                for (int c = 0; c < ch[L]; ++c) acc += wout[(size_t)h * ch[L] + c] * cur[(size_t)t * cmax + c];
                zz[j] = acc;
            }
            free(cur); free(nxt);
        }
}

/* ------------------------------------------------------------------------- */
/* Backward of the stack above (Section 3.1.1's scorer under the gradient of
 * Section 3.1.2): given dL/dz [B,H,T] (zero where the logit is undefined), the
 * gradients of every layer's weights and biases (summed over the batch), of the
 * output map, and of the inputs k, v [B,H,T,d].  Plain chain rule, layer by
 * layer: Swish'(y) = s + y s (1 - s) with s = sigmoid(y); a layer's input at
 * negative time is the constant zero and receives nothing.                   */
void oracle_scores_stack_bwd(int B, int H, int T, int d, int L, int ks, int dil,
                             const int* ch, const double* const* wl, const double* const* bl,
                             const double* wout, const double* bout,
                             const double* k, const double* v, const double* dz,
                             double* const* dwl, double* const* dbl, double* dwout, double* dbout,
                             double* dk, double* dv)
{
    const int half = L * (ks - 1) * dil / 2;
    int cmax = 0;
    for (int l = 0; l <= L; ++l) if (ch[l] > cmax) cmax = ch[l];
    (void)bout;
    for (int l = 0; l < L; ++l) {
        memset(dwl[l], 0, sizeof(double) * (size_t)H * ch[l + 1] * ks * ch[l]);
        memset(dbl[l], 0, sizeof(double) * (size_t)H * ch[l + 1]);
    }
    memset(dwout, 0, sizeof(double) * (size_t)H * ch[L]);
    memset(dbout, 0, sizeof(double) * (size_t)H);
    /* heads in parallel, the batch in order inside: the sums over b have a fixed order */
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < H; ++h) {
        /* act[l]: input of layer l (act[0] = x), pre[l]: pre-activation of layer l */
        double** act = (double**)malloc(sizeof(double*) * (size_t)(L + 1));
        double** pre = (double**)malloc(sizeof(double*) * (size_t)L);
        for (int l = 0; l <= L; ++l) act[l] = (double*)malloc(sizeof(double) * (size_t)T * cmax);
        for (int l = 0; l < L; ++l) pre[l] = (double*)malloc(sizeof(double) * (size_t)T * cmax);
        double* g = (double*)malloc(sizeof(double) * (size_t)T * cmax);
        double* gp = (double*)malloc(sizeof(double) * (size_t)T * cmax);
        for (int b = 0; b < B; ++b) {
            const size_t bh = (size_t)b * H + h;
            const double* kk = k + bh * T * d;
            const double* vv = v + bh * T * d;
            const double* dzz = dz + bh * T;
            for (int t = 0; t < T; ++t) {
                for (int c = 0; c < d; ++c) act[0][(size_t)t * cmax + c] = kk[(size_t)t * d + c];
                for (int c = 0; c < d; ++c) act[0][(size_t)t * cmax + d + c] = vv[(size_t)t * d + c];
            }
            for (int l = 0; l < L; ++l) {
                const int cin = ch[l], cout = ch[l + 1];
                const double* Wl = wl[l] + (size_t)h * cout * ks * cin;
                const double* Bl = bl[l] ? bl[l] + (size_t)h * cout : NULL;
                for (int t = 0; t < T; ++t)
                    for (int o = 0; o < cout; ++o) {
                        double acc = Bl ? Bl[o] : 0.0;
                        for (int tau = 0; tau < ks; ++tau) {
                            int p = t - (ks - 1 - tau) * dil;
                            if (p < 0) continue;
                            const double* wv = Wl + ((size_t)o * ks + tau) * cin;
                            for (int c = 0; c < cin; ++c) acc += wv[c] * act[l][(size_t)p * cmax + c];
                        }
                        pre[l][(size_t)t * cmax + o] = acc;
                        act[l + 1][(size_t)t * cmax + o] = acc * sigmoid(acc);
                    }
            }
            /* output map: z_j = bout + <wout, act[L][j + half]> */
            memset(g, 0, sizeof(double) * (size_t)T * cmax);
            for (int j = 0; j + half <= T - 1; ++j) {
                const int t = j + half;
                const double dzt = dzz[j];
                dbout[h] += dzt;
                for (int c = 0; c < ch[L]; ++c) {
                    dwout[(size_t)h * ch[L] + c] += dzt * act[L][(size_t)t * cmax + c];
                    g[(size_t)t * cmax + c] = dzt * wout[(size_t)h * ch[L] + c];
                }
            }
            for (int l = L - 1; l >= 0; --l) {
                const int cin = ch[l], cout = ch[l + 1];
                const double* Wl = wl[l] + (size_t)h * cout * ks * cin;
                double* dW = dwl[l] + (size_t)h * cout * ks * cin;
                double* dBl = dbl[l] + (size_t)h * cout;
                memset(gp, 0, sizeof(double) * (size_t)T * cmax);
                for (int t = 0; t < T; ++t)
                    for (int o = 0; o < cout; ++o) {
                        const double y = pre[l][(size_t)t * cmax + o], sg = sigmoid(y);
                        const double delta = g[(size_t)t * cmax + o] * (sg + y * sg * (1.0 - sg));
                        if (delta == 0.0) continue;
                        dBl[o] += delta;
                        for (int tau = 0; tau < ks; ++tau) {
                            int p = t - (ks - 1 - tau) * dil;
                            if (p < 0) continue;
                            const double* wv = Wl + ((size_t)o * ks + tau) * cin;
                            double* dwv = dW + ((size_t)o * ks + tau) * cin;
                            for (int c = 0; c < cin; ++c) {
                                dwv[c] += delta * act[l][(size_t)p * cmax + c];
                                gp[(size_t)p * cmax + c] += delta * wv[c];
                            }
                        }
                    }
                double* tmp = g; g = gp; gp = tmp;
            }
            double* dkk = dk + bh * T * d;
            double* dvv = dv + bh * T * d;
            for (int t = 0; t < T; ++t) {
                for (int c = 0; c < d; ++c) dkk[(size_t)t * d + c] = g[(size_t)t * cmax + c];
                for (int c = 0; c < d; ++c) dvv[(size_t)t * d + c] = g[(size_t)t * cmax + d + c];
            }
        }
        for (int l = 0; l <= L; ++l) free(act[l]);
        for (int l = 0; l < L; ++l) free(pre[l]);
        free(act); free(pre); free(g); free(gp);
    }
}

/* ------------------------------------------------------------------------- */
/* One-shot selection after a T-token prompt (Eq. 5 restricted to tokens already
 * out of the final window, plus the capped capacity of Section 3.1.3).
 * Candidates: j <= T-1-W with (j < sink or z_j > zthr).  Keep the first
 * min(R, #candidates) in the total order, emit ascending by position.        */
typedef struct { int sinkflag; double z; int pos; } cand_t;

static int cand_before(const cand_t* a, const cand_t* b)
{
    if (a->sinkflag != b->sinkflag) return a->sinkflag > b->sinkflag;
    if (a->sinkflag) return a->pos < b->pos;
    if (a->z != b->z) return a->z > b->z;
    return a->pos < b->pos;
}
static int cand_cmp(const void* pa, const void* pb)
{
    const cand_t* a = (const cand_t*)pa; const cand_t* b = (const cand_t*)pb;
    if (cand_before(a, b)) return -1;
    if (cand_before(b, a)) return 1;
    return 0;
}
static int int_cmp(const void* a, const void* b)
{
    int x = *(const int*)a, y = *(const int*)b;
    return (x > y) - (x < y);
}

void oracle_select(int B, int H, int T, int W, int R, int sink, double zthr,
                   const double* z, int32_t* idx, int32_t* cnt, int32_t* ncand)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const double* zz = z + ((size_t)b * H + h) * T;
            int32_t* out = idx + ((size_t)b * H + h) * R;
            int nelig = T - W; if (nelig < 0) nelig = 0;
            cand_t* c = (cand_t*)malloc(sizeof(cand_t) * (size_t)(nelig > 0 ? nelig : 1));
            int n = 0;
            for (int j = 0; j < nelig; ++j) {
                int s = j < sink;
                if (s || zz[j] > zthr) { c[n].sinkflag = s; c[n].z = zz[j]; c[n].pos = j; ++n; }
            }
            qsort(c, (size_t)n, sizeof(cand_t), cand_cmp);
            int keep = n < R ? n : R;
            int* pos = (int*)malloc(sizeof(int) * (size_t)(keep > 0 ? keep : 1));
            for (int i = 0; i < keep; ++i) pos[i] = c[i].pos;
            qsort(pos, (size_t)keep, sizeof(int), int_cmp);
            for (int i = 0; i < R; ++i) out[i] = i < keep ? pos[i] : -1;
            cnt[(size_t)b * H + h] = keep;
            if (ncand) ncand[(size_t)b * H + h] = n;
            free(c); free(pos);
        }
}

/* ------------------------------------------------------------------------- */
/* Prefill attention (Section 3.1.3, "Cached prefilling and decoding"): query i
 * attends over its window {max(0,i-W+1)..i} plus every retained index that is
 * already out of its window (idx <= i-W), softmax(scale * q.k) with natural-log
 * logsumexp.  `qpos` (nq positions per head, may be NULL = all T queries in
 * order) selects which query rows are produced: o [B,H,nq,d], lse [B,H,nq].   */
void oracle_attn_prefill(int B, int H, int T, int d, int W, int R, double scale,
                         const double* q, const double* k, const double* v,
                         const int32_t* idx, const int32_t* cnt,
                         const int32_t* qpos, int nq,
                         double* o, double* lse)
{
    if (!qpos) nq = T;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const size_t bh = (size_t)b * H + h;
            const double* qq = q + bh * T * d;
            const double* kk = k + bh * T * d;
            const double* vv = v + bh * T * d;
            const int32_t* id = idx + bh * R;
            const int n_ret = cnt[bh];
            int* set = (int*)malloc(sizeof(int) * (size_t)(W + R + 1));
            double* s = (double*)malloc(sizeof(double) * (size_t)(W + R + 1));
            for (int a = 0; a < nq; ++a) {
                const int i = qpos ? qpos[bh * nq + a] : a;
                int n = 0;
                for (int m = 0; m < n_ret; ++m) if (id[m] <= i - W) set[n++] = id[m];
                int lo = i - W + 1; if (lo < 0) lo = 0;
                for (int j = lo; j <= i; ++j) set[n++] = j;
                double mx = NEG_INF;
                for (int m = 0; m < n; ++m) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += qq[(size_t)i * d + c] * kk[(size_t)set[m] * d + c];
                    s[m] = acc * scale;
                    if (s[m] > mx) mx = s[m];
                }
                double den = 0.0;
                for (int m = 0; m < n; ++m) { s[m] = exp(s[m] - mx); den += s[m]; }
                double* oo = o + (bh * nq + a) * d;
                for (int c = 0; c < d; ++c) oo[c] = 0.0;
                for (int m = 0; m < n; ++m) {
                    double p = s[m] / den;
                    for (int c = 0; c < d; ++c) oo[c] += p * vv[(size_t)set[m] * d + c];
                }
                lse[bh * nq + a] = mx + log(den);
            }
            free(set); free(s);
        }
}

/* ------------------------------------------------------------------------- */
/* Streaming simulation (Section 3.1.3, decoding paragraph), token by token from
 * an empty cache.  When token n arrives (n = 0..T-1): the window becomes
 * {n-W+1..n}; token p = n-W (if >= 0) has just left it and is offered to the
 * pool: skipped unless (p < sink or z_p > zthr); appended if the pool has room;
 * otherwise it replaces the worst entry (lowest z, the youngest among equals;
 * sink entries are never evicted) iff z_p is strictly greater.  Then query n
 * attends over window + pool.  z is the score array of the WHOLE sequence: every
 * popped token's right context has arrived by then (requires W >= half).
 * Outputs for steps n >= n_from only: o [B,H,T-n_from,d], lse [B,H,T-n_from];
 * final pool positions ascending in pool_idx [B,H,R] (-1 unused), pool_cnt.   */
void oracle_stream(int B, int H, int T, int d, int W, int R, int sink, double zthr,
                   double scale, int n_from,
                   const double* q, const double* k, const double* v, const double* z,
                   double* o, double* lse, int32_t* pool_idx, int32_t* pool_cnt)
{
    const int nout = T - n_from;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const size_t bh = (size_t)b * H + h;
            const double* qq = q + bh * T * d;
            const double* kk = k + bh * T * d;
            const double* vv = v + bh * T * d;
            const double* zz = z + bh * T;
            int* pool = (int*)malloc(sizeof(int) * (size_t)(R > 0 ? R : 1));
            int* set = (int*)malloc(sizeof(int) * (size_t)(W + R + 1));
            double* s = (double*)malloc(sizeof(double) * (size_t)(W + R + 1));
            int cnt = 0;
            for (int n = 0; n < T; ++n) {
                const int p = n - W;
                if (p >= 0 && R > 0 && (p < sink || zz[p] > zthr)) {
                    if (cnt < R) pool[cnt++] = p;
                    else if (p >= sink) {
                        int worst = -1;
                        for (int m = 0; m < cnt; ++m) {
                            if (pool[m] < sink) continue;
                            if (worst < 0 || zz[pool[m]] < zz[pool[worst]] ||
                                (zz[pool[m]] == zz[pool[worst]] && pool[m] > pool[worst]))
                                worst = m;
                        }
                        if (worst >= 0 && zz[p] > zz[pool[worst]]) pool[worst] = p;
                    }
                }
                if (n < n_from) continue;
                int m_ = 0;
                for (int m = 0; m < cnt; ++m) set[m_++] = pool[m];
                int lo = n - W + 1; if (lo < 0) lo = 0;
                for (int j = lo; j <= n; ++j) set[m_++] = j;
                double mx = NEG_INF;
                for (int m = 0; m < m_; ++m) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += qq[(size_t)n * d + c] * kk[(size_t)set[m] * d + c];
                    s[m] = acc * scale;
                    if (s[m] > mx) mx = s[m];
                }
                double den = 0.0;
                for (int m = 0; m < m_; ++m) { s[m] = exp(s[m] - mx); den += s[m]; }
                double* oo = o + (bh * nout + (n - n_from)) * d;
                for (int c = 0; c < d; ++c) oo[c] = 0.0;
                for (int m = 0; m < m_; ++m) {
                    double pw = s[m] / den;
                    for (int c = 0; c < d; ++c) oo[c] += pw * vv[(size_t)set[m] * d + c];
                }
                lse[bh * nout + (n - n_from)] = mx + log(den);
            }
            qsort(pool, (size_t)cnt, sizeof(int), int_cmp);
            for (int m = 0; m < R; ++m) pool_idx[bh * R + m] = m < cnt ? pool[m] : -1;
            pool_cnt[bh] = cnt;
            free(pool); free(set); free(s);
        }
}

/* ------------------------------------------------------------------------- */
/* Backward (Section 3.1.2): attention backward over exactly the sets the
 * forward used, then the straight-through surrogate of Eq. 6,
 *   dL/dr_j := <v_j, dL/dv_j>   (dL/dv_j = the attention's full dV_j),
 * plus, optionally, Eq. 7's derivative lambda_h * 1[r_j > tau]; then through the
 * sigmoid and the single-layer scorer to its weights, bias and (flag) inputs.
 * Outputs dq,dk,dv [B,H,T,d], dw [H,K,2d], dbias [H] (may be NULL), and the
 * intermediate dz [B,H,T] (may be NULL) for inspection.
 * Scores undefined at the tail (j > T-1-half) receive no gradient.           */
void oracle_attn_bwd(int B, int H, int T, int d, int W, int R, int K, double scale,
                     double zthr, int cnn_input_grad,
                     const double* q, const double* k, const double* v, const double* dO,
                     const double* z, const int32_t* idx, const int32_t* cnt,
                     const double* w, const double* lambda,
                     double* dq, double* dk, double* dv, double* dw, double* dbias,
                     double* dz_out)
{
    const int half = K / 2;
    memset(dw, 0, sizeof(double) * (size_t)H * K * 2 * d);
    if (dbias) memset(dbias, 0, sizeof(double) * (size_t)H);
    /* per-(b,h) partial weight gradients, summed over b afterwards in a fixed order */
    double* dw_part = (double*)calloc((size_t)B * H * K * 2 * d, sizeof(double));
    double* db_part = (double*)calloc((size_t)B * H, sizeof(double));
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const size_t bh = (size_t)b * H + h;
            const double* qq = q + bh * T * d;
            const double* kk = k + bh * T * d;
            const double* vv = v + bh * T * d;
            const double* gg = dO + bh * T * d;
            const double* zz = z + bh * T;
            double* dqq = dq + bh * T * d;
            double* dkk = dk + bh * T * d;
            double* dvv = dv + bh * T * d;
            const int32_t* id = idx + bh * R;
            const int n_ret = cnt[bh];
            memset(dqq, 0, sizeof(double) * (size_t)T * d);
            memset(dkk, 0, sizeof(double) * (size_t)T * d);
            memset(dvv, 0, sizeof(double) * (size_t)T * d);
            int* set = (int*)malloc(sizeof(int) * (size_t)(W + R + 1));
            double* pr = (double*)malloc(sizeof(double) * (size_t)(W + R + 1));
            double* oi = (double*)malloc(sizeof(double) * (size_t)d);
            for (int i = 0; i < T; ++i) {
                int n = 0;
                for (int m = 0; m < n_ret; ++m) if (id[m] <= i - W) set[n++] = id[m];
                int lo = i - W + 1; if (lo < 0) lo = 0;
                for (int j = lo; j <= i; ++j) set[n++] = j;
                double mx = NEG_INF;
                for (int m = 0; m < n; ++m) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += qq[(size_t)i * d + c] * kk[(size_t)set[m] * d + c];
                    pr[m] = acc * scale;
                    if (pr[m] > mx) mx = pr[m];
                }
                double den = 0.0;
                for (int m = 0; m < n; ++m) { pr[m] = exp(pr[m] - mx); den += pr[m]; }
                for (int c = 0; c < d; ++c) oi[c] = 0.0;
                for (int m = 0; m < n; ++m) {
                    pr[m] /= den;
                    for (int c = 0; c < d; ++c) oi[c] += pr[m] * vv[(size_t)set[m] * d + c];
                }
                double delta = 0.0;
                for (int c = 0; c < d; ++c) delta += gg[(size_t)i * d + c] * oi[c];
                for (int m = 0; m < n; ++m) {
                    const int j = set[m];
                    double dp = 0.0;
                    for (int c = 0; c < d; ++c) dp += gg[(size_t)i * d + c] * vv[(size_t)j * d + c];
                    const double ds = pr[m] * (dp - delta);
                    for (int c = 0; c < d; ++c) {
                        dvv[(size_t)j * d + c] += pr[m] * gg[(size_t)i * d + c];
                        dqq[(size_t)i * d + c] += scale * ds * kk[(size_t)j * d + c];
                        dkk[(size_t)j * d + c] += scale * ds * qq[(size_t)i * d + c];
                    }
                }
            }
            /* straight-through surrogate and the scorer's backward */
            double* dz = (double*)calloc((size_t)T, sizeof(double));
            for (int j = 0; j + half <= T - 1; ++j) {
                double dr = 0.0;
                for (int c = 0; c < d; ++c) dr += vv[(size_t)j * d + c] * dvv[(size_t)j * d + c];
                const double r = sigmoid(zz[j]);
                if (lambda && zz[j] > zthr) dr += lambda[h];
                dz[j] = dr * r * (1.0 - r);
            }
            double* dwp = dw_part + bh * K * 2 * d;
            for (int j = 0; j + half <= T - 1; ++j) {
                db_part[bh] += dz[j];
                for (int t = 0; t < K; ++t) {
                    const int p = j + t - half;
                    if (p < 0) continue;
                    for (int c = 0; c < d; ++c) {
                        dwp[((size_t)t * 2) * d + c] += dz[j] * kk[(size_t)p * d + c];
                        dwp[((size_t)t * 2 + 1) * d + c] += dz[j] * vv[(size_t)p * d + c];
                    }
                }
            }
            if (cnn_input_grad) {
                for (int j = 0; j + half <= T - 1; ++j)
                    for (int t = 0; t < K; ++t) {
                        const int p = j + t - half;
                        if (p < 0) continue;
                        const double* wt = w + ((size_t)h * K + t) * 2 * d;
                        for (int c = 0; c < d; ++c) {
                            dkk[(size_t)p * d + c] += dz[j] * wt[c];
                            dvv[(size_t)p * d + c] += dz[j] * wt[d + c];
                        }
                    }
            }
            if (dz_out) memcpy(dz_out + bh * T, dz, sizeof(double) * (size_t)T);
            free(dz); free(set); free(pr); free(oi);
        }
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const size_t bh = (size_t)b * H + h;
            for (int e = 0; e < K * 2 * d; ++e) dw[(size_t)h * K * 2 * d + e] += dw_part[bh * K * 2 * d + e];
            if (dbias) dbias[h] += db_part[bh];
        }
    free(dw_part); free(db_part);
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
