/*
 * CPU oracle for the deterministic fused-upcast linear layer  y = x * up(W_bf16)^T (+ b)
 * (paper Eq. 2, design rules R1-R4).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, scalar, obviously-correct restatement of the
 * reduction order; it shares no code with the CUDA path and is never on the product path.  Only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * The result of the method is not "the dot product": it is the outcome of one specific sequence of
 * binary32 roundings (R1: every multiply-accumulate is one IEEE-754 FMA; R3: K is cut into contiguous
 * segments whose partial sums are added in ascending order; R4: nothing depends on M).  The oracle
 * therefore replays the sequence step by step, in the order family (V, L, P, seg_len):
 *
 *   - a segment [k_lo, k_hi) is walked in chunks of C = V*L elements, ascending;
 *   - inside a chunk, "lane" l (0 <= l < L) owns the V consecutive elements  c + l*V + j, j = 0..V-1;
 *   - element j of a lane is accumulated into that lane's sub-chain  p = j mod P, so there are L*P
 *     leaves, leaf index  l*P + p; every accumulation is  a = fmaf(x, up(w), a)  starting from +0.0f;
 *     elements at or beyond k_hi are skipped (not zero-filled);
 *   - the L*P leaves are summed by a balanced binary tree, adjacent leaves first;
 *   - the segment sums are added left to right in ascending segment order (R3, "fixed ascending
 *     segment order"), and the bias, when present, is added last with one rounding (Eq. 2).
 *
 * The paper's own kernels are the member (V, L, P) = (1, 1, 1) of this family (strictly ascending k
 * inside a segment, supplement C on R2).  The production constants are chosen by oracle.py.
 *
 * Parity status: the arithmetic is pinned by hand-traced examples, closed forms, an exact-rational
 * re-implementation, an exact integer special case and an FP64 error bound (tests/test_oracle_*.py).
 * The production constants themselves (V, L, P, bucket edge, split rule) are design choices that
 * the paper does not print: for those, "parity unpinned" beyond the frozen definition.
 *
 * Build: gcc -O2 -std=c99 -ffp-contract=off -fno-fast-math -fopenmp -fPIC -shared (see build_oracle.py).
 * fmaf() comes from libm and is correctly rounded; it is never emulated through double.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#if defined(__x86_64__) || defined(__i386__)
#include <xmmintrin.h>
#define ORACLE_HAVE_MXCSR 1
#endif

#define ORACLE_MAX_LEAVES 4096

/* up(): widen a BF16 bit pattern to binary32 by placing it in the high half (exact; Eq. 2). */
float det_oracle_up(uint16_t h)
{
    uint32_t bits = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

/* Weight formats (the paper's probes cover BF16 and FP32 weights; its abstract speaks of "16-bit
 * weights", which also admits IEEE binary16).  Every format widens exactly to binary32. */
enum { ORACLE_W_BF16 = 0, ORACLE_W_FP16 = 1, ORACLE_W_FP32 = 2 };

/* up() for IEEE binary16: every binary16 value (subnormals included) is a binary32 value. */
float det_oracle_up_fp16(uint16_t h)
{
    const uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
    const uint32_t e = (h >> 10) & 0x1Fu;
    const uint32_t m = h & 0x3FFu;
    uint32_t bits;
    if (e == 0) {
        if (m == 0) {
            bits = sign;                                   /* signed zero */
        } else {
            /* subnormal: m * 2^-24, normalised by hand */
            uint32_t mm = m;
            int shift = 0;
            while ((mm & 0x400u) == 0) { mm <<= 1; ++shift; }
            bits = sign | ((uint32_t)(113 - shift) << 23) | ((mm & 0x3FFu) << 13);
        }
    } else if (e == 31) {
        bits = sign | 0x7F800000u | (m << 13);            /* infinity / NaN */
    } else {
        bits = sign | ((e + 112u) << 23) | (m << 13);
    }
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

static inline float oracle_weight(const void *wrow, int64_t k, int wfmt)
{
    if (wfmt == ORACLE_W_FP32) return ((const float *)wrow)[k];
    if (wfmt == ORACLE_W_FP16) return det_oracle_up_fp16(((const uint16_t *)wrow)[k]);
    return det_oracle_up(((const uint16_t *)wrow)[k]);
}

static inline size_t oracle_weight_bytes(int wfmt) { return wfmt == ORACLE_W_FP32 ? 4 : 2; }

/* Gradual underflow must be on: flush-to-zero / denormals-are-zero would change results for
 * subnormal operands (R1 asks for IEEE-754 arithmetic).  Returns the previous control word. */
static unsigned oracle_enter_ieee(void)
{
#ifdef ORACLE_HAVE_MXCSR
    unsigned old = _mm_getcsr();
    _mm_setcsr(old & ~(0x8000u | 0x0040u));   /* clear FTZ (bit 15) and DAZ (bit 6) */
    return old;
#else
    return 0;
#endif
}
static void oracle_leave_ieee(unsigned old)
{
#ifdef ORACLE_HAVE_MXCSR
    _mm_setcsr(old);
#else
    (void)old;
#endif
}

/* One output element y[m,n]: xrow = x[m,:], wrow = W[n,:], bias = &b[n] or NULL. */
static float oracle_one(const float *xrow, const void *wrow, int wfmt, const float *bias,
                        int64_t K, int V, int L, int P, int64_t seg_len)
{
    float a[ORACLE_MAX_LEAVES];
    const int nleaf = L * P;
    const int64_t C = (int64_t)V * L;
    float t = 0.0f;
    int64_t s = 0;
    for (int64_t k_lo = 0; k_lo < K; k_lo += seg_len, ++s) {
        int64_t k_hi = k_lo + seg_len;
        if (k_hi > K) k_hi = K;
        for (int i = 0; i < nleaf; ++i) a[i] = 0.0f;
        for (int64_t c = k_lo; c < k_hi; c += C) {          /* chunks ascending */
            for (int l = 0; l < L; ++l) {
                for (int j = 0; j < V; ++j) {                /* elements ascending */
                    int64_t k = c + (int64_t)l * V + j;
                    if (k < k_hi) {
                        int leaf = l * P + (j % P);
                        a[leaf] = fmaf(xrow[k], oracle_weight(wrow, k, wfmt), a[leaf]);
                    }
                }
            }
        }
        for (int w = nleaf; w > 1; w /= 2)                   /* adjacent leaves first */
            for (int i = 0; i < w / 2; ++i)
                a[i] = a[2 * i] + a[2 * i + 1];
        t = (s == 0) ? a[0] : (t + a[0]);                    /* ascending segment order */
    }
    return bias ? (t + *bias) : t;                           /* bias last, one rounding */
}

static int oracle_args_ok(int64_t M, int64_t N, int64_t K, int V, int L, int P, int64_t seg_len)
{
    if (M < 0 || N < 0 || K < 1 || V < 1 || L < 1 || P < 1 || seg_len < 1) return 0;
    int nleaf = L * P;
    if (nleaf > ORACLE_MAX_LEAVES || (nleaf & (nleaf - 1)) != 0) return 0;  /* balanced tree */
    if (seg_len % ((int64_t)V * L) != 0 && seg_len < K) return 0;          /* segments start on chunk edges */
    return 1;
}

/* Full problem.  x: [M,K] row-major FP32; W: [N,K] row-major in the given weight format (BF16 or
 * FP16 bit patterns, or FP32 values); b: [N] or NULL; y: [M,N] row-major.  Returns 0 on success, 1 on
 * bad arguments. */
int det_oracle_linear_w(const float *x, const void *W, int wfmt, const float *b, float *y,
                        int64_t M, int64_t N, int64_t K,
                        int V, int L, int P, int64_t seg_len, int nthreads)
{
    if (!oracle_args_ok(M, N, K, V, L, P, seg_len) || wfmt < 0 || wfmt > 2) return 1;
    const size_t wb = oracle_weight_bytes(wfmt);
#ifdef _OPENMP
    if (nthreads < 1) nthreads = omp_get_max_threads();
#else
    (void)nthreads;
#endif
    #pragma omp parallel num_threads(nthreads)
    {
        unsigned csr = oracle_enter_ieee();
        #pragma omp for schedule(static)
        for (int64_t n = 0; n < N; ++n)
            for (int64_t m = 0; m < M; ++m)
                y[m * N + n] = oracle_one(x + m * K, (const char *)W + (size_t)n * K * wb, wfmt, b ? b + n : NULL,
                                          K, V, L, P, seg_len);
        oracle_leave_ieee(csr);
    }
    return 0;
}

int det_oracle_linear(const float *x, const uint16_t *W, const float *b, float *y,
                      int64_t M, int64_t N, int64_t K,
                      int V, int L, int P, int64_t seg_len, int nthreads)
{
    return det_oracle_linear_w(x, W, ORACLE_W_BF16, b, y, M, N, K, V, L, P, seg_len, nthreads);
}

/* Selected outputs only: out[i] = y[ms[i], ns[i]] (for full-size problems where the whole matrix
 * would take too long). */
int det_oracle_linear_sampled_w(const float *x, const void *W, int wfmt, const float *b,
                                const int64_t *ms, const int64_t *ns, int64_t count, float *out,
                                int64_t M, int64_t N, int64_t K,
                                int V, int L, int P, int64_t seg_len, int nthreads)
{
    if (!oracle_args_ok(M, N, K, V, L, P, seg_len) || count < 0 || wfmt < 0 || wfmt > 2) return 1;
    for (int64_t i = 0; i < count; ++i)
        if (ms[i] < 0 || ms[i] >= M || ns[i] < 0 || ns[i] >= N) return 1;
    const size_t wb = oracle_weight_bytes(wfmt);
#ifdef _OPENMP
    if (nthreads < 1) nthreads = omp_get_max_threads();
#else
    (void)nthreads;
#endif
    #pragma omp parallel num_threads(nthreads)
    {
        unsigned csr = oracle_enter_ieee();
        #pragma omp for schedule(static)
        for (int64_t i = 0; i < count; ++i)
            out[i] = oracle_one(x + ms[i] * K, (const char *)W + (size_t)ns[i] * K * wb, wfmt, b ? b + ns[i] : NULL,
                                K, V, L, P, seg_len);
        oracle_leave_ieee(csr);
    }
    return 0;
}

int det_oracle_linear_sampled(const float *x, const uint16_t *W, const float *b,
                              const int64_t *ms, const int64_t *ns, int64_t count, float *out,
                              int64_t M, int64_t N, int64_t K,
                              int V, int L, int P, int64_t seg_len, int nthreads)
{
    return det_oracle_linear_sampled_w(x, W, ORACLE_W_BF16, b, ms, ns, count, out, M, N, K, V, L, P, seg_len, nthreads);
}

/* Greedy argmax per row with the lower index winning a tie (the tie rule stated in the end-to-end
 * determinism section).  -0.0 and +0.0 compare equal; if a row holds a NaN, the first NaN's index
 * is returned (a NaN never occurs for finite inputs). */
int det_oracle_argmax_rows(const float *y, int64_t M, int64_t N, int32_t *idx)
{
    if (M < 0 || N < 1) return 1;
    for (int64_t m = 0; m < M; ++m) {
        const float *row = y + m * N;
        int64_t best = 0;
        if (!isnan(row[0])) {
            for (int64_t n = 1; n < N; ++n) {
                if (isnan(row[n])) { best = n; break; }
                if (row[n] > row[best]) best = n;
            }
        }
        idx[m] = (int32_t)best;
    }
    return 0;
}

/* ---- fixed-order RMSNorm ---------------------------------------------------------------------
 * An extension in the paper's spirit, not one of its kernels: the paper leaves RMSNorm to vendor
 * FP32 kernels and names the reductions outside the linear layers as the residual channel of
 * divergence.  Here the row's sum of squares is reduced in the decode order family
 * (V = 4, L = 32, P = 1, one segment): chunks of 128 elements ascending, lane l owns the 4
 * consecutive elements c + 4 l + j, each element enters its lane's accumulator with one
 * fmaf(x, x, acc) from +0.0f, elements beyond H are skipped, and the 32 lane sums are added by the
 * balanced tree, adjacent lanes first.  Then, each step one IEEE binary32 operation:
 *     mean = ss / (float)H;  t = mean + eps;  r = 1.0f / sqrtf(t);  y[h] = (x[h] * r) * g[h].
 */
float det_oracle_sum_squares(const float *x, int64_t H)
{
    unsigned mx = oracle_enter_ieee();
    float a[32];
    for (int l = 0; l < 32; ++l) a[l] = 0.0f;
    for (int64_t c = 0; c < H; c += 128)
        for (int l = 0; l < 32; ++l)
            for (int j = 0; j < 4; ++j) {
                const int64_t k = c + 4 * (int64_t)l + j;
                if (k < H) a[l] = fmaf(x[k], x[k], a[l]);
            }
    for (int w = 32; w > 1; w /= 2)
        for (int i = 0; i < w / 2; ++i) a[i] = a[2 * i] + a[2 * i + 1];
    oracle_leave_ieee(mx);
    return a[0];
}

int det_oracle_rmsnorm(const float *x, const float *g, float eps, int64_t M, int64_t H, float *y)
{
    if (M < 0 || H < 1 || !x || !g || !y) return 1;
    unsigned mx = oracle_enter_ieee();
    for (int64_t m = 0; m < M; ++m) {
        const float *xr = x + m * H;
        float *yr = y + m * H;
        const float ss = det_oracle_sum_squares(xr, H);
        const float mean = ss / (float)H;
        const float t = mean + eps;
        const float root = sqrtf(t);
        const float r = 1.0f / root;
        for (int64_t h = 0; h < H; ++h) {
            const float xs = xr[h] * r;
            yr[h] = xs * g[h];
        }
    }
    oracle_leave_ieee(mx);
    return 0;
}

/*
 * Fixed-order decode attention (an extension: the paper keeps vendor attention and names the reductions
 * outside the linear layers -- "fixed-order attention" in particular -- as the residual channel of
 * cross-run divergence).  One query row per (batch, head) attends to T cached keys and values:
 *
 *   q [B, Hq, D], k and v [B, Hkv, T, D] (Hq a multiple of Hkv; query head h reads KV head h / (Hq / Hkv)),
 *   o [B, Hq, D], all binary32, row-major.
 *
 * Every step is one IEEE-754 binary32 operation, in an order fixed by (T, D) alone:
 *   1. s_j = dot(q, k_j) * scale.  The dot product runs in the decode lane order over D: chunks of 128
 *      ascending, "lane" l owns the 4 consecutive elements c + 4l + jj, one fmaf per element from +0.0f,
 *      elements beyond D skipped, the 32 lane sums added by the adjacent-first tree; then one multiply.
 *   2. m = max_j s_j (comparisons only: order-free).
 *   3. e_j = exp_det(s_j - m): one subtraction, then det_oracle_exp below (its own fixed sequence).
 *   4. l = sum_j e_j in the same lane order over j: chunks of 128 keys ascending, lane l owns keys
 *      c + 4l + jj, one addition per key from +0.0f, keys beyond T skipped, adjacent-first lane tree.
 *   5. for every d: the keys are cut into segments of 256 (the last may be short); inside a segment
 *      a = fmaf(e_j, v_j[d], a) from +0.0f with j ascending; the segment sums are added left to right in
 *      ascending segment order; o[d] = that sum / l (one division).
 *
 * det_oracle_exp(x), defined for x <= 0 (the only arguments step 3 produces):
 *   x < -104            -> +0.0f
 *   t = x * LOG2E;  n = rintf(t) (nearest, ties to even);
 *   f = fmaf(n, -LN2_HI, x);  f = fmaf(n, -LN2_LO, f);                       (|f| <= 0.35)
 *   p = 1/5040;  p = fmaf(p, f, 1/720);  p = fmaf(p, f, 1/120);  p = fmaf(p, f, 1/24);  p = fmaf(p, f, 1/6);
 *   p = fmaf(p, f, 1/2);  p = fmaf(p, f, 1);  p = fmaf(p, f, 1);             (Taylor, degree 7)
 *   result = p * 2^n, as one exact scaling when n >= -126, else (p * 2^(n+64)) * 2^-64 (the second
 *   multiplication rounds once into the subnormal range).
 * The constants are the binary32 roundings of log2(e), of the two-term split of ln 2 and of the
 * reciprocal factorials (bit patterns in the code).  Accurate to within 2 ulp; what matters here is that
 * the sequence is fixed, so any IEEE-754 implementation reproduces the bits.
 */
static float oracle_f32(uint32_t bits)
{
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

float det_oracle_exp(float x)
{
    unsigned mx = oracle_enter_ieee();
    float r;
    if (x < -104.0f) {
        r = 0.0f;
    } else {
        const float LOG2E = oracle_f32(0x3FB8AA3Bu);      /* 1.44269502162933349609375        */
        const float LN2_HI = oracle_f32(0x3F317200u);     /* 0.693145751953125 (low bits zero) */
        const float LN2_LO = oracle_f32(0x35BFBE8Eu);     /* 1.42860676533018704503775e-06     */
        const float t = x * LOG2E;
        const float n = rintf(t);
        float f = fmaf(n, -LN2_HI, x);
        f = fmaf(n, -LN2_LO, f);
        float p = oracle_f32(0x39500D01u);                /* 1/5040 */
        p = fmaf(p, f, oracle_f32(0x3AB60B61u));          /* 1/720 */
        p = fmaf(p, f, oracle_f32(0x3C088889u));          /* 1/120 */
        p = fmaf(p, f, oracle_f32(0x3D2AAAABu));          /* 1/24  */
        p = fmaf(p, f, oracle_f32(0x3E2AAAABu));          /* 1/6   */
        p = fmaf(p, f, 0.5f);
        p = fmaf(p, f, 1.0f);
        p = fmaf(p, f, 1.0f);
        const int ni = (int)n;
        if (ni >= -126) {
            r = p * oracle_f32((uint32_t)(ni + 127) << 23);
        } else {
            const float u = p * oracle_f32((uint32_t)(ni + 64 + 127) << 23);
            r = u * oracle_f32((uint32_t)(-64 + 127) << 23);
        }
    }
    oracle_leave_ieee(mx);
    return r;
}

/* dot product of two length-D vectors in the decode lane order (step 1 above, before the scale) */
static float oracle_lane_dot(const float *a, const float *b, int64_t D)
{
    float acc[32];
    for (int l = 0; l < 32; ++l) acc[l] = 0.0f;
    for (int64_t c = 0; c < D; c += 128)
        for (int l = 0; l < 32; ++l)
            for (int j = 0; j < 4; ++j) {
                const int64_t k = c + 4 * (int64_t)l + j;
                if (k < D) acc[l] = fmaf(a[k], b[k], acc[l]);
            }
    for (int w = 32; w > 1; w /= 2)
        for (int i = 0; i < w / 2; ++i) acc[i] = acc[2 * i] + acc[2 * i + 1];
    return acc[0];
}

/* sum of T values in the lane order over j (step 4 above) */
static float oracle_lane_sum(const float *e, int64_t T)
{
    float acc[32];
    for (int l = 0; l < 32; ++l) acc[l] = 0.0f;
    for (int64_t c = 0; c < T; c += 128)
        for (int l = 0; l < 32; ++l)
            for (int j = 0; j < 4; ++j) {
                const int64_t k = c + 4 * (int64_t)l + j;
                if (k < T) acc[l] = acc[l] + e[k];
            }
    for (int w = 32; w > 1; w /= 2)
        for (int i = 0; i < w / 2; ++i) acc[i] = acc[2 * i] + acc[2 * i + 1];
    return acc[0];
}

/* the two reductions on their own (exported for the pins) */
float det_oracle_lane_dot(const float *a, const float *b, int64_t D)
{
    unsigned mx = oracle_enter_ieee();
    const float r = oracle_lane_dot(a, b, D);
    oracle_leave_ieee(mx);
    return r;
}

float det_oracle_lane_sum(const float *e, int64_t T)
{
    unsigned mx = oracle_enter_ieee();
    const float r = oracle_lane_sum(e, T);
    oracle_leave_ieee(mx);
    return r;
}

/* scratch: e [T] floats (caller-provided) */
static void oracle_attention_one(const float *q, const float *k, const float *v, float scale, int64_t T, int64_t D,
                                 float *o, float *e)
{
    for (int64_t j = 0; j < T; ++j) e[j] = oracle_lane_dot(q, k + j * D, D) * scale;
    float m = e[0];
    for (int64_t j = 1; j < T; ++j)
        if (e[j] > m) m = e[j];
    for (int64_t j = 0; j < T; ++j) e[j] = det_oracle_exp(e[j] - m);
    const float l = oracle_lane_sum(e, T);
    for (int64_t d = 0; d < D; ++d) {
        float t = 0.0f;
        for (int64_t j0 = 0; j0 < T; j0 += 256) {
            const int64_t j1 = j0 + 256 < T ? j0 + 256 : T;
            float a = 0.0f;
            for (int64_t j = j0; j < j1; ++j) a = fmaf(e[j], v[j * D + d], a);
            t = (j0 == 0) ? a : t + a;
        }
        o[d] = t / l;
    }
}

int det_oracle_attention_decode(const float *q, const float *k, const float *v, float scale, int64_t B, int64_t Hq,
                                int64_t Hkv, int64_t T, int64_t D, float *o, float *scratch /* [T] per thread: T * threads */)
{
    if (!q || !k || !v || !o || !scratch || B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || T < 1 || D < 1) return 1;
    unsigned mx = oracle_enter_ieee();
    const int64_t G = Hq / Hkv;
    int64_t bh;
#pragma omp parallel for schedule(static)
    for (bh = 0; bh < B * Hq; ++bh) {
        unsigned mxt = oracle_enter_ieee();
        const int64_t b = bh / Hq, h = bh % Hq, hk = h / G;
#ifdef _OPENMP
        float *e = scratch + (int64_t)omp_get_thread_num() * T;
#else
        float *e = scratch;
#endif
        oracle_attention_one(q + (b * Hq + h) * D, k + ((b * Hkv + hk) * T) * D, v + ((b * Hkv + hk) * T) * D, scale, T, D,
                             o + (b * Hq + h) * D, e);
        oracle_leave_ieee(mxt);
    }
    oracle_leave_ieee(mx);
    return 0;
}

int det_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
