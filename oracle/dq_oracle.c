/*
 * D-Quant CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, single-translation-unit C implementation of what the D-Quant hot
 * path computes, written from the paper (D-Quant: Driftable Entropy Coding for KV
 * Cache Quantization) step by step, in the paper's order and notation.  It shares
 * no code, header, table or constant generator with the CUDA library.  Only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Passages followed:
 *   Eq. (rans)            Enc/Dec state update, precision p = 8
 *   Eq. (budget)          B = 8C - sigma
 *   Eq. (affine_token)    s = (max - min)/(M-1), o = min
 *   Eq. (drift), (lagrangian), Algorithm 1   encoder of one stream
 *   Algorithm 2           decoder of one stream
 *   Sec. 4.2              Hadamard rotation, windowed channel mean for keys,
 *                         probability model from Gaussian order statistics
 *   Sec. 4.4              sharpening p' ~ p^alpha
 *   Appendix A            reconstruction k = s*v + o + mu, folded contractions
 *
 * Where the paper is silent the numerical contract below fixes one reading (the
 * same list is in the design notes of the repository):
 *   - a stream is the n values of one (token, KV head); a table with n > 128
 *     describes the paper's default grouping instead (Sec. 5.1: a token is
 *     quantised as a single group): the stream spans n/128 consecutive KV heads
 *     of a token, each head rotated and mean-centred on its own, one (s, o) pair
 *     and one container for the whole group;
 *   - sigma = 32, L = 2^23, 32-bit state, byte-wise renormalisation (Algorithm 2
 *     reads bytes);
 *   - the record is [s fp16][o fp16][state u32 LE][payload bytes][zero padding];
 *   - the probability of level m is the N(0,1) mass of its cell on a grid that
 *     spans +-E[max of n normals], cells clipped to that span;
 *   - the bisection of log2(lambda) is done as a geometric mean sqrt(lo*hi);
 *   - code length is summed in 1/65536-bit fixed point, rounded up per symbol.
 * Opt-in variants of the codec (off unless a table asks for them; the defaults above are
 * untouched by them):
 *   - early exit of Drift (table field early_exit): Algorithm 1's bisection ends at a known
 *     multiplier when every one of its 12 tests passes; that assignment is evaluated first
 *     and returned if it meets the budget, else the full bisection runs (App. C: most
 *     streams have budget to spare, so most take the short path);
 *   - sigma = 24 (table field sigma): the state lives in [2^15, 2^23) and its final value
 *     takes 3 bytes of the container instead of 4 (Eq. budget: B = 8C - sigma), one byte
 *     per stream back for symbols; streams of at most 640 values (five heads) only;
 *   - paired symbols (table field pair): one rANS symbol is the pair of levels of two
 *     consecutive values (2i, 2i + 1), u = m_2i M + m_2i+1, over an alphabet of M^2 <= 256
 *     pairs whose model is the product of the sharpened level model with itself, made
 *     integer by the same rule as the level table (Sec. 3.1: the coder is the same Eq. rans
 *     on a larger alphabet; a decoder then takes n / 2 steps for n values).  Drift assigns
 *     a pair at a time: argmin over the M^2 pairs of D_a + D_b + lambda r_ab.
 *
 * Pins (tests/test_oracle_*.py): closed-form storage accounting, the feasibility
 * boundary and NMSE curve of Table 2, rANS round trip, Shannon bound, orthonormal
 * self-inverse Hadamard, brute-force drift optimality, textbook special cases; the
 * Refit of Algorithm 1 against a library least-squares solve rounded once to binary16,
 * with its summation order shown to change no record (tests/test_oracle_refit.py).
 * PARITY UNPINNED by the paper (defined only by this build's contract): the mean
 * carry-forward rule for appended tokens and the automatic choice of alpha.  (The INT8
 * window-mean quantiser is pinned to a library per-tensor quantiser.)
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define DQO_MAX_LEVELS 16
#define DQO_MAX_N 1024
#define DQO_P 8            /* rANS precision: sum f = 2^p (Sec. 3.1)              */
#define DQO_TOT 256
#define DQO_SIGMA 32       /* bits of final state stored in the record (default)   */
#define DQO_WINDOW 128     /* tokens per channel-mean window                       */
#define DQO_PAGE 16        /* tokens per physical page                             */
#define DQO_HEAD 128       /* head dimension of the token-level entry points       */

typedef struct {
    int M, n, rec, C, B;           /* levels, stream length, record bytes, C=rec-4, B=8C-32 */
    int mstar, feasible, has_mean, rotate;
    double alpha, E;               /* sharpening exponent, E[max of n N(0,1)]       */
    double p[DQO_MAX_LEVELS];      /* analytic cell probabilities                   */
    double q[DQO_MAX_LEVELS];      /* sharpened                                     */
    int32_t f[DQO_MAX_LEVELS];     /* integer frequencies, sum 256                  */
    int32_t c[DQO_MAX_LEVELS + 1]; /* cumulative                                    */
    float r[DQO_MAX_LEVELS];       /* ideal cost -log2(f/256) in bits (Alg. 1)      */
    uint32_t R[DQO_MAX_LEVELS];    /* ceil(r * 65536)                               */
    uint8_t lut_m[DQO_TOT], lut_f[DQO_TOT], lut_d[DQO_TOT]; /* T[z] = (m, f_m, z - c_m) */
    int sigma;                     /* bits of final state in the record: 32 (default) or 24  */
    int early_exit;                /* 1: Drift first tries the multiplier the bisection ends at when all tests pass */
    /* paired-symbol variant: alphabet of the pairs u = a M + b (a: value 2i, b: value 2i + 1) */
    int pair, ustar;               /* 1: rANS symbols are pairs; most probable pair                    */
    int32_t pf[DQO_TOT];           /* integer pair frequencies, sum 256                               */
    int32_t pc[DQO_TOT + 1];       /* cumulative                                                      */
    float pr[DQO_TOT];             /* ideal cost of a pair, -log2(pf/256) bits                        */
    uint32_t pR[DQO_TOT];          /* ceil(pr * 65536)                                                */
    uint8_t plut_u[DQO_TOT], plut_f[DQO_TOT], plut_d[DQO_TOT]; /* T[z] = (u, pf_u, z - pc_u)          */
} dqo_table;

/* lower bound L of the normalised state interval [L, 2^8 L): 2^23 for sigma = 32, 2^15 for 24 */
static uint32_t dqo_L(const dqo_table *T) { return 1u << (T->sigma - 9); }

/* ------------------------------------------------------------------ numbers */

static double dqo_cdf(double x) { return 0.5 * erfc(-x / sqrt(2.0)); }
static double dqo_pdf(double x) { return exp(-0.5 * x * x) / sqrt(2.0 * M_PI); }

/* E[max of n iid N(0,1)] = int x n phi(x) Phi(x)^(n-1) dx, composite Simpson on
 * [-8, 8] with 2^16 intervals ("Gaussian order statistics", Sec. 4.2). */
double dqo_expected_max(int n)
{
    const int N = 65536;
    const double a = -8.0, b = 8.0, h = (b - a) / N;
    double sum = 0.0;
    for (int i = 0; i <= N; ++i) {
        double x = a + i * h;
        double g = x * n * dqo_pdf(x) * pow(dqo_cdf(x), n - 1);
        double w = (i == 0 || i == N) ? 1.0 : ((i & 1) ? 4.0 : 2.0);
        sum += w * g;
    }
    return sum * h / 3.0;
}

float dqo_bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* binary64 -> binary16, round to nearest even, one rounding (Alg. 1, fp16(s), fp16(o)) */
uint16_t dqo_f64_to_f16(double v)
{
    uint64_t b;
    memcpy(&b, &v, 8);
    uint16_t sign = (uint16_t)((b >> 63) << 15);
    int ex = (int)((b >> 52) & 0x7ff);
    uint64_t mant = b & ((1ull << 52) - 1);
    if (ex == 0x7ff) return (uint16_t)(sign | 0x7c00 | (mant ? 0x200 : 0));
    if (ex == 0) return sign; /* binary64 subnormals are far below half's range */
    int e = ex - 1023;
    if (e > 15) return (uint16_t)(sign | 0x7c00);
    uint64_t m = (1ull << 52) | mant;
    int shift, hexp;
    if (e >= -14) { shift = 42; hexp = e + 15; m = mant; }
    else { shift = 42 + (-14 - e); hexp = 0; }
    if (shift >= 54) return sign;
    uint64_t keep = m >> shift;
    uint64_t rem = m & ((1ull << shift) - 1);
    uint64_t half = 1ull << (shift - 1);
    if (rem > half || (rem == half && (keep & 1))) keep += 1;
    uint32_t out = ((uint32_t)hexp << 10) + (uint32_t)keep; /* a carry bumps the exponent */
    if (out >= 0x7c00) out = 0x7c00;
    return (uint16_t)(sign | out);
}

float dqo_f16_to_f32(uint16_t h)
{
    int sign = h >> 15, ex = (h >> 10) & 31, mant = h & 1023;
    double v;
    if (ex == 31) v = mant ? NAN : INFINITY;
    else if (ex == 0) v = ldexp((double)mant, -24);
    else v = ldexp((double)(1024 + mant), ex - 25);
    return (float)(sign ? -v : v);
}

/* ------------------------------------------------------------------- tables */

/* Integer frequencies of a K-symbol alphabet with targets t[k] = 256 * probability: floor, at
 * least 1, then adjusted to sum 256. */
static void dqo_integer_freqs(const double *t, int K, int32_t *f)
{
    int tot = 0;
    for (int k = 0; k < K; ++k) {
        int fl = (int)floor(t[k]);
        f[k] = fl < 1 ? 1 : fl;
        tot += f[k];
    }
    while (tot < DQO_TOT) { /* largest remainder; tie -> lowest index */
        int best = 0;
        for (int k = 1; k < K; ++k)
            if (t[k] - f[k] > t[best] - f[best]) best = k;
        f[best] += 1; tot += 1;
    }
    while (tot > DQO_TOT) { /* largest excess among f > 1; tie -> highest index */
        int best = -1;
        for (int k = 0; k < K; ++k)
            if (f[k] > 1 && (best < 0 || f[k] - t[k] >= f[best] - t[best])) best = k;
        f[best] -= 1; tot -= 1;
    }
}

/* Pair alphabet of the paired-symbol variant: probability of the pair (a, b) = q_a q_b. */
static void dqo_fill_pair_freqs(dqo_table *T)
{
    int M = T->M, K = M * M;
    double t[DQO_TOT];
    for (int a = 0; a < M; ++a)
        for (int b = 0; b < M; ++b) t[a * M + b] = DQO_TOT * (T->q[a] * T->q[b]);
    dqo_integer_freqs(t, K, T->pf);
    T->pc[0] = 0;
    T->ustar = 0;
    for (int u = 0; u < K; ++u) {
        T->pc[u + 1] = T->pc[u] + T->pf[u];
        double r = (double)DQO_P - log2((double)T->pf[u]);
        T->pr[u] = (float)r;
        T->pR[u] = (uint32_t)ceil(r * 65536.0);
        if (T->pf[u] > T->pf[T->ustar]) T->ustar = u;
    }
    for (int u = 0; u < K; ++u)
        for (int z = T->pc[u]; z < T->pc[u + 1]; ++z) {
            T->plut_u[z] = (uint8_t)u;
            T->plut_f[z] = (uint8_t)T->pf[u];
            T->plut_d[z] = (uint8_t)(z - T->pc[u]);
        }
    T->feasible = ((int64_t)(T->n / 2) * T->pR[T->ustar] <= (int64_t)T->B * 65536);
}

static void dqo_fill_freqs(dqo_table *T)
{
    int M = T->M;
    double qs = 0.0, t[DQO_MAX_LEVELS];
    for (int m = 0; m < M; ++m) { T->q[m] = pow(T->p[m], T->alpha); qs += T->q[m]; }
    for (int m = 0; m < M; ++m) {
        T->q[m] /= qs;
        t[m] = DQO_TOT * T->q[m];
    }
    dqo_integer_freqs(t, M, T->f);
    T->c[0] = 0;
    T->mstar = 0;
    for (int m = 0; m < M; ++m) {
        T->c[m + 1] = T->c[m] + T->f[m];
        double r = (double)DQO_P - log2((double)T->f[m]);
        T->r[m] = (float)r;
        T->R[m] = (uint32_t)ceil(r * 65536.0);
        if (T->f[m] > T->f[T->mstar]) T->mstar = m;
    }
    for (int m = 0; m < M; ++m)
        for (int z = T->c[m]; z < T->c[m + 1]; ++z) {
            T->lut_m[z] = (uint8_t)m;
            T->lut_f[z] = (uint8_t)T->f[m];
            T->lut_d[z] = (uint8_t)(z - T->c[m]);
        }
    T->feasible = ((int64_t)T->n * T->R[T->mstar] <= (int64_t)T->B * 65536);
    if (T->pair) dqo_fill_pair_freqs(T);
}

/* entropy of the integer table in bits per value */
static double dqo_entropy256(const dqo_table *T)
{
    double H = 0.0;
    if (T->pair) {
        for (int u = 0; u < T->M * T->M; ++u) {
            double pu = T->pf[u] / 256.0;
            H -= pu * log2(pu);
        }
        return H / 2.0;
    }
    for (int m = 0; m < T->M; ++m) {
        double pm = T->f[m] / 256.0;
        H -= pm * log2(pm);
    }
    return H;
}

/* Build the probability model and rANS tables of one tensor kind.
 * alpha >= 0: used as given.  alpha < 0: smallest alpha in {1.4, 1.5, ..., 32.0}
 * whose table has entropy <= B/n and lets the all-central stream fit.
 * Returns 0, or -1 for bad arguments, -2 when no feasible table exists. */
int dqo_build_table_ex(int M, int n, int rec_bytes, double alpha, int has_mean, int rotate,
                       int sigma, int early_exit, int pair, dqo_table *T)
{
    if (M < 2 || M > DQO_MAX_LEVELS || n < 1 || n > DQO_MAX_N || rec_bytes < 9) return -1;
    if (sigma != 32 && sigma != 24) return -1;
    if (pair && (n % 2)) return -1;                    /* M <= 16 keeps the pair alphabet within 2^p */
    /* With the 24-bit state an encode step may lose up to log2(1 + 2^-7) bits to floor(x / f)
     * (x >= 2^15, f < 2^8).  The budget test keeps sum r <= B = 8(C - 3); the stream then fits
     * its C bytes as long as the accumulated loss stays below one byte: n log2(1 + 2^-7) < 8,
     * i.e. n <= 712.  Longer streams would need a byte of margin, which is the byte the
     * variant saves, so they are not offered. */
    if (sigma == 24 && n > 640) return -1;
    memset(T, 0, sizeof *T);
    T->M = M; T->n = n; T->rec = rec_bytes; T->C = rec_bytes - 4;
    T->sigma = sigma; T->early_exit = early_exit ? 1 : 0; T->pair = pair ? 1 : 0;
    T->B = 8 * T->C - sigma;                           /* Eq. (budget) */
    T->has_mean = has_mean; T->rotate = rotate;
    T->E = dqo_expected_max(n);
    double E = T->E, delta = 2.0 * E / (M - 1), ps = 0.0;
    for (int m = 0; m < (M + 1) / 2; ++m) {
        double lev = -E + m * delta;
        double lo = fmax(-E, lev - delta / 2), hi = fmin(E, lev + delta / 2);
        T->p[m] = dqo_cdf(hi) - dqo_cdf(lo);
        T->p[M - 1 - m] = T->p[m];
    }
    for (int m = 0; m < M; ++m) ps += T->p[m];
    for (int m = 0; m < M; ++m) T->p[m] /= ps;
    if (alpha >= 0.0) {
        T->alpha = alpha;
        dqo_fill_freqs(T);
        return T->feasible ? 0 : -2;
    }
    for (int k = 14; k <= 320; ++k) {
        T->alpha = k / 10.0;
        dqo_fill_freqs(T);
        if (T->feasible && dqo_entropy256(T) <= (double)T->B / n) return 0;
    }
    return -2;
}

/* The paper's codec: sigma = 32, no early exit. */
int dqo_build_table(int M, int n, int rec_bytes, double alpha, int has_mean, int rotate,
                    dqo_table *T)
{
    return dqo_build_table_ex(M, n, rec_bytes, alpha, has_mean, rotate, DQO_SIGMA, 0, 0, T);
}

int dqo_table_size(void) { return (int)sizeof(dqo_table); }

/* ---------------------------------------------------------------- Hadamard */

/* Fast Walsh-Hadamard transform in binary32: stages h = 1, 2, 4, ... ; each pair
 * (i, i+h) with (i & h) == 0 becomes (a + b, a - b); then a scale by 1/sqrt(n)
 * rounded to binary32.  Per-head rotation of Sec. 4.2. */
void dqo_fwht_f32(float *x, int n)
{
    for (int h = 1; h < n; h <<= 1)
        for (int i = 0; i < n; ++i)
            if ((i & h) == 0) {
                float a = x[i], b = x[i + h];
                x[i] = a + b;
                x[i + h] = a - b;
            }
    float sc = (float)(1.0 / sqrt((double)n));
    for (int i = 0; i < n; ++i) x[i] = x[i] * sc;
}

void dqo_fwht_f64(double *x, int n)
{
    for (int h = 1; h < n; h <<= 1)
        for (int i = 0; i < n; ++i)
            if ((i & h) == 0) {
                double a = x[i], b = x[i + h];
                x[i] = a + b;
                x[i + h] = a - b;
            }
    double sc = 1.0 / sqrt((double)n);
    for (int i = 0; i < n; ++i) x[i] *= sc;
}

/* ------------------------------------------------------------------- drift */

/* One sweep of Drift at the multiplier lam: every rANS symbol takes the candidate that minimises
 * distortion + lam * ideal cost (the lowest index among equal costs); returns the fixed-point code
 * length of the assignment.  t[m] = grid level m.  A symbol is one value, or with the paired-symbol
 * variant the values (2i, 2i + 1) with the M^2 candidates u = a M + b taken in ascending u. */
static int64_t dqo_assign(const float *z, int n, const float *t, float lam, const dqo_table *T,
                          uint8_t *m_out)
{
    int M = T->M;
    int64_t len = 0;
    if (T->pair) {
        for (int i = 0; i < n / 2; ++i) {
            int best = 0;
            float bestc = 0.0f;
            for (int a = 0; a < M; ++a)
                for (int b = 0; b < M; ++b) {
                    float da = z[2 * i] - t[a], db = z[2 * i + 1] - t[b];
                    float Da = da * da, Db = db * db;
                    float D = Da + Db;
                    float cost = fmaf(lam, T->pr[a * M + b], D);
                    if ((a == 0 && b == 0) || cost < bestc) { bestc = cost; best = a * M + b; }
                }
            m_out[2 * i] = (uint8_t)(best / M);
            m_out[2 * i + 1] = (uint8_t)(best % M);
            len += T->pR[best];
        }
        return len;
    }
    for (int j = 0; j < n; ++j) {
        int best = 0;
        float bestc = 0.0f;
        for (int m = 0; m < M; ++m) {
            float d = z[j] - t[m];
            float D = d * d;
            float cost = fmaf(lam, T->r[m], D);
            if (m == 0 || cost < bestc) { bestc = cost; best = m; }
        }
        m_out[j] = (uint8_t)best;
        len += T->R[best];
    }
    return len;
}

/* Function Drift of Algorithm 1: Lagrangian bisection (T = 12) on log2(lambda),
 * realised as the geometric mean of the bracket; returns argmin at `hi`.
 * z: stream values, (s, o): grid.  Writes symbols to m_out and returns the
 * fixed-point code length sum_j R[m_j] (compare with B * 65536). */
int64_t dqo_drift(const float *z, int n, float s, float o, const dqo_table *T, uint8_t *m_out)
{
    int M = T->M;
    float t[DQO_MAX_LEVELS];
    for (int m = 0; m < M; ++m) t[m] = fmaf((float)m, s, o);
    float maxD = -INFINITY, minD = INFINITY;
    for (int j = 0; j < n; ++j)
        for (int m = 0; m < M; ++m) {
            float d = z[j] - t[m];
            float D = d * d;
            if (D > maxD) maxD = D;
            if (D < minD) minD = D;
        }
    const int64_t budget = (int64_t)T->B * 65536;
    /* upper end of the bracket: a multiplier at which 1/8 bit outweighs any difference in
     * distortion between two candidates (a pair's distortion is the sum of two values') */
    float lam_hi = (T->pair ? 16.0f : 8.0f) * (maxD - minD);
    float lam_lo = lam_hi * 0x1p-40f;
    int64_t len = 0;
    if (T->early_exit) {
        /* When each of the 12 tests passes, the bracket's upper end walks hi <- sqrt(lo * hi)
         * twelve times with lo fixed; the assignment at that multiplier is what the loop below
         * would return.  Evaluate it first and stop if it meets the budget. */
        float lam_e = lam_hi;
        for (int it = 0; it < 12; ++it) lam_e = sqrtf(lam_lo * lam_e);
        len = dqo_assign(z, n, t, lam_e, T, m_out);
        if (len <= budget) return len;
    }
    for (int it = 0; it <= 12; ++it) {
        float lam = (it < 12) ? sqrtf(lam_lo * lam_hi) : lam_hi;
        len = dqo_assign(z, n, t, lam, T, m_out);
        if (it < 12) {
            if (len <= budget) lam_hi = lam; else lam_lo = lam;
        }
    }
    return len;
}

/* -------------------------------------------------------------------- rANS */

/* Eq. (rans) Enc applied to symbols n-1 ... 0 (so that decoding runs forward),
 * byte-wise renormalisation.  Writes the final state (sigma / 8 bytes LE) followed by the
 * emitted bytes in reverse order of emission into `payload` (capacity cap bytes).
 * Returns the number of renormalisation bytes k, or -1 if sigma / 8 + k > cap. */
int dqo_rans_encode(const uint8_t *sym, int n, const dqo_table *T, uint8_t *payload, int cap)
{
    uint8_t tmp[2 * DQO_MAX_N];
    int k = 0, sb = T->sigma / 8;                      /* bytes of final state */
    uint32_t L = dqo_L(T), x = L;
    int step = T->pair ? 2 : 1;                        /* values per rANS symbol */
    for (int j = n - step; j >= 0; j -= step) {
        uint32_t f, c;
        if (T->pair) { int u = sym[j] * T->M + sym[j + 1]; f = (uint32_t)T->pf[u]; c = (uint32_t)T->pc[u]; }
        else { f = (uint32_t)T->f[sym[j]]; c = (uint32_t)T->c[sym[j]]; }
        while (x >= f * L) { tmp[k++] = (uint8_t)(x & 255u); x >>= 8; }   /* x_max = f (L / 2^p) 2^8 */
        x = (x / f) * DQO_TOT + (x % f) + c;
    }
    if (sb + k > cap) return -1;
    for (int i = 0; i < sb; ++i) payload[i] = (uint8_t)(x >> (8 * i));
    for (int i = 0; i < k; ++i) payload[sb + i] = tmp[k - 1 - i];
    for (int i = sb + k; i < cap; ++i) payload[i] = 0;
    return k;
}

/* Algorithm 2.  payload = C bytes (state first).  Reads never pass payload[cap-1]
 * (a malformed record gives wrong symbols, not an out-of-bounds read).
 * end[0] = final state, end[1] = final ptr. */
void dqo_rans_decode(const uint8_t *payload, int cap, int n, const dqo_table *T, uint8_t *sym,
                     uint32_t *end)
{
    uint32_t x = 0, L = dqo_L(T);
    int ptr = T->sigma / 8;
    for (int i = 0; i < ptr; ++i) x |= (uint32_t)payload[i] << (8 * i);
    int step = T->pair ? 2 : 1;
    for (int i = 0; i + step <= n; i += step) {
        uint32_t z = x & (DQO_TOT - 1);
        uint32_t f, d;
        if (T->pair) {
            f = T->plut_f[z]; d = T->plut_d[z];
            sym[i] = (uint8_t)(T->plut_u[z] / T->M);
            sym[i + 1] = (uint8_t)(T->plut_u[z] % T->M);
        } else {
            f = T->lut_f[z]; d = T->lut_d[z];
            sym[i] = T->lut_m[z];
        }
        x = f * (x >> DQO_P) + d;
        while (x < L && ptr < cap) { x = (x << 8) | payload[ptr]; ptr += 1; }
    }
    if (end) { end[0] = x; end[1] = (uint32_t)ptr; }
}

/* ------------------------------------------------------- one stream encoder */

/* Algorithm 1 for one stream of already rotated, mean-removed values z[n]
 * (n a multiple of 32).  rec receives T->rec bytes.  stats (nullable, 4 words):
 * [0] += streams that fell back to the all-central assignment, [1] += degenerate
 * (constant) streams, [2] += streams whose refit was rejected, [3] = max bytes used.
 * sym_out (nullable) receives the final symbols. */
/* the most probable symbol everywhere (a pair's two levels with the paired-symbol variant) */
static void dqo_all_central(const dqo_table *T, uint8_t *m)
{
    for (int j = 0; j < T->n; ++j)
        m[j] = (uint8_t)(!T->pair ? T->mstar : (j % 2 == 0 ? T->ustar / T->M : T->ustar % T->M));
}

void dqo_encode_stream(const float *z, const dqo_table *T, uint8_t *rec, uint32_t *stats,
                       uint8_t *sym_out)
{
    int n = T->n, M = T->M;
    uint8_t m[DQO_MAX_N];
    uint16_t s16 = 0, o16 = 0;
    const int64_t budget = (int64_t)T->B * 65536;
    float mx = -INFINITY, mn = INFINITY;
    for (int j = 0; j < n; ++j) { if (z[j] > mx) mx = z[j]; if (z[j] < mn) mn = z[j]; }
    int degenerate = !(mx > mn);
    if (!degenerate) {
        float o = mn;                                  /* FitMinMax, Eq. (affine_token) */
        float s = (mx - mn) / (float)(M - 1);
        dqo_drift(z, n, s, o, T, m);                   /* first Drift                   */
        /* Refit: least squares of z on m.  Sums in binary64 in a fixed order.  A block is
         * the whole stream when n <= 128, else 128 consecutive values (one head): within a
         * block each of 32 lanes adds its consecutive elements in order, then an
         * xor-butterfly 16,8,4,2,1 joins the lanes; block sums are added in block order. */
        int64_t Sm = 0, Smm = 0;
        double Sz = 0.0, Smz = 0.0;
        int blk = n > DQO_HEAD ? DQO_HEAD : n, bper = blk / 32;
        for (int b0 = 0; b0 < n; b0 += blk) {
            double lz[32], lmz[32];
            for (int l = 0; l < 32; ++l) {
                double a = 0.0, b = 0.0;
                for (int e = 0; e < bper; ++e) {
                    int j = b0 + l * bper + e;
                    if (e == 0) { a = (double)z[j]; b = (double)m[j] * (double)z[j]; }
                    else { a = a + (double)z[j]; b = b + (double)m[j] * (double)z[j]; }
                    Sm += m[j]; Smm += (int64_t)m[j] * m[j];
                }
                lz[l] = a; lmz[l] = b;
            }
            for (int d = 16; d >= 1; d >>= 1) {
                double tz[32], tmz[32];
                for (int l = 0; l < 32; ++l) { tz[l] = lz[l] + lz[l ^ d]; tmz[l] = lmz[l] + lmz[l ^ d]; }
                memcpy(lz, tz, sizeof tz); memcpy(lmz, tmz, sizeof tmz);
            }
            if (b0 == 0) { Sz = lz[0]; Smz = lmz[0]; }
            else { Sz = Sz + lz[0]; Smz = Smz + lmz[0]; }
        }
        int64_t den = (int64_t)n * Smm - Sm * Sm;
        double sd = (double)s, od = (double)o;
        if (den != 0) {
            sd = ((double)n * Smz - (double)Sm * Sz) / (double)den;
            od = (Sz - sd * (double)Sm) / (double)n;
        }
        s16 = dqo_f64_to_f16(sd);                      /* fp16 metadata                 */
        o16 = dqo_f64_to_f16(od);
        float sf = dqo_f16_to_f32(s16), of = dqo_f16_to_f32(o16);
        if (!(isfinite(sf) && sf > 0.0f && isfinite(of))) {
            s16 = dqo_f64_to_f16((double)s);
            o16 = dqo_f64_to_f16((double)o);
            sf = dqo_f16_to_f32(s16); of = dqo_f16_to_f32(o16);
            if (stats) stats[2] += 1;
        }
        if (!(sf > 0.0f)) degenerate = 1;
        else {
            int64_t len = dqo_drift(z, n, sf, of, T, m); /* second Drift on the fp16 grid */
            if (len > budget) {
                dqo_all_central(T, m);
                if (stats) stats[0] += 1;
            }
        }
    }
    if (degenerate) {
        s16 = 0;
        o16 = dqo_f64_to_f16((double)mn);
        dqo_all_central(T, m);
        if (stats) stats[1] += 1;
    }
    rec[0] = (uint8_t)s16; rec[1] = (uint8_t)(s16 >> 8);
    rec[2] = (uint8_t)o16; rec[3] = (uint8_t)(o16 >> 8);
    int k = dqo_rans_encode(m, n, T, rec + 4, T->C);
    if (k < 0) { memset(rec + 4, 0, (size_t)T->C); k = 0; } /* excluded by the budget test */
    if (stats && (uint32_t)(4 + T->sigma / 8 + k) > stats[3]) stats[3] = (uint32_t)(4 + T->sigma / 8 + k);
    if (sym_out) memcpy(sym_out, m, (size_t)n);
}

/* ------------------------------------------------------- rotary embedding */

/* Rotary position embedding of one head vector x[d] in binary32 (keys only; applied before the
 * Hadamard rotation when the caller hands over keys that have not been rotated yet).  cs / sn are
 * the caller's tables for this token's position, d/2 entries each.  style 1 pairs element j with
 * j + d/2 (the "rotate half" convention), style 2 pairs 2j with 2j + 1:
 *   (a, b) -> (a cos_j - b sin_j, b cos_j + a sin_j), each product and each sum rounded once. */
void dqo_rope_f32(float *x, int d, const float *cs, const float *sn, int style)
{
    int half = d / 2;
    for (int j = 0; j < half; ++j) {
        int ia = style == 1 ? j : 2 * j, ib = style == 1 ? j + half : 2 * j + 1;
        float a = x[ia], b = x[ib];
        float ac = a * cs[j], bs = b * sn[j], bc = b * cs[j], as = a * sn[j];
        x[ia] = ac - bs;
        x[ib] = bc + as;
    }
}

/* ----------------------------------------------------------- window means */

static void dqo_quantise_mean(float *mu, int n, int8_t *q, float *scale)
{
    float amax = 0.0f;
    for (int j = 0; j < n; ++j) { float a = fabsf(mu[j]); if (a > amax) amax = a; }
    float sc = amax / 127.0f;
    *scale = sc;
    for (int j = 0; j < n; ++j) {
        float v = 0.0f;
        if (sc != 0.0f) {
            v = rintf(mu[j] / sc);
            if (v > 127.0f) v = 127.0f;
            if (v < -127.0f) v = -127.0f;
        }
        q[j] = (int8_t)v;
    }
}

/* Windowed channel mean of keys (Sec. 4.2), window = 128 tokens, stored INT8 with
 * one binary32 scale per (sequence, window, head).
 * mode 0 (compute): every maximal run of consecutive call tokens with the same
 *   (seq_id, pos / 128) gives that window's mean: binary32 sequential sum over the
 *   run, times 1/count, rotated, quantised.
 * mode 1 (reuse): a token with pos % 128 == 0 first copies the previous window's
 *   (q, scale) into its own window slot (window 0: zeros); nothing else changes. */
void dqo_window_means(const uint16_t *k_bf16, int T_tok, int Hkv, int n, const int32_t *seq_id,
                      const int32_t *pos, int8_t *mean_q, float *mean_scale, int Wmax, int mode,
                      int rotate, const float *rope_cos, const float *rope_sin, int rope_style)
{
    if (mode == 1) {
        for (int t = 0; t < T_tok; ++t) {
            if (pos[t] % DQO_WINDOW) continue;
            int w = pos[t] / DQO_WINDOW;
            for (int h = 0; h < Hkv; ++h) {
                size_t dst = ((size_t)seq_id[t] * Wmax + w) * Hkv + h;
                if (w == 0) { memset(mean_q + dst * n, 0, (size_t)n); mean_scale[dst] = 0.0f; }
                else {
                    size_t src = ((size_t)seq_id[t] * Wmax + (w - 1)) * Hkv + h;
                    memcpy(mean_q + dst * n, mean_q + src * n, (size_t)n);
                    mean_scale[dst] = mean_scale[src];
                }
            }
        }
        return;
    }
    int t0 = 0;
    while (t0 < T_tok) {
        int t1 = t0 + 1;
        while (t1 < T_tok && seq_id[t1] == seq_id[t0] &&
               pos[t1] / DQO_WINDOW == pos[t0] / DQO_WINDOW) ++t1;
        int w = pos[t0] / DQO_WINDOW;
        float inv = 1.0f / (float)(t1 - t0);
        for (int h = 0; h < Hkv; ++h) {
            float mu[DQO_MAX_N], acc[DQO_MAX_N], kt[DQO_MAX_N];
            for (int j = 0; j < n; ++j) acc[j] = 0.0f;
            for (int t = t0; t < t1; ++t) {   /* sequential binary32 sum over the run, per channel */
                for (int j = 0; j < n; ++j) kt[j] = dqo_bf16_to_f32(k_bf16[((size_t)t * Hkv + h) * n + j]);
                if (rope_style)
                    dqo_rope_f32(kt, n, rope_cos + (size_t)pos[t] * (n / 2), rope_sin + (size_t)pos[t] * (n / 2), rope_style);
                for (int j = 0; j < n; ++j) acc[j] = acc[j] + kt[j];
            }
            for (int j = 0; j < n; ++j) mu[j] = acc[j] * inv;
            if (rotate) dqo_fwht_f32(mu, n);
            size_t dst = ((size_t)seq_id[t0] * Wmax + w) * Hkv + h;
            dqo_quantise_mean(mu, n, mean_q + dst * n, mean_scale + dst);
        }
        t0 = t1;
    }
}

/* ------------------------------------------------------------ token encoder */

/* Streams per token and head dimension seen by the token-level entry points: a table with
 * n <= 128 has one stream per (token, KV head); n = hs * 128 has one stream per group of hs
 * consecutive KV heads (hs = Hkv: the whole token, the paper's default). */
static int dqo_heads_per_stream(const dqo_table *T) { return T->n > DQO_HEAD ? T->n / DQO_HEAD : 1; }
static int dqo_head_dim(const dqo_table *T) { return T->n > DQO_HEAD ? DQO_HEAD : T->n; }

/* containers are laid out [page, stream group, 16, rec] */
static size_t dqo_rec_offset(int slot, int grp, int groups, int rec)
{
    return (((size_t)(slot / DQO_PAGE) * groups + grp) * DQO_PAGE + (size_t)(slot % DQO_PAGE)) * rec;
}

/* Encode T_tok tokens of one tensor kind (Fig. 1 pipeline: Hadamard, mean removal
 * for keys, affine grid, drift, rANS).  x_bf16 is [T, Hkv, d]; each head is rotated (and,
 * for keys, centred on its window mean) on its own; the hs heads of a stream group are
 * concatenated in head order.  Containers are addressed by slot = page * 16 + index in page. */
void dqo_encode_tokens(const dqo_table *T, const uint16_t *x_bf16, int T_tok, int Hkv,
                       const int32_t *seq_id, const int32_t *pos, const int32_t *slot,
                       uint8_t *cont, const int8_t *mean_q, const float *mean_scale, int Wmax,
                       uint32_t *stats, const float *rope_cos, const float *rope_sin, int rope_style)
{
    int d = dqo_head_dim(T), hs = dqo_heads_per_stream(T), groups = Hkv / hs;
    uint32_t st[4] = {0, 0, 0, 0};
#pragma omp parallel
    {
        uint32_t lst[4] = {0, 0, 0, 0};
#pragma omp for schedule(static)
        for (int64_t tg = 0; tg < (int64_t)T_tok * groups; ++tg) {
            int t = (int)(tg / groups), grp = (int)(tg % groups);
            float z[DQO_MAX_N];
            for (int k = 0; k < hs; ++k) {
                int h = grp * hs + k;
                float *zh = z + k * d;
                for (int j = 0; j < d; ++j) zh[j] = dqo_bf16_to_f32(x_bf16[((size_t)t * Hkv + h) * d + j]);
                if (rope_style)   /* keys handed over before their rotary embedding */
                    dqo_rope_f32(zh, d, rope_cos + (size_t)pos[t] * (d / 2), rope_sin + (size_t)pos[t] * (d / 2), rope_style);
                if (T->rotate) dqo_fwht_f32(zh, d);
                if (T->has_mean) {
                    size_t mi = ((size_t)seq_id[t] * Wmax + pos[t] / DQO_WINDOW) * Hkv + h;
                    float sc = mean_scale[mi];
                    for (int j = 0; j < d; ++j) zh[j] = zh[j] - sc * (float)mean_q[mi * d + j];
                }
            }
            dqo_encode_stream(z, T, cont + dqo_rec_offset(slot[t], grp, groups, T->rec), lst, NULL);
        }
#pragma omp critical
        {
            st[0] += lst[0]; st[1] += lst[1]; st[2] += lst[2];
            if (lst[3] > st[3]) st[3] = lst[3];
        }
    }
    if (stats) {
        stats[0] += st[0]; stats[1] += st[1]; stats[2] += st[2];
        if (st[3] > stats[3]) stats[3] = st[3];
    }
}

/* ------------------------------------------------------------ token decoder */

/* Decode one record: all n symbols of the stream and (nullable) the dequantised values in
 * the rotated domain, xhat_j = fma(m_j, s, o), Appendix A (the key mean is added by the
 * callers, per head). */
static void dqo_decode_record(const dqo_table *T, const uint8_t *rec, uint8_t *sym, float *xhat)
{
    int n = T->n;
    uint16_t s16 = (uint16_t)(rec[0] | (rec[1] << 8)), o16 = (uint16_t)(rec[2] | (rec[3] << 8));
    float s = dqo_f16_to_f32(s16), o = dqo_f16_to_f32(o16);
    dqo_rans_decode(rec + 4, T->C, n, T, sym, NULL);
    if (!xhat) return;
    for (int j = 0; j < n; ++j) xhat[j] = fmaf((float)sym[j], s, o);
}

/* symbols / dequant are [T, Hkv, d] */
void dqo_decode_tokens(const dqo_table *T, const uint8_t *cont, const int8_t *mean_q,
                       const float *mean_scale, int Wmax, const int32_t *seq_id,
                       const int32_t *pos, const int32_t *slot, int T_tok, int Hkv,
                       uint8_t *symbols, float *dequant)
{
    int d = dqo_head_dim(T), hs = dqo_heads_per_stream(T), groups = Hkv / hs;
#pragma omp parallel for schedule(static)
    for (int64_t tg = 0; tg < (int64_t)T_tok * groups; ++tg) {
        int t = (int)(tg / groups), grp = (int)(tg % groups);
        uint8_t sym[DQO_MAX_N];
        float xh[DQO_MAX_N];
        dqo_decode_record(T, cont + dqo_rec_offset(slot[t], grp, groups, T->rec), sym, xh);
        for (int k = 0; k < hs; ++k) {
            int h = grp * hs + k;
            size_t dst = ((size_t)t * Hkv + h) * d;
            for (int j = 0; j < d; ++j) symbols[dst + j] = sym[k * d + j];
            if (!dequant) continue;
            if (T->has_mean && mean_q) {
                size_t mi = ((size_t)seq_id[t] * Wmax + pos[t] / DQO_WINDOW) * Hkv + h;
                float msc = mean_scale[mi];
                for (int j = 0; j < d; ++j)
                    dequant[dst + j] = xh[k * d + j] + msc * (float)mean_q[mi * d + j];
            } else
                for (int j = 0; j < d; ++j) dequant[dst + j] = xh[k * d + j];
        }
    }
}

/* ----------------------------------------------------------------- attention */

/* Decode-step attention in binary64 over the dequantised cache: for query head hq
 * and KV head g = hq / (Hq/Hkv): logits = sm_scale * <q', khat_t>, softmax over
 * t < seq_len, out' = sum a_t vhat_t; q' = Hq/sqrt(n) when keys are rotated and
 * out = H out'/sqrt(n) when values were rotated by the encoder.
 * Residual window (Sec. 5.1: the most recent tokens are kept in BF16): when resid_k is
 * given, sequence b has resid_lens[b] further tokens stored uncompressed and unrotated,
 * bf16 [B][resid_cap][Hkv][n]; they join the same softmax with logits sm_scale * <q, k_t>
 * and contribute a_t v_t to the (unrotated) output.
 * only_b/only_hq >= 0 restrict the work to one (b, hq) (others are left untouched). */
void dqo_attention(const dqo_table *TK, const dqo_table *TV, const uint16_t *q_bf16,
                   const uint8_t *k_cont, const uint8_t *v_cont, const int8_t *mean_q,
                   const float *mean_scale, int Wmax, const int32_t *page_table, int max_pages,
                   const int32_t *seq_lens, int B, int Hq, int Hkv, double sm_scale, double *out,
                   int only_b, int only_hq, const uint16_t *resid_k, const uint16_t *resid_v,
                   const int32_t *resid_lens, int resid_cap)
{
    int n = dqo_head_dim(TK), G = Hq / Hkv;   /* n: head dimension from here on */
    int hsk = dqo_heads_per_stream(TK), hsv = dqo_heads_per_stream(TV);
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
    for (int b = 0; b < B; ++b)
        for (int g = 0; g < Hkv; ++g) {
            if (only_b >= 0 && b != only_b) continue;
            if (only_hq >= 0 && only_hq / G != g) continue;
            int len = seq_lens[b] > 0 ? seq_lens[b] : 0;
            int rlen = (resid_k && resid_lens[b] > 0) ? resid_lens[b] : 0;
            if (len + rlen <= 0) {
                for (int hq = g * G; hq < (g + 1) * G; ++hq)
                    for (int j = 0; j < n; ++j) out[((size_t)b * Hq + hq) * n + j] = 0.0;
                continue;
            }
            float *kh = (float *)malloc((size_t)(len + 1) * n * sizeof(float));
            float *vh = (float *)malloc((size_t)(len + 1) * n * sizeof(float));
            double *lg = (double *)malloc((size_t)(len + rlen) * sizeof(double));
            uint8_t sym[DQO_MAX_N];
            float xh[DQO_MAX_N];
            for (int t = 0; t < len; ++t) {
                int slot = page_table[(size_t)b * max_pages + t / DQO_PAGE] * DQO_PAGE + t % DQO_PAGE;
                /* the stream that holds head g is decoded whole; head g's slice is kept */
                dqo_decode_record(TK, k_cont + dqo_rec_offset(slot, g / hsk, Hkv / hsk, TK->rec), sym, xh);
                for (int j = 0; j < n; ++j) kh[(size_t)t * n + j] = xh[(g % hsk) * n + j];
                if (TK->has_mean) {
                    size_t mi = ((size_t)b * Wmax + t / DQO_WINDOW) * Hkv + g;
                    float msc = mean_scale[mi];
                    for (int j = 0; j < n; ++j)
                        kh[(size_t)t * n + j] = kh[(size_t)t * n + j] + msc * (float)mean_q[mi * n + j];
                }
                dqo_decode_record(TV, v_cont + dqo_rec_offset(slot, g / hsv, Hkv / hsv, TV->rec), sym, xh);
                for (int j = 0; j < n; ++j) vh[(size_t)t * n + j] = xh[(g % hsv) * n + j];
            }
            for (int hq = g * G; hq < (g + 1) * G; ++hq) {
                if (only_hq >= 0 && hq != only_hq) continue;
                double qraw[DQO_MAX_N], qr[DQO_MAX_N], acc[DQO_MAX_N], racc[DQO_MAX_N];
                for (int j = 0; j < n; ++j)
                    qr[j] = qraw[j] = (double)dqo_bf16_to_f32(q_bf16[((size_t)b * Hq + hq) * n + j]);
                if (TK->rotate) dqo_fwht_f64(qr, n);
                double mxl = -INFINITY;
                for (int t = 0; t < len; ++t) {
                    double d = 0.0;
                    for (int j = 0; j < n; ++j) d += qr[j] * (double)kh[(size_t)t * n + j];
                    lg[t] = sm_scale * d;
                    if (lg[t] > mxl) mxl = lg[t];
                }
                for (int t = 0; t < rlen; ++t) {
                    const uint16_t *kr = resid_k + (((size_t)b * resid_cap + t) * Hkv + g) * n;
                    double d = 0.0;
                    for (int j = 0; j < n; ++j) d += qraw[j] * (double)dqo_bf16_to_f32(kr[j]);
                    lg[len + t] = sm_scale * d;
                    if (lg[len + t] > mxl) mxl = lg[len + t];
                }
                double den = 0.0;
                for (int j = 0; j < n; ++j) { acc[j] = 0.0; racc[j] = 0.0; }
                for (int t = 0; t < len; ++t) {
                    double a = exp(lg[t] - mxl);
                    den += a;
                    for (int j = 0; j < n; ++j) acc[j] += a * (double)vh[(size_t)t * n + j];
                }
                for (int t = 0; t < rlen; ++t) {
                    const uint16_t *vr = resid_v + (((size_t)b * resid_cap + t) * Hkv + g) * n;
                    double a = exp(lg[len + t] - mxl);
                    den += a;
                    for (int j = 0; j < n; ++j) racc[j] += a * (double)dqo_bf16_to_f32(vr[j]);
                }
                if (TV->rotate) dqo_fwht_f64(acc, n);   /* compressed part back to the unrotated domain */
                for (int j = 0; j < n; ++j) out[((size_t)b * Hq + hq) * n + j] = (acc[j] + racc[j]) / den;
            }
            free(kh); free(vh); free(lg);
        }
}

int dqo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
