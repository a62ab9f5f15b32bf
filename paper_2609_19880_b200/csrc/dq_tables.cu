// Host-side construction of the calibration-free rANS tables (Sec. 3.1 "Entropy Coding",
// Sec. 4.2 last paragraph, Sec. 4.4 "Distribution sharpening").  No device work.
#include <cuda_fp16.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "dq_internal.h"

namespace {

constexpr int kTotal = 256;  // 2^p, p = 8

inline double normal_cdf(double x) { return 0.5 * std::erfc(-x * M_SQRT1_2); }

// E[max of n iid standard normals] = integral of x n phi(x) Phi(x)^(n-1).  The integrand is
// analytic and vanishes to all orders at +-9, so the trapezoid rule converges geometrically.
double expected_maximum(int n) {
    const int nodes = 1 << 17;
    const double lo = -9.0, hi = 9.0, step = (hi - lo) / nodes;
    const double inv_sqrt_2pi = 0.3989422804014326779;
    double acc = 0.0;
    for (int i = 1; i < nodes; ++i) {
        const double x = lo + step * i;
        acc += x * std::exp(-0.5 * x * x) * std::pow(normal_cdf(x), n - 1);
    }
    return acc * step * n * inv_sqrt_2pi;
}

struct Model {
    std::vector<double> cell;  // analytic cell masses, normalised
};

Model cell_masses(int M, int n) {
    const double span = expected_maximum(n);
    const double width = 2.0 * span / (M - 1);
    Model mod;
    mod.cell.assign(M, 0.0);
    for (int m = 0; 2 * m < M + 1 && m < M; ++m) {
        const double centre = -span + width * m;
        const double left = std::max(-span, centre - 0.5 * width);
        const double right = std::min(span, centre + 0.5 * width);
        const double mass = normal_cdf(right) - normal_cdf(left);
        mod.cell[m] = mass;
        mod.cell[M - 1 - m] = mass;  // the model is symmetric
    }
    double total = 0.0;
    for (double v : mod.cell) total += v;
    for (double& v : mod.cell) v /= total;
    return mod;
}

// Sharpened model p' ~ p^alpha, normalised (Sec. 4.4).
std::vector<double> sharpened(const Model& mod, double alpha) {
    std::vector<double> q(mod.cell.size());
    double norm = 0.0;
    for (size_t m = 0; m < q.size(); ++m) norm += (q[m] = std::pow(mod.cell[m], alpha));
    for (double& v : q) v = v / norm;
    return q;
}

// Integer frequencies summing to 256 for targets 256 * probability: floor with a floor of 1, then
// largest remainders up (ties to the lowest index) or largest excesses down among f > 1 (ties to
// the highest index).
void integer_frequencies(const std::vector<double>& target, int32_t* f) {
    const int M = (int)target.size();
    int sum = 0;
    for (int m = 0; m < M; ++m) {
        f[m] = std::max(1, (int)std::floor(target[m]));
        sum += f[m];
    }
    for (; sum < kTotal; ++sum) {
        int pick = 0;
        for (int m = 1; m < M; ++m)
            if (target[m] - f[m] > target[pick] - f[pick]) pick = m;
        ++f[pick];
    }
    for (; sum > kTotal; --sum) {
        int pick = -1;
        for (int m = 0; m < M; ++m)
            if (f[m] > 1 && (pick < 0 || f[m] - target[m] >= f[pick] - target[pick])) pick = m;
        --f[pick];
    }
}

// Level table: 256 * q_m.  Pair table (paired-symbol variant): 256 * (q_a q_b), u = a M + b.
void level_frequencies(const Model& mod, double alpha, int32_t* f) {
    std::vector<double> target = sharpened(mod, alpha);
    for (double& v : target) v = kTotal * v;
    integer_frequencies(target, f);
}

void pair_frequencies(const Model& mod, double alpha, int32_t* f) {
    const std::vector<double> q = sharpened(mod, alpha);
    const int M = (int)q.size();
    std::vector<double> target((size_t)M * M);
    for (int a = 0; a < M; ++a)
        for (int b = 0; b < M; ++b) target[(size_t)a * M + b] = kTotal * (q[a] * q[b]);
    integer_frequencies(target, f);
}

// High byte of the binary16 pattern of a level 0..8 (their low byte is zero).
uint32_t level_code(int m) { return (uint32_t)__half_as_ushort(__float2half((float)m)) >> 8; }

// Pair alphabet: costs, most probable pair and the decode table
//   lut[z] = code(b) << 24 | f_u << 16 | code(a) << 8 | (z - c_u).
void finish_pairs(dq_table_info& t) {
    const int M = t.levels, K = M * M;
    t.ustar = 0;
    int c = 0;
    for (int u = 0; u < K; ++u) {
        const double bits = 8.0 - std::log2((double)t.pair_f[u]);
        t.pair_R[u] = (uint32_t)std::ceil(bits * 65536.0);
        if (t.pair_f[u] > t.pair_f[t.ustar]) t.ustar = u;
        for (int z = c; z < c + t.pair_f[u]; ++z)
            t.lut[z] = (level_code(u % M) << 24) | ((uint32_t)t.pair_f[u] << 16) | (level_code(u / M) << 8) | (uint32_t)(z - c);
        c += t.pair_f[u];
    }
}

void finish(dq_table_info& t) {
    t.c[0] = 0;
    t.mstar = 0;
    for (int m = 0; m < t.levels; ++m) {
        t.c[m + 1] = t.c[m] + t.f[m];
        const double bits = 8.0 - std::log2((double)t.f[m]);
        t.r[m] = (float)bits;
        t.R[m] = (uint32_t)std::ceil(bits * 65536.0);
        if (t.f[m] > t.f[t.mstar]) t.mstar = m;
    }
    for (int m = 0; m < t.levels; ++m) {
        const uint32_t level_bits = __half_as_ushort(__float2half((float)m));
        for (int z = t.c[m]; z < t.c[m + 1]; ++z)
            t.lut[z] = ((uint32_t)t.f[m] << 24) | (level_bits << 8) | (uint32_t)(z - t.c[m]);
    }
    if (t.pair_symbols) finish_pairs(t);
}

bool all_central_fits(const dq_table_info& t) {
    const int64_t n = (int64_t)t.head_dim * t.heads_per_stream;
    if (t.pair_symbols) return (n / 2) * t.pair_R[t.ustar] <= (int64_t)t.budget_bits * 65536;
    return n * t.R[t.mstar] <= (int64_t)t.budget_bits * 65536;
}

// bits per value
double table_entropy(const dq_table_info& t) {
    double h = 0.0;
    if (t.pair_symbols) {
        for (int u = 0; u < t.levels * t.levels; ++u) {
            const double p = t.pair_f[u] / (double)kTotal;
            h -= p * std::log2(p);
        }
        return 0.5 * h;
    }
    for (int m = 0; m < t.levels; ++m) {
        const double p = t.f[m] / (double)kTotal;
        h -= p * std::log2(p);
    }
    return h;
}

}  // namespace

int dq_host_build(int levels, double bits_per_elem, const dq_table_opts* opts, dq_tables* out) {
    if (!opts || !out) return DQ_ERR_ARG;
    if (opts->head_dim != DQ_HEAD_DIM) return DQ_ERR_UNSUPPORTED;
    if (levels < 2 || !(bits_per_elem > 0.0) || !std::isfinite(bits_per_elem)) return DQ_ERR_ARG;
    if (levels > DQ_MAX_LEVELS) return DQ_ERR_UNSUPPORTED;
    if (opts->heads_per_stream < 0 || opts->heads_per_stream > DQ_MAX_STREAM_HEADS) return DQ_ERR_UNSUPPORTED;
    const int hs = opts->heads_per_stream > 1 ? opts->heads_per_stream : 1;
    const int n = DQ_HEAD_DIM * hs;   // stream length: the model's n (Sec. 4.2, last paragraph)
    const double rec_d = std::floor(bits_per_elem * n / 8.0 + 1e-9);
    if (rec_d > (hs > 1 ? DQ_MAX_WIDE_REC_BYTES : DQ_MAX_REC_BYTES)) return DQ_ERR_UNSUPPORTED;
    const int rec = (int)rec_d;
    if (rec < 9) return DQ_ERR_INFEASIBLE;  // header alone is 8 bytes
    const int sigma = opts->sigma_bits == 0 ? 32 : opts->sigma_bits;
    if (sigma != 32 && sigma != 24) return DQ_ERR_ARG;
    if (sigma == 24 && hs > 1) return DQ_ERR_UNSUPPORTED;   // the short state is offered for 128-value streams
    const bool pair = opts->pair_symbols != 0;
    if (pair && levels > DQ_MAX_PAIR_LEVELS) return DQ_ERR_UNSUPPORTED;

    dq_table_info& t = out->info;
    std::memset(out, 0, sizeof *out);
    t.levels = levels;
    t.head_dim = DQ_HEAD_DIM;
    t.heads_per_stream = hs;
    t.rec_words = (rec + 3) / 4;
    t.rec_bytes = rec;
    t.container_bytes = rec - 4;              // Eq. (budget): C bytes hold state + payload
    t.budget_bits = 8 * t.container_bytes - sigma;  // B = 8C - sigma
    t.sigma_bits = sigma;
    t.drift_early_exit = opts->drift_early_exit ? 1 : 0;
    t.pair_symbols = pair ? 1 : 0;
    t.has_mean = opts->has_mean ? 1 : 0;
    t.rotate = opts->rotate ? 1 : 0;

    const Model mod = cell_masses(levels, n);
    bool ok = false;
    if (opts->alpha >= 0.0) {
        t.alpha = opts->alpha;
        level_frequencies(mod, t.alpha, t.f);
        if (pair) pair_frequencies(mod, t.alpha, t.pair_f);
        finish(t);
        ok = all_central_fits(t);
    } else {
        for (int tenth = 14; tenth <= 320 && !ok; ++tenth) {
            t.alpha = tenth / 10.0;
            level_frequencies(mod, t.alpha, t.f);
            if (pair) pair_frequencies(mod, t.alpha, t.pair_f);
            finish(t);
            ok = all_central_fits(t) && table_entropy(t) <= (double)t.budget_bits / n;
        }
    }
    if (!ok) return DQ_ERR_INFEASIBLE;

    DqDevTable& d = out->dev;
    d.M = levels;
    d.rec = rec;
    d.mstar = t.mstar;
    d.budget_bits = t.budget_bits;
    d.has_mean = t.has_mean;
    d.rotate = t.rotate;
    d.hs = hs;
    d.rec_words = t.rec_words;
    d.sigma = sigma;
    d.early_exit = t.drift_early_exit;
    d.pair = t.pair_symbols;
    d.ustar = t.ustar;
    // Enc(x, m) = floor(x / f) 2^p + x mod f + c = x + c + floor(x / f) (2^p - f); the quotient of a
    // 31-bit x by f comes from one high multiply with rcp = ceil(2^(31 + s) / f), s = ceil(log2 f),
    // followed by a shift of s - 1.  f = 1: rcp = 2^32 - 1 gives x - 1 and the bias absorbs it.
    auto enc_entry = [](uint32_t f, uint32_t c, uint32_t& rcp_out, uint32_t& aux_out) {
        uint32_t rcp = 0xffffffffu, rsh = 0, bias = c + 255u;
        if (f > 1) {
            uint32_t s = 0;
            while ((1u << s) < f) ++s;
            rcp = (uint32_t)((((uint64_t)1 << (s + 31)) + f - 1) / f);
            rsh = s - 1;
            bias = c;
        }
        rcp_out = rcp;
        aux_out = bias | ((256u - f) << 10) | (rsh << 19);
    };
    for (int m = 0; m < levels; ++m) {
        enc_entry((uint32_t)t.f[m], (uint32_t)t.c[m], d.enc_rcp[m], d.enc_aux[m]);
        d.r[m] = t.r[m];
        d.R[m] = t.R[m];
    }
    if (pair) {
        uint32_t c = 0;
        for (int u = 0; u < levels * levels; ++u) {
            enc_entry((uint32_t)t.pair_f[u], c, out->penc.enc_rcp[u], out->penc.enc_aux[u]);
            out->penc.r[u] = (float)(8.0 - std::log2((double)t.pair_f[u]));
            out->penc.R[u] = t.pair_R[u];
            c += (uint32_t)t.pair_f[u];
        }
    }
    std::memcpy(d.lut, t.lut, sizeof d.lut);
    return DQ_OK;
}
