// Host-side entry points of libqamw: codebook training, channel scales, sign
// mask and the small closed-form helpers.  No CUDA calls in this file.
#include <algorithm>
#include <cfloat>
#include <cmath>
#include <cstring>
#include <thread>
#include <vector>

#include "qamw_internal.h"

using namespace qamw;

namespace {

// SplitMix64 finaliser (Steele, Lea, Flood 2014).
inline uint64_t mix64(uint64_t x) {
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ULL;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBULL;
    x ^= x >> 31;
    return x;
}

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ULL;

inline double uniform01(uint64_t stream_key, uint64_t n) {
    uint64_t h = mix64(stream_key + kGolden * (n + 1));
    return (double(h >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

// Unit circular Gaussian samples by Box-Muller, sample i from counters 2i and 2i+1.
void gaussian_pairs(uint64_t seed, uint64_t begin, uint64_t end, double* out) {
    const uint64_t key = mix64(seed ^ 0xD1B54A32D192ED03ULL);
    const double two_pi = 6.283185307179586476925286766559;
    for (uint64_t i = begin; i < end; ++i) {
        double u1 = uniform01(key, 2 * i), u2 = uniform01(key, 2 * i + 1);
        double rad = std::sqrt(-2.0 * std::log(u1));
        out[2 * i] = rad * std::cos(two_pi * u2);
        out[2 * i + 1] = rad * std::sin(two_pi * u2);
    }
}

template <class F>
void parallel_chunks(int n_chunks, F&& body) {
    unsigned hw = std::thread::hardware_concurrency();
    int n_threads = int(std::min<unsigned>(hw ? hw : 1u, unsigned(n_chunks)));
    if (n_threads <= 1) {
        for (int c = 0; c < n_chunks; ++c) body(c);
        return;
    }
    std::vector<std::thread> pool;
    for (int t = 0; t < n_threads; ++t)
        pool.emplace_back([&, t] {
            for (int c = t; c < n_chunks; c += n_threads) body(c);
        });
    for (auto& th : pool) th.join();
}

// One Lloyd assignment pass, exact nearest codeword (lowest index on ties), through a coarse
// grid of exact candidate lists; points outside the grid are scanned exhaustively.
// Samples are processed in kChunks fixed chunks so that the sums do not depend on the number
// of worker threads.
constexpr int kChunks = 64;

double assign_pass(const std::vector<double>& samples, uint64_t n, const std::vector<double>& cb, int K,
                   std::vector<double>* sums /* kChunks*K*2 or null */, std::vector<int64_t>* counts /* kChunks*K */) {
    CellLists cells;
    int grid = std::max(3, (default_grid(K) / 4) * 2 + 1);
    bool ok = build_cell_lists(cb.data(), K, grid, &cells);
    auto column_of = [&](double z) {  // a point near a boundary may get either neighbour: both lists hold its answer
        const int c = cells.map.half + int(std::lround(cell_map_value(cells.map, z)));
        return size_t(std::min(grid - 1, std::max(0, c)));
    };
    std::vector<double> chunk_err(kChunks, 0.0);
    if (sums) std::fill(sums->begin(), sums->end(), 0.0);
    if (counts) std::fill(counts->begin(), counts->end(), int64_t(0));
    parallel_chunks(kChunks, [&](int c) {
        uint64_t lo = n * uint64_t(c) / kChunks, hi = n * uint64_t(c + 1) / kChunks;
        double err = 0.0;
        double* s = sums ? sums->data() + size_t(c) * K * 2 : nullptr;
        int64_t* cnt = counts ? counts->data() + size_t(c) * K : nullptr;
        for (uint64_t i = lo; i < hi; ++i) {
            double zx = samples[2 * i], zy = samples[2 * i + 1];
            double best = INFINITY;
            int arg = 0;
            auto consider = [&](int k) {
                double dx = zx - cb[2 * size_t(k)], dy = zy - cb[2 * size_t(k) + 1];
                double d = dx * dx + dy * dy;
                if (d < best) {
                    best = d;
                    arg = k;
                }
            };
            if (ok && std::fabs(zx) < 16000.0 && std::fabs(zy) < 16000.0) {
                const auto& list = cells.lists[column_of(zy) * grid + column_of(zx)];
                for (uint16_t k : list) consider(int(k));
            } else {
                for (int k = 0; k < K; ++k) consider(k);
            }
            err += best;
            if (s) {
                s[2 * arg] += zx;
                s[2 * arg + 1] += zy;
                cnt[arg]++;
            }
        }
        chunk_err[size_t(c)] = err;
    });
    double total = 0.0;
    for (double e : chunk_err) total += e;
    return total / double(n);
}

}  // namespace

extern "C" int qamw_train_codebook(int K, uint64_t n_samples, uint64_t seed, int max_iters, double rel_tol,
                                   float* codebook_out, double* train_mse_out) {
    if (!codebook_out) return QAMW_ERR_ARG;
    if (K < 1 || K > QAMW_MAX_K || !is_pow2(K)) return QAMW_ERR_SHAPE;
    if (n_samples < uint64_t(K) || max_iters < 0 || !(rel_tol >= 0.0)) return QAMW_ERR_ARG;
    std::vector<double> samples(static_cast<size_t>(2 * n_samples), 0.0);
    parallel_chunks(kChunks, [&](int c) {
        gaussian_pairs(seed, n_samples * uint64_t(c) / kChunks, n_samples * uint64_t(c + 1) / kChunks, samples.data());
    });
    std::vector<double> cb(static_cast<size_t>(2 * K), 0.0);
    const double root2 = 1.4142135623730950488016887242097;
    for (int c = 0; c < 2 * K; ++c) cb[size_t(c)] = root2 * samples[size_t(c)];
    std::vector<double> sums(static_cast<size_t>(kChunks) * K * 2, 0.0);
    std::vector<int64_t> counts(static_cast<size_t>(kChunks) * K, 0);
    double prev = INFINITY;
    int updates = 0, t = 0;
    for (;;) {
        double D = assign_pass(samples, n_samples, cb, K, &sums, &counts);
        ++t;
        if (t > 1 && prev - D <= rel_tol * prev) break;
        if (updates >= max_iters) break;
        for (int k = 0; k < K; ++k) {
            double sx = 0, sy = 0;
            int64_t cnt = 0;
            for (int c = 0; c < kChunks; ++c) {
                sx += sums[(size_t(c) * K + k) * 2];
                sy += sums[(size_t(c) * K + k) * 2 + 1];
                cnt += counts[size_t(c) * K + k];
            }
            if (cnt > 0) {
                cb[2 * size_t(k)] = sx / double(cnt);
                cb[2 * size_t(k) + 1] = sy / double(cnt);
            }
        }
        ++updates;
        prev = D;
    }
    // order by (squared radius, angle) so that indices are reproducible
    std::vector<int> order(static_cast<size_t>(K), 0);
    for (int k = 0; k < K; ++k) order[size_t(k)] = k;
    auto r2 = [&](int k) { return cb[2 * size_t(k)] * cb[2 * size_t(k)] + cb[2 * size_t(k) + 1] * cb[2 * size_t(k) + 1]; };
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        double ra = r2(a), rb = r2(b);
        if (ra != rb) return ra < rb;
        return std::atan2(cb[2 * size_t(a) + 1], cb[2 * size_t(a)]) < std::atan2(cb[2 * size_t(b) + 1], cb[2 * size_t(b)]);
    });
    for (int k = 0; k < K; ++k) {
        codebook_out[2 * k] = float(cb[2 * size_t(order[size_t(k)])]);
        codebook_out[2 * k + 1] = float(cb[2 * size_t(order[size_t(k)]) + 1]);
    }
    if (train_mse_out) {
        for (int c = 0; c < 2 * K; ++c) cb[size_t(c)] = double(codebook_out[c]);
        *train_mse_out = assign_pass(samples, n_samples, cb, K, nullptr, nullptr);
    }
    return QAMW_OK;
}

extern "C" int qamw_channel_scales(const float* act_rms, int d_in, float alpha, float* s_out) {
    if (!act_rms || !s_out || d_in <= 0) return QAMW_ERR_ARG;
    std::vector<double> t(static_cast<size_t>(d_in), 0.0);
    double mean_t = 0.0;
    for (int j = 0; j < d_in; ++j) {
        double r = double(act_rms[j]);
        if (!(r > double(FLT_MIN))) r = double(FLT_MIN);
        t[size_t(j)] = double(alpha) * std::log(r);
        mean_t += t[size_t(j)];
    }
    mean_t /= double(d_in);
    for (int j = 0; j < d_in; ++j) {
        double s = std::exp(t[size_t(j)] - mean_t);
        s = std::min(16.0, std::max(1.0 / 16.0, s));
        s_out[j] = float(s);
    }
    return QAMW_OK;
}

extern "C" int qamw_make_signs(uint64_t seed, int d_in, int8_t* signs_out) {
    if (!signs_out || d_in <= 0) return QAMW_ERR_ARG;
    for (int j = 0; j < d_in; ++j) signs_out[j] = (mix64(seed + kGolden * uint64_t(j + 1)) >> 63) ? int8_t(-1) : int8_t(1);
    return QAMW_OK;
}

extern "C" int qamw_block_size_rule(int d_in) {
    if (d_in <= 0) return 0;
    int b = 1;
    while (b < QAMW_MAX_BLOCK && d_in % (2 * b) == 0) b *= 2;
    return b;
}

extern "C" size_t qamw_packed_row_bytes(int d_in, int K) {
    if (d_in <= 0 || d_in % 2 || K < 1 || !is_pow2(K)) return 0;
    return (size_t(d_in / 2) * size_t(ilog2(K)) + 7) / 8;
}

extern "C" double qamw_bpw(int d_out, int d_in, int K, int has_channel_scales) {
    if (d_out <= 0 || d_in <= 0 || K < 1) return 0.0;
    double bpw = 0.5 * ilog2(K) + 16.0 / d_in;
    if (has_channel_scales) bpw += 16.0 / d_out;
    return bpw;
}

extern "C" int qamw_status_to_error(int32_t status_word) {
    return (status_word & 1) ? QAMW_ERR_NONFINITE : QAMW_OK;
}

// ---------------------------------------------------------------------------------------------
// polar baseline (Section 3.5): amplitude levels and the table of reconstruction points
// ---------------------------------------------------------------------------------------------
namespace {
constexpr double kRayleighCutoff = 8.0;  // integration cut-off of the remark after the polar distortion corollary

// Moments int_a^b r^q f(r) dr, q = 0, 1, 2, of the unit Rayleigh density f(r) = r exp(-r^2/2), in
// closed form (antiderivatives -e, -r e + sqrt(pi/2) erf(r/sqrt 2), -(r^2 + 2) e with e = exp(-r^2/2)).
void rayleigh_moments(double a, double b, double m[3]) {
    const double ea = std::exp(-0.5 * a * a), eb = std::exp(-0.5 * b * b);
    const double root = 1.2533141373155002512078826424055;  // sqrt(pi / 2)
    m[0] = ea - eb;
    m[1] = a * ea - b * eb + root * (std::erf(b / 1.4142135623730950488) - std::erf(a / 1.4142135623730950488));
    m[2] = (a * a + 2.0) * ea - (b * b + 2.0) * eb;
}

double rayleigh_distortion(const std::vector<double>& l) {
    const int n = int(l.size());
    double D = 0.0;
    for (int j = 0; j < n; ++j) {
        const double lo = j == 0 ? 0.0 : 0.5 * (l[j - 1] + l[j]);
        const double hi = j == n - 1 ? kRayleighCutoff : 0.5 * (l[j] + l[j + 1]);
        double m[3];
        rayleigh_moments(lo, hi, m);
        D += m[2] - 2.0 * l[j] * m[1] + l[j] * l[j] * m[0];
    }
    return D;
}
}  // namespace

extern "C" int qamw_polar_train(int Ba, float* levels_out, double* c_lm_out) {
    if (!levels_out) return QAMW_ERR_ARG;
    if (Ba < 0 || Ba > 12) return QAMW_ERR_SHAPE;
    const int n = 1 << Ba;
    std::vector<double> l(n), next(n);
    for (int j = 0; j < n; ++j) l[j] = std::sqrt(-2.0 * std::log(1.0 - (j + 0.5) / n));  // quantiles of the law
    for (int it = 0; it < 200000; ++it) {
        double move = 0.0;
        for (int j = 0; j < n; ++j) {
            const double lo = j == 0 ? 0.0 : 0.5 * (l[j - 1] + l[j]);
            const double hi = j == n - 1 ? kRayleighCutoff : 0.5 * (l[j] + l[j + 1]);
            double m[3];
            rayleigh_moments(lo, hi, m);
            next[j] = m[0] > 0.0 ? m[1] / m[0] : l[j];
            move = std::max(move, std::fabs(next[j] - l[j]));
        }
        l.swap(next);
        if (move < 1e-13) break;
    }
    for (int j = 0; j < n; ++j) {
        levels_out[j] = float(l[j]);
        l[j] = double(levels_out[j]);
    }
    if (c_lm_out) *c_lm_out = rayleigh_distortion(l);
    return QAMW_OK;
}

extern "C" int qamw_polar_codebook(const float* levels, int Ba, int Bp, float* codebook_out) {
    if (!levels || !codebook_out) return QAMW_ERR_ARG;
    if (Ba < 0 || Bp < 0 || Ba + Bp < 1 || (1 << (Ba + Bp)) > QAMW_MAX_K) return QAMW_ERR_SHAPE;
    const double pi = 3.14159265358979323846264338327950288;
    const int Na = 1 << Ba, Np = 1 << Bp;
    for (int p = 0; p < Np; ++p) {
        const double phi = (2.0 * p + 1.0) * pi / double(Np);  // bin centres at odd multiples of pi / N_p
        for (int a = 0; a < Na; ++a) {
            const int idx = (p << Ba) | a;
            codebook_out[2 * idx] = float(double(levels[a]) * std::cos(phi));
            codebook_out[2 * idx + 1] = float(double(levels[a]) * std::sin(phi));
        }
    }
    return QAMW_OK;
}
