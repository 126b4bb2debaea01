// Exact spatial search table for the 2-D nearest-codeword search (host side).
//
// Section 3.6 of the paper defines the quantiser as the Euclidean-nearest entry
// of the codebook.  An exhaustive scan of K = 2048 entries per pair would make
// the encoder ALU-bound by three orders of magnitude, so the device looks the
// pair up in a grid: every cell stores the complete list of codewords whose
// nearest-neighbour (Voronoi) region meets the cell, hence scanning the list
// gives the same answer as scanning the codebook.
//
// Geometry.  Each axis of [-8, 8) is cut into 4096 fine bins of width 1/256
// (powers of two, so the device's fma(z, 256, 2048) is exact up to its final
// rounding).  A byte look-up table maps a fine bin to one of `grid` coarse
// columns; column boundaries sit on fine-bin edges, near the quantiles of
// N(0, 2), which is the marginal of the high-rate optimal point density
// f^(1/2) of a unit circular Gaussian source -- so every coarse cell holds
// about the same number of codewords.  Points outside [-8, 8)^2 are not covered
// and are scanned exhaustively by the device.
//
// Construction for one cell Q (enlarged by a margin that covers the rounding of
// the device's f32 index computation):
//   1. U = min_i max_{z in Q} |z - c_i|^2.  Whatever z in Q is, its nearest
//      codeword is no farther than sqrt(U), so a codeword whose minimum
//      distance to Q exceeds U can never win inside Q.  This gives a superset A.
//   2. For every i in A the rectangle is clipped by the half-planes
//      |z - c_i|^2 <= |z - c_j|^2 (j in A, relaxed by a small slack); i stays
//      iff the clipped polygon is not empty, i.e. iff the region of i really
//      meets Q.  Competitors outside A cannot be nearest in Q, so clipping
//      against A alone is exact.
#include <algorithm>
#include <cmath>
#include <cstring>

#include "qamw_internal.h"

namespace qamw {
namespace {

struct Pt {
    double x, y;
};

// Sutherland-Hodgman step: keep the part of convex polygon `in` with a*x + b*y <= c.
int clip_halfplane(const Pt* in, int n, double a, double b, double c, Pt* out) {
    int m = 0;
    for (int i = 0; i < n; ++i) {
        const Pt& p = in[i];
        const Pt& q = in[(i + 1) % n];
        double fp = a * p.x + b * p.y - c;
        double fq = a * q.x + b * q.y - c;
        if (fp <= 0) out[m++] = p;
        if ((fp < 0 && fq > 0) || (fp > 0 && fq < 0)) {
            double t = fp / (fp - fq);
            out[m++] = Pt{p.x + t * (q.x - p.x), p.y + t * (q.y - p.y)};
        }
    }
    return m;
}

// Quantile of N(0, 2) by bisection on its CDF (1 + erf(x/2))/2; only used to place cell
// boundaries, so its accuracy does not affect exactness.
double quantile_n02(double p) {
    double lo = -16.0, hi = 16.0;
    for (int it = 0; it < 80; ++it) {
        double mid = 0.5 * (lo + hi);
        if (0.5 * (1.0 + std::erf(0.5 * mid)) < p) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

}  // namespace

static void rect_candidates_rec(const double* cb, int K, double x0, double x1, double y0, double y1, bool refine,
                                int depth, std::vector<uint16_t>* out, std::vector<double>* scratch) {
    out->clear();
    scratch->resize(size_t(K));
    double U = INFINITY;
    for (int i = 0; i < K; ++i) {
        double cx = cb[2 * i], cy = cb[2 * i + 1];
        double fx = std::max(std::fabs(cx - x0), std::fabs(cx - x1));
        double fy = std::max(std::fabs(cy - y0), std::fabs(cy - y1));
        double dmax2 = fx * fx + fy * fy;
        if (dmax2 < U) U = dmax2;
        double nx = cx < x0 ? x0 - cx : (cx > x1 ? cx - x1 : 0.0);
        double ny = cy < y0 ? y0 - cy : (cy > y1 ? cy - y1 : 0.0);
        (*scratch)[size_t(i)] = nx * nx + ny * ny;
    }
    const double lim = U * (1.0 + 1e-12) + 1e-300;
    std::vector<uint16_t> A;
    for (int i = 0; i < K; ++i)
        if ((*scratch)[size_t(i)] <= lim) A.push_back(uint16_t(i));
    if (!refine || A.size() <= 1) {
        *out = A;
        return;
    }
    if (A.size() > 24 && depth < 6) {
        // A large rectangle makes bound 1 loose: cover it by its four quadrants instead and
        // take the union (a region meets the rectangle iff it meets one of the quadrants).
        double xm = 0.5 * (x0 + x1), ym = 0.5 * (y0 + y1);
        std::vector<uint16_t> part, all;
        const double qx[2][2] = {{x0, xm}, {xm, x1}}, qy[2][2] = {{y0, ym}, {ym, y1}};
        for (int a = 0; a < 2; ++a)
            for (int b = 0; b < 2; ++b) {
                rect_candidates_rec(cb, K, qx[a][0], qx[a][1], qy[b][0], qy[b][1], true, depth + 1, &part, scratch);
                all.insert(all.end(), part.begin(), part.end());
            }
        std::sort(all.begin(), all.end());
        all.erase(std::unique(all.begin(), all.end()), all.end());
        *out = all;
        return;
    }
    Pt poly[2][72];
    for (uint16_t i : A) {
        double cix = cb[2 * i], ciy = cb[2 * i + 1];
        double ci2 = cix * cix + ciy * ciy;
        int cur = 0, n = 4;
        poly[0][0] = Pt{x0, y0};
        poly[0][1] = Pt{x1, y0};
        poly[0][2] = Pt{x1, y1};
        poly[0][3] = Pt{x0, y1};
        for (uint16_t j : A) {
            if (j == i) continue;
            double cjx = cb[2 * j], cjy = cb[2 * j + 1];
            double cj2 = cjx * cjx + cjy * cjy;
            // |z-ci|^2 <= |z-cj|^2  <=>  2 z.(cj - ci) <= |cj|^2 - |ci|^2
            double slack = 1e-11 * (1.0 + ci2 + cj2);
            n = clip_halfplane(poly[cur], n, 2 * (cjx - cix), 2 * (cjy - ciy), cj2 - ci2 + slack, poly[cur ^ 1]);
            cur ^= 1;
            if (n == 0 || n > 64) break;  // n > 64 cannot happen for a convex clip; kept as a guard
        }
        if (n != 0) out->push_back(i);
    }
}

void rect_candidates(const double* cb, int K, double x0, double x1, double y0, double y1, bool refine,
                     std::vector<uint16_t>* out, std::vector<double>* scratch) {
    rect_candidates_rec(cb, K, x0, x1, y0, y1, refine, 0, out, scratch);
}

int default_grid(int K) {
    int g = int(std::ceil(2.1 * std::sqrt(double(K)) / 8.0)) * 8;
    return std::max(4, std::min(g, 192));
}

bool build_cell_lists(const double* cb, int K, int grid, bool refine, CellLists* out) {
    if (grid < 1 || grid > 255) return false;
    out->grid = grid;
    // coarse boundaries (in fine-bin units) near the quantiles of N(0, 2), strictly increasing
    std::vector<int> edge(static_cast<size_t>(grid + 1), 0);
    edge[0] = 0;
    edge[size_t(grid)] = kFineBins;
    for (int i = 1; i < grid; ++i) {
        double q = quantile_n02(double(i) / double(grid));
        int e = int(std::lround(q * kFineScale + kFineOffset));
        e = std::max(e, edge[size_t(i - 1)] + 1);
        e = std::min(e, kFineBins - (grid - i));
        edge[size_t(i)] = e;
    }
    out->edges.resize(size_t(grid + 1));
    for (int i = 0; i <= grid; ++i) out->edges[size_t(i)] = (double(edge[size_t(i)]) - kFineOffset) / kFineScale;
    out->lut.assign(size_t(kFineBins), 0);
    for (int i = 0; i < grid; ++i)
        for (int f = edge[size_t(i)]; f < edge[size_t(i + 1)]; ++f) out->lut[size_t(f)] = uint8_t(i);
    // 2^-10 of a fine bin covers the rounding of fma(z, 256, 2048) (at most 2^-12 of a bin)
    const double margin = 1.0 / (1024.0 * kFineScale);
    out->lists.assign(size_t(grid) * grid, {});
    out->max_list = 0;
    out->n_candidates = 0;
    std::vector<double> scratch;
    for (int iy = 0; iy < grid; ++iy)
        for (int ix = 0; ix < grid; ++ix) {
            auto& list = out->lists[size_t(iy) * grid + ix];
            rect_candidates(cb, K, out->edges[size_t(ix)] - margin, out->edges[size_t(ix + 1)] + margin,
                            out->edges[size_t(iy)] - margin, out->edges[size_t(iy + 1)] + margin, refine, &list,
                            &scratch);
            out->max_list = std::max(out->max_list, int(list.size()));
            out->n_candidates += int(list.size());
        }
    return true;
}

// Device layout: one 8-byte record per cell holding up to four candidate indices in
// ascending order (the last one repeated as padding).  A cell with more candidates
// stores {0xFFFF, offset, count, 0} and its list goes to the overflow array.
bool pack_search_table(const CellLists& cl, SearchTable* out) {
    out->grid = cl.grid;
    out->lut = cl.lut;
    out->cells.assign(size_t(cl.grid) * cl.grid * 4, 0);
    out->overflow.clear();
    out->n_overflow_cells = 0;
    out->max_list = cl.max_list;
    out->n_candidates = cl.n_candidates;
    for (size_t c = 0; c < cl.lists.size(); ++c) {
        const auto& list = cl.lists[c];
        uint16_t* rec = &out->cells[c * 4];
        if (list.empty()) return false;
        if (list.size() <= 4) {
            for (size_t t = 0; t < 4; ++t) rec[t] = list[std::min(t, list.size() - 1)];
        } else {
            if (out->overflow.size() + list.size() > 0xFFFF) return false;
            rec[0] = 0xFFFF;
            rec[1] = uint16_t(out->overflow.size());
            rec[2] = uint16_t(list.size());
            rec[3] = 0;
            out->overflow.insert(out->overflow.end(), list.begin(), list.end());
            ++out->n_overflow_cells;
        }
    }
    while (out->overflow.size() % 8) out->overflow.push_back(0);  // keeps the next array 16-byte aligned
    return true;
}

bool choose_search_table(const float* codebook, int K, int grid, size_t budget_bytes, SearchTable* out) {
    std::vector<double> cb(static_cast<size_t>(2 * K), 0.0);
    for (int i = 0; i < 2 * K; ++i) cb[size_t(i)] = double(codebook[i]);
    int g = grid > 0 ? grid : default_grid(K);
    for (; g >= 1; g = (grid > 0 || g <= 8) ? g - 1 : g - 8) {
        if (size_t(g) * g * 8 + kFineBins > budget_bytes) {
            if (grid > 0) return false;
            continue;
        }
        CellLists cl;
        SearchTable t;
        if (build_cell_lists(cb.data(), K, g, true, &cl) && pack_search_table(cl, &t) && t.bytes() <= budget_bytes) {
            *out = std::move(t);
            return true;
        }
        if (grid > 0) return false;
    }
    return false;
}

}  // namespace qamw

using namespace qamw;

extern "C" int qamw_search_table_build(const float* codebook_host, int K, int grid, size_t budget_bytes,
                                       uint8_t* lut_out, uint16_t* cells_out, size_t cells_cap,
                                       uint16_t* overflow_out, size_t overflow_cap, int32_t* info_out) {
    if (!codebook_host || !info_out) return QAMW_ERR_ARG;
    if (K < 1 || K > QAMW_MAX_K || !is_pow2(K)) return QAMW_ERR_SHAPE;
    SearchTable t;
    if (!choose_search_table(codebook_host, K, grid, budget_bytes, &t)) return QAMW_ERR_NOMEM;
    info_out[0] = t.grid;
    info_out[1] = t.n_candidates;
    info_out[2] = t.max_list;
    info_out[3] = t.n_overflow_cells;
    info_out[4] = int32_t(t.overflow.size());
    info_out[5] = int32_t(t.bytes());
    if (lut_out) std::memcpy(lut_out, t.lut.data(), t.lut.size());
    if (cells_out) {
        if (cells_cap < t.cells.size()) return QAMW_ERR_NOMEM;
        std::memcpy(cells_out, t.cells.data(), t.cells.size() * 2);
    }
    if (overflow_out) {
        if (overflow_cap < t.overflow.size()) return QAMW_ERR_NOMEM;
        std::memcpy(overflow_out, t.overflow.data(), t.overflow.size() * 2);
    }
    return QAMW_OK;
}
