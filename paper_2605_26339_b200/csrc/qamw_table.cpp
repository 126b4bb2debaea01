// Exact spatial search table for the 2-D nearest-codeword search (host side).
//
// Section 3.6 of the paper defines the quantiser as the Euclidean-nearest entry
// of the codebook.  An exhaustive scan of K = 2048 entries per pair would make
// the encoder ALU-bound by three orders of magnitude, so the device looks the
// pair up in a grid: every cell stores the complete list of codewords whose
// nearest-neighbour (Voronoi) region meets the cell, hence scanning the list
// gives the same answer as scanning the codebook.
//
// Geometry.  Each axis is cut into 4096 fine bins of width 1/256 over [-8, 8)
// (powers of two, so the device's fma(z, 256, 2048) is exact up to its final
// rounding); the first and last bin also take everything beyond (the device
// clamps the bin index), out to |z| < 16384.  A byte look-up table maps a fine
// bin to one of `grid` coarse columns.  Column boundaries sit on fine-bin
// edges: the inner ones near the quantiles of N(0, 2) -- the marginal of the
// high-rate optimal point density f^(1/2) of a unit circular Gaussian source,
// so that every inner cell holds about the same number of codewords -- followed
// by a few geometrically widening tail columns for heavy-tailed inputs.
//
// Construction.  The Voronoi polygon of every codeword (clipped to the square
// |z| <= 16384 and relaxed by a small slack, so it can only grow) is obtained by
// clipping that square with the bisector half-planes of all other codewords.
// A codeword is listed in a cell iff its polygon meets the cell's rectangle
// enlarged by a margin that covers the rounding of the device's bin computation.
#include <algorithm>
#include <cmath>
#include <cstring>

#include "qamw_internal.h"

namespace qamw {
namespace {

struct Pt {
    double x, y;
};

constexpr double kFar = 16384.0;  // the table covers |z| < kFar

// Sutherland-Hodgman step: keep the part of convex polygon `in` with a*x + b*y <= c.
void clip_halfplane(const std::vector<Pt>& in, double a, double b, double c, std::vector<Pt>* out) {
    out->clear();
    const size_t n = in.size();
    for (size_t i = 0; i < n; ++i) {
        const Pt& p = in[i];
        const Pt& q = in[(i + 1) % n];
        double fp = a * p.x + b * p.y - c;
        double fq = a * q.x + b * q.y - c;
        if (fp <= 0) out->push_back(p);
        if ((fp < 0 && fq > 0) || (fp > 0 && fq < 0)) {
            double t = fp / (fp - fq);
            out->push_back(Pt{p.x + t * (q.x - p.x), p.y + t * (q.y - p.y)});
        }
    }
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

// Voronoi polygon of codeword i inside [-kFar, kFar]^2, bisectors relaxed outwards by a slack.
void voronoi_polygon(const double* cb, int K, int i, std::vector<Pt>* poly, std::vector<Pt>* tmp) {
    const double cix = cb[2 * i], ciy = cb[2 * i + 1];
    const double ci2 = cix * cix + ciy * ciy;
    *poly = {Pt{-kFar, -kFar}, Pt{kFar, -kFar}, Pt{kFar, kFar}, Pt{-kFar, kFar}};
    double reach2 = 8.0 * kFar * kFar;  // upper bound of the squared distance from c_i to any vertex
    for (int j = 0; j < K; ++j) {
        if (j == i) continue;
        const double cjx = cb[2 * j], cjy = cb[2 * j + 1];
        const double ddx = cjx - cix, ddy = cjy - ciy;
        const double d2 = ddx * ddx + ddy * ddy;
        // the bisector lies at distance |cj - ci| / 2 from c_i: it cannot cut a polygon inside that radius
        if (d2 > 4.0 * reach2 * (1.0 + 1e-9)) continue;
        const double cj2 = cjx * cjx + cjy * cjy;
        const double slack = 1e-11 * (1.0 + ci2 + cj2);
        // |z-ci|^2 <= |z-cj|^2  <=>  2 z.(cj - ci) <= |cj|^2 - |ci|^2
        clip_halfplane(*poly, 2 * ddx, 2 * ddy, cj2 - ci2 + slack, tmp);
        if (tmp->size() != poly->size() || std::memcmp(tmp->data(), poly->data(), poly->size() * sizeof(Pt)) != 0) {
            poly->swap(*tmp);
            reach2 = 0.0;
            for (const Pt& p : *poly) {
                double ex = p.x - cix, ey = p.y - ciy;
                reach2 = std::max(reach2, ex * ex + ey * ey);
            }
        }
        if (poly->empty()) break;  // cannot happen for distinct codewords; duplicates end up empty
    }
}

}  // namespace

int default_grid(int K) {
    int g = int(std::ceil(2.1 * std::sqrt(double(K)) / 8.0)) * 8;
    return std::max(4, std::min(g, 192));
}

// Coarse boundaries in fine-bin units: edge[0] = 0 < ... < edge[grid] = kFineBins.
static std::vector<int> make_edges(int grid) {
    // number of widening tail columns per side (none for tiny grids)
    const int tails = grid >= 24 ? 3 : (grid >= 12 ? 1 : 0);
    const int core = grid - 2 * tails;
    std::vector<double> pos;  // boundaries for z > 0, in z units
    std::vector<double> inner;
    for (int i = 1; i < core; ++i) inner.push_back(quantile_n02(double(i) / double(core)));
    std::vector<double> all(inner);
    if (tails > 0 && core >= 2) {
        double last = inner.back();
        double w = core >= 3 ? (inner[inner.size() - 1] - inner[inner.size() - 2]) * 1.5 : 1.0;
        std::vector<double> up;
        double e = last;
        for (int t = 0; t < tails; ++t) {
            e += w;
            w *= 1.5;
            up.push_back(std::min(e, 7.9 - 0.1 * (tails - 1 - t)));
        }
        for (double u : up) all.push_back(u);
        for (double u : up) all.push_back(-u);
    }
    std::sort(all.begin(), all.end());
    std::vector<int> edge(static_cast<size_t>(grid + 1), 0);
    edge[0] = 0;
    edge[size_t(grid)] = kFineBins;
    for (int i = 1; i < grid; ++i) {
        double q = (size_t(i - 1) < all.size()) ? all[size_t(i - 1)] : 7.9;
        int e = int(std::lround(q * kFineScale + kFineOffset));
        e = std::max(e, edge[size_t(i - 1)] + 1);
        e = std::min(e, kFineBins - (grid - i));
        edge[size_t(i)] = e;
    }
    return edge;
}

bool build_cell_lists(const double* cb, int K, int grid, CellLists* out) {
    if (grid < 1 || grid > 255) return false;
    out->grid = grid;
    std::vector<int> edge = make_edges(grid);
    out->edges.resize(size_t(grid + 1));
    for (int i = 0; i <= grid; ++i) out->edges[size_t(i)] = (double(edge[size_t(i)]) - kFineOffset) / kFineScale;
    // the outermost columns also own everything beyond the fine range (the device clamps the bin)
    out->edges[0] = -kFar;
    out->edges[size_t(grid)] = kFar;
    out->lut.assign(size_t(kFineBins), 0);
    for (int i = 0; i < grid; ++i)
        for (int f = edge[size_t(i)]; f < edge[size_t(i + 1)]; ++f) out->lut[size_t(f)] = uint8_t(i);
    // 2^-10 of a fine bin covers the rounding of fma(z, 256, 2048) (at most 2^-12 of a bin)
    const double margin = 1.0 / (1024.0 * kFineScale);
    out->lists.assign(size_t(grid) * grid, {});
    std::vector<Pt> poly, tmp, a, b;
    auto column_of = [&](double z) {  // coarse column containing z (clamped like the device)
        double f = std::floor(z * kFineScale + kFineOffset);
        int fi = int(std::min(double(kFineBins - 1), std::max(0.0, f)));
        return int(out->lut[size_t(fi)]);
    };
    for (int i = 0; i < K; ++i) {
        voronoi_polygon(cb, K, i, &poly, &tmp);
        if (poly.empty()) continue;
        double bx0 = INFINITY, bx1 = -INFINITY, by0 = INFINITY, by1 = -INFINITY;
        for (const Pt& p : poly) {
            bx0 = std::min(bx0, p.x); bx1 = std::max(bx1, p.x);
            by0 = std::min(by0, p.y); by1 = std::max(by1, p.y);
        }
        const int ix0 = column_of(bx0 - 2 * margin), ix1 = column_of(bx1 + 2 * margin);
        const int iy0 = column_of(by0 - 2 * margin), iy1 = column_of(by1 + 2 * margin);
        for (int iy = iy0; iy <= iy1; ++iy)
            for (int ix = ix0; ix <= ix1; ++ix) {
                const double x0 = out->edges[size_t(ix)] - margin, x1 = out->edges[size_t(ix + 1)] + margin;
                const double y0 = out->edges[size_t(iy)] - margin, y1 = out->edges[size_t(iy + 1)] + margin;
                clip_halfplane(poly, -1, 0, -x0, &a);          // x >= x0
                if (a.empty()) continue;
                clip_halfplane(a, 1, 0, x1, &b);               // x <= x1
                if (b.empty()) continue;
                clip_halfplane(b, 0, -1, -y0, &a);             // y >= y0
                if (a.empty()) continue;
                clip_halfplane(a, 0, 1, y1, &b);               // y <= y1
                if (b.empty()) continue;
                out->lists[size_t(iy) * grid + ix].push_back(uint16_t(i));
            }
    }
    out->max_list = 0;
    out->n_candidates = 0;
    for (const auto& l : out->lists) {
        if (l.empty()) return false;  // every cell is met by at least one region
        out->max_list = std::max(out->max_list, int(l.size()));
        out->n_candidates += int(l.size());
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
        if (build_cell_lists(cb.data(), K, g, &cl) && pack_search_table(cl, &t) && t.bytes() <= budget_bytes) {
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
