// Exact spatial search table for the 2-D nearest-codeword search (host side).
//
// Section 3.6 of the paper defines the quantiser as the Euclidean-nearest entry
// of the codebook.  An exhaustive scan of K = 2048 entries per pair would make
// the encoder ALU-bound by three orders of magnitude, so the device looks the
// pair up in a grid: every cell stores the complete list of codewords whose
// nearest-neighbour (Voronoi) region meets the cell, hence scanning the list
// gives the same answer as scanning the codebook.
//
// Geometry.  Both axes use the same map from a coordinate to a column, an odd
// polynomial followed by rounding to the nearest integer (CellMap in
// qamw_internal.h).  Its slope a (1 - z^2 / T)^2 follows the high-rate optimal
// point density f^(1/2) of a unit circular Gaussian source closely enough that
// the inner cells hold about the same number of codewords each, while the
// device pays three fused multiply-adds per axis instead of a table look-up.
// The coordinate is clamped to +-zmax first, so the outermost columns also take
// everything beyond, out to |z| < 16384.
//
// Construction.  The Voronoi polygon of every codeword (clipped to the square
// |z| <= 16384 and relaxed by a small slack, so it can only grow) is obtained by
// clipping that square with the bisector half-planes of all other codewords.
// A codeword is listed in a cell iff its polygon meets the cell's rectangle
// enlarged by a margin that covers the rounding of the device's f32 evaluation.
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
    // about 2.2 sqrt(K) columns, and never fewer than 31: a small table is cheap, and with fewer
    // columns the outermost ones are crowded enough to overflow
    const int half = std::max(15, std::min(int(std::lround(1.08 * std::sqrt(double(K)))), 127));
    return 2 * half + 1;
}

// Slope a ((1 - t / T)^2 + eps), t = z^2: the value a z (1 + eps - 2 t / (3 T) + t^2 / (5 T^2)) is
// increasing everywhere.  Up to sqrt(T) the cells widen like the spacing of the codewords of a
// Gaussian source; between sqrt(T) and zmax = rho sqrt(T) the slope rises again, which spends a few
// columns on the far tail, where heavy-tailed inputs (outlier channels) put many of their pairs.
// `a` makes the value at zmax half + 0.4, so the rounded value stays within +-half.
CellMap make_cell_map(int grid, const MapShape& shape) {
    CellMap m;
    m.grid = grid;
    m.half = (grid - 1) / 2;
    const double T = shape.T, zmax = shape.rho * std::sqrt(T), t = zmax * zmax;
    const double a = (double(m.half) + 0.4) / (zmax * (1.0 + shape.eps - 2.0 * t / (3.0 * T) + t * t / (5.0 * T * T)));
    m.c0 = float(a * (1.0 + shape.eps));
    m.c1 = float(-2.0 * a / (3.0 * T));
    m.c2 = float(a / (5.0 * T * T));
    m.zmax = float(zmax);
    return m;
}

double cell_map_value(const CellMap& m, double z) {
    const double c = std::min(std::max(z, -double(m.zmax)), double(m.zmax));
    const double t = c * c;
    return c * (double(m.c0) + t * (double(m.c1) + t * double(m.c2)));
}

namespace {
// Smallest z in [-zmax, zmax] with cell_map_value(z) >= v (the map is increasing there).
double cell_map_inverse(const CellMap& m, double v) {
    double lo = -double(m.zmax), hi = double(m.zmax);
    if (cell_map_value(m, lo) >= v) return lo;
    if (cell_map_value(m, hi) < v) return hi;
    for (int it = 0; it < 100; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (cell_map_value(m, mid) < v) lo = mid; else hi = mid;
    }
    return hi;
}

double normal_cdf(double x, double sd) { return 0.5 * std::erfc(-x / (sd * std::sqrt(2.0))); }
}  // namespace

void voronoi_polygons(const double* cb, int K, VoronoiSet* out) {
    out->start.assign(size_t(K) + 1, 0);
    out->xy.clear();
    std::vector<Pt> poly, tmp;
    for (int i = 0; i < K; ++i) {
        voronoi_polygon(cb, K, i, &poly, &tmp);
        for (const Pt& p : poly) {
            out->xy.push_back(p.x);
            out->xy.push_back(p.y);
        }
        out->start[size_t(i) + 1] = int(out->xy.size() / 2);
    }
}

bool build_cell_lists(const VoronoiSet& vs, int K, const CellMap& m, CellLists* out) {
    const int grid = m.grid;
    if (grid < 1 || grid > 255 || grid % 2 == 0) return false;
    out->map = m;
    {   // the map must be increasing on [-zmax, zmax] and stay inside +-(half + 0.45)
        double prev = cell_map_value(m, 0.0);
        for (int i = 1; i <= 4096; ++i) {
            const double v = cell_map_value(m, double(m.zmax) * i / 4096.0);
            if (!(v > prev)) return false;
            prev = v;
        }
        if (!(prev < double(m.half) + 0.45)) return false;
    }
    // The device's f32 evaluation differs from the exact map by a few units of 2^-24 * half; a margin
    // of 2^-8 of a column, on both sides of every boundary, covers it (and the tie rule of the
    // rounding) many times over.
    const double du = 1.0 / 256.0;
    out->lo.assign(size_t(grid), 0.0);
    out->hi.assign(size_t(grid), 0.0);
    for (int j = 0; j < grid; ++j) {
        const double v = double(j - m.half);
        out->lo[size_t(j)] = j == 0 ? -kFar : cell_map_inverse(m, v - 0.5 - du);
        out->hi[size_t(j)] = j == grid - 1 ? kFar : cell_map_inverse(m, v + 0.5 + du);
    }
    out->lists.assign(size_t(grid) * grid, {});
    std::vector<Pt> poly, a, b;
    auto column_of = [&](double z) {  // exact map; callers widen the range by one column
        const int c = m.half + int(std::lround(cell_map_value(m, z)));
        return std::min(grid - 1, std::max(0, c));
    };
    for (int i = 0; i < K; ++i) {
        poly.clear();
        for (int v = vs.start[size_t(i)]; v < vs.start[size_t(i) + 1]; ++v)
            poly.push_back(Pt{vs.xy[2 * size_t(v)], vs.xy[2 * size_t(v) + 1]});
        if (poly.empty()) continue;
        double bx0 = INFINITY, bx1 = -INFINITY, by0 = INFINITY, by1 = -INFINITY;
        for (const Pt& p : poly) {
            bx0 = std::min(bx0, p.x); bx1 = std::max(bx1, p.x);
            by0 = std::min(by0, p.y); by1 = std::max(by1, p.y);
        }
        const int ix0 = std::max(0, column_of(bx0) - 1), ix1 = std::min(grid - 1, column_of(bx1) + 1);
        const int iy0 = std::max(0, column_of(by0) - 1), iy1 = std::min(grid - 1, column_of(by1) + 1);
        for (int iy = iy0; iy <= iy1; ++iy)
            for (int ix = ix0; ix <= ix1; ++ix) {
                const double x0 = out->lo[size_t(ix)], x1 = out->hi[size_t(ix)];
                const double y0 = out->lo[size_t(iy)], y1 = out->hi[size_t(iy)];
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

bool build_cell_lists(const double* cb, int K, int grid, CellLists* out) {
    VoronoiSet vs;
    voronoi_polygons(cb, K, &vs);
    return build_cell_lists(vs, K, make_cell_map(grid, MapShape{}), out);
}

// Expected number of list entries that a point has to scan beyond the four of a cell record, for
// points drawn from 0.9 N(0, I) + 0.1 N(0, 4 I): pairs after the rotation are close to Gaussian,
// with a heavier tail where an outlier channel dominates its block.  Used to rank map shapes.
double overflow_cost(const CellLists& cl) {
    const int grid = cl.map.grid;
    double cost = 0.0;
    for (int comp = 0; comp < 2; ++comp) {
        const double sd = comp ? 2.0 : 1.0, weight = comp ? 0.1 : 0.9;
        std::vector<double> mass(static_cast<size_t>(grid), 0.0);
        for (int j = 0; j < grid; ++j) {  // columns without their margins: split at the midpoints of the overlaps
            const double lo = j == 0 ? -INFINITY : 0.5 * (cl.lo[size_t(j)] + cl.hi[size_t(j) - 1]);
            const double hi = j == grid - 1 ? INFINITY : 0.5 * (cl.hi[size_t(j)] + cl.lo[size_t(j) + 1]);
            mass[size_t(j)] = (std::isinf(hi) ? 1.0 : normal_cdf(hi, sd)) - (std::isinf(lo) ? 0.0 : normal_cdf(lo, sd));
        }
        for (int iy = 0; iy < grid; ++iy)
            for (int ix = 0; ix < grid; ++ix) {
                const size_t n = cl.lists[size_t(iy) * grid + ix].size();
                if (n > 4) cost += weight * mass[size_t(ix)] * mass[size_t(iy)] * double(n);
            }
    }
    return cost;
}

// Device layout: one 8-byte record per cell holding up to four candidate indices in
// ascending order (the last one repeated as padding).  A cell with more candidates
// stores {0xFFFF, offset, count, 0} and its list goes to the overflow array.
bool pack_search_table(const CellLists& cl, SearchTable* out) {
    out->map = cl.map;
    out->cells.assign(size_t(cl.map.grid) * cl.map.grid * 4, 0);
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
    // the device copies the table in 16-byte pieces: pad it to a whole number of them
    while ((out->cells.size() + out->overflow.size()) % 8) out->overflow.push_back(0);
    return true;
}

bool choose_search_table(const float* codebook, int K, int grid, size_t budget_bytes, SearchTable* out) {
    std::vector<double> cb(static_cast<size_t>(2 * K), 0.0);
    for (int i = 0; i < 2 * K; ++i) cb[size_t(i)] = double(codebook[i]);
    VoronoiSet vs;
    voronoi_polygons(cb.data(), K, &vs);
    // A few map shapes around the default: how many cells end up with more than four candidates
    // depends on how the column boundaries happen to fall between the codewords of this codebook.
    std::vector<MapShape> shapes;
    for (double T : {17.0, 18.0, 19.0})
        for (double eps : {0.015, 0.02})
            for (double rho : {1.22, 1.27}) shapes.push_back(MapShape{T, eps, rho});
    for (int g = grid > 0 ? grid : default_grid(K); g >= 1; g -= 2) {
        if (size_t(g) * g * 8 <= budget_bytes) {
            bool found = false;
            double best = INFINITY;
            for (const MapShape& shape : shapes) {
                CellLists cl;
                SearchTable t;
                if (!build_cell_lists(vs, K, make_cell_map(g, shape), &cl) || !pack_search_table(cl, &t) ||
                    t.bytes() > budget_bytes)
                    continue;
                const double cost = overflow_cost(cl);
                if (cost < best) {
                    best = cost;
                    *out = std::move(t);
                    found = true;
                }
            }
            if (found) return true;
        }
        if (grid > 0) return false;
    }
    return false;
}

}  // namespace qamw

using namespace qamw;

extern "C" int qamw_search_table_build(const float* codebook_host, int K, int grid, size_t budget_bytes,
                                       float* map_out, uint16_t* cells_out, size_t cells_cap,
                                       uint16_t* overflow_out, size_t overflow_cap, int32_t* info_out) {
    if (!codebook_host || !info_out) return QAMW_ERR_ARG;
    if (K < 1 || K > QAMW_MAX_K || !is_pow2(K)) return QAMW_ERR_SHAPE;
    if (grid < 0 || grid > 255 || (grid > 0 && grid % 2 == 0)) return QAMW_ERR_ARG;
    SearchTable t;
    if (!choose_search_table(codebook_host, K, grid, budget_bytes, &t)) return QAMW_ERR_NOMEM;
    info_out[0] = t.map.grid;
    info_out[1] = t.n_candidates;
    info_out[2] = t.max_list;
    info_out[3] = t.n_overflow_cells;
    info_out[4] = int32_t(t.overflow.size());
    info_out[5] = int32_t(t.bytes());
    if (map_out) {
        map_out[0] = t.map.zmax;
        map_out[1] = t.map.c0;
        map_out[2] = t.map.c1;
        map_out[3] = t.map.c2;
    }
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
