// Internal declarations shared by the translation units of libqamw (not part of the C ABI).
#ifndef QAMW_INTERNAL_H_
#define QAMW_INTERNAL_H_

#include <cstdint>
#include <vector>

#include "qamw.h"

namespace qamw {

inline bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }
inline int ilog2(int64_t v) {
    int l = 0;
    while ((int64_t(1) << l) < v) ++l;
    return l;
}

// Column (and, with the same map, row) of the search grid that holds coordinate z:
//     c = min(max(z, -zmax), zmax);  t = c * c;
//     column = half + rn(c * (c0 + t * (c1 + t * c2)))            (rn: to nearest integer)
// an odd polynomial with slope a ((1 - t / T)^2 + eps): cells are narrow where a Gaussian source
// puts its codewords, widen up to sqrt(T) and get a few more columns between there and
// zmax = rho sqrt(T) for heavy-tailed inputs; the outermost columns take everything beyond.  The
// device evaluates it in f32 (three fused multiply-adds, the last one onto 1.5 * 2^23 + half, which
// leaves the integer in the low mantissa bits).  grid = 2 * half + 1 is odd.
struct CellMap {
    int grid = 0, half = 0;
    float zmax = 0.f, c0 = 0.f, c1 = 0.f, c2 = 0.f;
};
struct MapShape {
    double T = 18.0, eps = 0.02, rho = 1.25;
};
CellMap make_cell_map(int grid, const MapShape& shape);
// The map in exact arithmetic on the f32 coefficients (before rounding to an integer).
double cell_map_value(const CellMap& m, double z);

// Host form of the search grid: per cell the full candidate list.
struct CellLists {
    CellMap map;
    // Column j can be returned by the device for z in [lo[j], hi[j]]: the interval of the exact map
    // widened by a margin that covers the device's rounding; the outermost reach +-16384.
    std::vector<double> lo, hi;
    std::vector<std::vector<uint16_t>> lists;  // [iy*grid + ix], ascending codeword indices
    int max_list = 0;
    int n_candidates = 0;
};

// Device form (see pack_search_table in qamw_table.cpp).
struct SearchTable {
    CellMap map;
    std::vector<uint16_t> cells;      // grid*grid records of 4 x u16
    std::vector<uint16_t> overflow;   // candidate lists of cells with more than 4 entries
    int n_overflow_cells = 0;
    int max_list = 0;
    int n_candidates = 0;
    size_t bytes() const { return cells.size() * 2 + overflow.size() * 2; }
};

// Nearest-neighbour (Voronoi) polygons of all codewords, clipped to |z| <= 16384: the vertices of
// codeword i are xy[2 * start[i]] .. xy[2 * start[i + 1]).
struct VoronoiSet {
    std::vector<int> start;
    std::vector<double> xy;
};
void voronoi_polygons(const double* cb, int K, VoronoiSet* out);

int default_grid(int K);
bool build_cell_lists(const VoronoiSet& vs, int K, const CellMap& map, CellLists* out);
bool build_cell_lists(const double* cb, int K, int grid, CellLists* out);  // default map shape
double overflow_cost(const CellLists& cl);
bool pack_search_table(const CellLists& cl, SearchTable* out);

// grid > 0 (odd): exactly that grid (fails if it does not fit); grid == 0: the default grid for K,
// shrunk until the table fits in budget_bytes.
bool choose_search_table(const float* codebook, int K, int grid, size_t budget_bytes, SearchTable* out);

void set_cuda_error(const char* what, int code);
void set_error_text(const char* text);

// One weight matrix as the batched (multi-matrix) kernels see it: plain device pointers and sizes.
struct MatDesc {
    const void* W;
    const float* chan_scale;
    const int8_t* signs;
    const float* sigma;
    const float* act_rms;
    uint8_t* packed;
    float* row_norm;
    void* w_hat;
    double* dist4;
    long long w_row_stride;       // elements
    long long packed_row_stride;  // bytes
    long long calib_offset;       // batched calibration: byte offset of this matrix's partial sums in the workspace,
    int calib_first_block;        //   the first block whose span touches it, and the number of slots it has
    int calib_slots;              //   ((blocks touching it) x (row groups per block)), each [pair_stride] doubles
    int d_out, d_in;
};

// Fast multi-matrix paths (qamw_rows.cu).  `descs` is a device array of n descriptors, or NULL with
// n == 1 and the single descriptor passed by value.  They return QAMW_ERR_SHAPE without launching
// when a matrix does not meet the fast kernels' layout rules; the caller then uses the general kernels.
int rows_decode(const MatDesc* descs_dev, const MatDesc* descs_host, int n, const void* spans_dev, int span_blocks,
                int block, int K, const float* codebook_dev, uint32_t flags, void* stream);
int rows_encode(const MatDesc* descs_dev, const MatDesc* descs_host, int n, const void* spans_dev, int span_blocks,
                int block, int K, int w_bf16, const ::qamw_codebook* cb, uint32_t flags, int32_t* status, void* stream,
                void* calib_base = nullptr);  // calib_base: run the calibration pass instead (cb may be NULL)
int sm_count();
int check_matrix_params(const qamw_params* p);
long long distortion_items(int d_out, int d_in);  // work items of the distortion kernel for one matrix
// zeroes every matrix's four sums, then one launch over all matrices (spans of the concatenated item list)
// Where the blocks of the batched distortion kernel leave their partial sums: records of four doubles,
// matrix by matrix; matrix m appears in the spans of blocks owner[m].first .. owner[m].last and block b's
// record for it is number owner[m].offset + b - owner[m].first.  counter is the ticket of the blocks;
// the one that finishes last adds the records up in a fixed order and resets it.
struct DistOwner {
    int first, last;  // blocks
    int offset;       // first record of the matrix
};
struct DistReduce {
    double* partial;
    const DistOwner* owner;
    unsigned int* counter;  // zero between launches
};
int distortion_batch_launch(const MatDesc* descs_dev, int n, const void* spans_dev, int blocks, int w_bf16,
                            const DistReduce& red, void* stream);  // QAMW_OK or the error code every entry point reports

}  // namespace qamw

struct qamw_codebook {
    int K = 0;
    int device = -1;
    // one device allocation: [codebook K*2 f32][cells grid^2 * 4 u16][overflow u16]
    void* d_blob = nullptr;
    size_t blob_bytes = 0;
    size_t off_cells = 0, off_overflow = 0;
    qamw::CellMap map;
    int n_candidates = 0, max_list = 0, n_overflow_cells = 0;
    std::vector<float> h_codebook;  // host copy (decode only needs the device codebook)
    // polar baseline: the blob then is [codebook K*2 f32][squared amplitude thresholds 2^Ba f32]
    // [boundary unit vectors 2^Bp / 2 float2] and off_cells / off_overflow point at the two tables
    bool polar = false;
    int polar_ba = 0, polar_bp = 0;
};

#endif  // QAMW_INTERNAL_H_
