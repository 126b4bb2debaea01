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

// Fine binning of one axis: bin = clamp(floor(z * kFineScale + kFineOffset), 0, kFineBins - 1).
constexpr int kFineBins = 4096;
constexpr double kFineScale = 256.0;
constexpr double kFineOffset = 2048.0;

// Host form of the search grid: per coarse cell the full candidate list.
struct CellLists {
    int grid = 0;
    std::vector<double> edges;        // grid+1 coarse boundaries (z units); the outermost are +-16384
    std::vector<uint8_t> lut;         // fine bin -> coarse column / row
    std::vector<std::vector<uint16_t>> lists;  // [iy*grid + ix], ascending codeword indices
    int max_list = 0;
    int n_candidates = 0;
};

// Device form (see pack_search_table in qamw_table.cpp).
struct SearchTable {
    int grid = 0;
    std::vector<uint8_t> lut;         // kFineBins bytes
    std::vector<uint16_t> cells;      // grid*grid records of 4 x u16
    std::vector<uint16_t> overflow;   // candidate lists of cells with more than 4 entries
    int n_overflow_cells = 0;
    int max_list = 0;
    int n_candidates = 0;
    size_t bytes() const { return lut.size() + cells.size() * 2 + overflow.size() * 2; }
};

int default_grid(int K);
bool build_cell_lists(const double* cb, int K, int grid, CellLists* out);
bool pack_search_table(const CellLists& cl, SearchTable* out);

// grid > 0: exactly that grid (fails if it does not fit); grid == 0: the default grid for K,
// shrunk until the table fits in budget_bytes.
bool choose_search_table(const float* codebook, int K, int grid, size_t budget_bytes, SearchTable* out);

void set_cuda_error(const char* what, int code);

}  // namespace qamw

struct qamw_codebook {
    int K = 0;
    int device = -1;
    // one device allocation: [codebook K*2 f32][cells grid^2 * 4 u16][overflow u16][lut 4096 u8]
    void* d_blob = nullptr;
    size_t blob_bytes = 0;
    size_t off_cells = 0, off_overflow = 0, off_lut = 0;
    int grid = 0;
    int n_candidates = 0, max_list = 0, n_overflow_cells = 0;
    std::vector<float> h_codebook;  // host copy (decode only needs the device codebook)
};

#endif  // QAMW_INTERNAL_H_
