// CUDA kernels (sm_100a) and device-side entry points of libqamw.
//
// Thread geometry shared by every row kernel.  A row of d_in elements is owned by one
// "group" of TG threads (a whole number of warps); a thread block holds GROUPS such groups,
// each working on its own row, and the grid is persistent (rows are strided over all groups).
// A thread keeps 32 elements of its row in registers as four "octets" of eight contiguous
// elements.  With L = max(1, b/32) threads per Hadamard block of size b, thread l of a block
// owns octets l, l+L, l+2L, l+3L of that block (for b < 32 a thread owns 32 contiguous
// elements, i.e. several whole blocks).  The butterfly stages h = 1, 2, 4 then stay inside an
// octet, stages 8 .. 4L are exchanged with warp shuffles (L <= 32, so never across warps) and
// the last two stages (b/4, b/2) combine the thread's own octets.  Stages are always executed
// in ascending order of h, which is what makes the f32 result reproducible bit for bit.
// The thread owns the same columns in every row, so the per-column factors (channel scale
// times sign, pair scales) live in registers for the whole kernel.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "qamw_internal.h"

namespace qamw {

static thread_local char g_last_error[256] = "";

void set_cuda_error(const char* what, int code) {
    std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(cudaError_t(code)));
}

}  // namespace qamw

using namespace qamw;

namespace {

constexpr int kMaxThreads = 512;   // threads per block (register budget: 128 per thread)
constexpr int kMaxGroups = 15;     // named barriers 1..15
constexpr unsigned kFull = 0xffffffffu;

struct RowGeom {
    int d_out, d_in;
    int log2b;        // log2 of the Hadamard block
    int tg;           // threads per group (multiple of 32)
    int groups;       // groups per thread block
    int vec;          // rows can be read with 16-byte loads
    int w_bf16;       // 1 = bf16 weights, 0 = f32
    long long w_row_stride;  // elements
};

// ---------------------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------------------

__device__ __forceinline__ void group_barrier(int group, int n_threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(group + 1), "r"(n_threads) : "memory");
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(kFull, v, s);
    return v;
}

// Element offset of octet m of this thread, given its index inside the group.
template <int LOG2B_T>
__device__ __forceinline__ int octet_offset(int tid_g, int m) {
    constexpr int L = 1 << (LOG2B_T >= 5 ? LOG2B_T - 5 : 0);
    if (LOG2B_T >= 5) {
        const int blk = tid_g / L, l = tid_g % L;
        return (blk << LOG2B_T) + 8 * (l + L * m);
    }
    return tid_g * 32 + 8 * m;
}

// One butterfly (a, c) -> (a + c, a - c), round-to-nearest f32, never fused.
__device__ __forceinline__ void bfly(float& a, float& c) {
    float s = __fadd_rn(a, c), d = __fsub_rn(a, c);
    a = s;
    c = d;
}

// Unnormalised Walsh-Hadamard butterfly of the thread's 4 x 8 elements, stages ascending.
// LOG2B_T >= 5: block size 2^LOG2B_T known at compile time; LOG2B_T == 0: block size < 32 given
// at run time (log2b in 1..4).
template <int LOG2B_T>
__device__ __forceinline__ void fwht_regs(float (&x)[4][8], int log2b_rt, int lane_in_block) {
    const int log2b = LOG2B_T ? LOG2B_T : log2b_rt;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        if (log2b >= 1) {
            bfly(x[m][0], x[m][1]); bfly(x[m][2], x[m][3]); bfly(x[m][4], x[m][5]); bfly(x[m][6], x[m][7]);
        }
        if (log2b >= 2) {
            bfly(x[m][0], x[m][2]); bfly(x[m][1], x[m][3]); bfly(x[m][4], x[m][6]); bfly(x[m][5], x[m][7]);
        }
        if (log2b >= 3) {
            bfly(x[m][0], x[m][4]); bfly(x[m][1], x[m][5]); bfly(x[m][2], x[m][6]); bfly(x[m][3], x[m][7]);
        }
    }
    if (LOG2B_T >= 6) {
        constexpr int L = 1 << (LOG2B_T >= 5 ? LOG2B_T - 5 : 0);
#pragma unroll
        for (int s = 1; s < L; s <<= 1) {
            // lower lane: v + p ; upper lane: p - v = fma(v, -1, p) (the product is exact)
            const float sgn = (lane_in_block & s) ? -1.0f : 1.0f;
#pragma unroll
            for (int m = 0; m < 4; ++m)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float p = __shfl_xor_sync(kFull, x[m][e], s);
                    x[m][e] = __fmaf_rn(x[m][e], sgn, p);
                }
        }
    }
    if (log2b >= 4) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            bfly(x[0][e], x[1][e]);
            bfly(x[2][e], x[3][e]);
        }
    }
    if (log2b >= 5) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            bfly(x[0][e], x[2][e]);
            bfly(x[1][e], x[3][e]);
        }
    }
}

// Raw bits of the thread's 32 weights of one row (bf16: 4 x 16 bytes, f32: 8 x 16 bytes).
template <bool BF16>
struct RawRow {
    uint4 v[BF16 ? 4 : 8];
};

template <bool BF16, int LOG2B_T>
__device__ __forceinline__ void load_row(RawRow<BF16>& raw, const void* W, long long row, const RowGeom& g, int tid_g) {
    const char* base = static_cast<const char*>(W) + row * g.w_row_stride * (BF16 ? 2 : 4);
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int e0 = octet_offset<LOG2B_T>(tid_g, m);
        if (g.vec) {
            if (e0 < g.d_in) {
                const uint4* p = reinterpret_cast<const uint4*>(base + size_t(e0) * (BF16 ? 2 : 4));
                if (BF16) {
                    raw.v[m] = __ldg(p);
                } else {
                    raw.v[2 * m] = __ldg(p);
                    raw.v[2 * m + 1] = __ldg(p + 1);
                }
            } else {
                if (BF16) {
                    raw.v[m] = make_uint4(0, 0, 0, 0);
                } else {
                    raw.v[2 * m] = make_uint4(0, 0, 0, 0);
                    raw.v[2 * m + 1] = make_uint4(0, 0, 0, 0);
                }
            }
        } else {
            // element-wise path for rows that are not 16-byte aligned or not a multiple of 8 long
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int j = e0 + e;
                uint32_t bits = 0;
                if (j < g.d_in) {
                    if (BF16) bits = reinterpret_cast<const uint16_t*>(base)[j];
                    else bits = reinterpret_cast<const uint32_t*>(base)[j];
                }
                w[e] = bits;
            }
            if (BF16) {
                raw.v[m] = make_uint4(w[0] | (w[1] << 16), w[2] | (w[3] << 16), w[4] | (w[5] << 16), w[6] | (w[7] << 16));
            } else {
                raw.v[2 * m] = make_uint4(w[0], w[1], w[2], w[3]);
                raw.v[2 * m + 1] = make_uint4(w[4], w[5], w[6], w[7]);
            }
        }
    }
}

template <bool BF16>
__device__ __forceinline__ void raw_to_float(const RawRow<BF16>& raw, float (&x)[4][8]) {
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        if (BF16) {
            const uint32_t w[4] = {raw.v[m].x, raw.v[m].y, raw.v[m].z, raw.v[m].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                x[m][2 * i] = __uint_as_float(w[i] << 16);
                x[m][2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
            }
        } else {
            const uint4 a = raw.v[2 * m], c = raw.v[2 * m + 1];
            x[m][0] = __uint_as_float(a.x); x[m][1] = __uint_as_float(a.y);
            x[m][2] = __uint_as_float(a.z); x[m][3] = __uint_as_float(a.w);
            x[m][4] = __uint_as_float(c.x); x[m][5] = __uint_as_float(c.y);
            x[m][6] = __uint_as_float(c.z); x[m][7] = __uint_as_float(c.w);
        }
    }
}

// Per-thread column constants: t_j = f32(s_j) * sign_j (0 beyond the row).
template <int LOG2B_T>
__device__ __forceinline__ void load_col_factors(float (&t)[4][8], const float* chan_scale, const int8_t* signs,
                                                 int d_in, int tid_g) {
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int e0 = octet_offset<LOG2B_T>(tid_g, m);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = e0 + e;
            float v = 0.f;
            if (j < d_in) v = (chan_scale ? chan_scale[j] : 1.0f) * float(signs[j]);
            t[m][e] = v;
        }
    }
}

// Scaling, row norm and butterfly of one row held in registers (the arithmetic contract of the
// encoder, steps x, r, h).  Returns the row norm r; x holds the unnormalised butterfly output.
// `red` is this group's reduction scratch (one double per warp, two buffers).
template <bool BF16, int LOG2B_T>
__device__ __forceinline__ float front_half(const RawRow<BF16>& raw, const float (&t)[4][8], float (&x)[4][8],
                                            const RowGeom& g, int group, int tid_g, int lane_in_block, double* red,
                                            int parity) {
    raw_to_float<BF16>(raw, x);
    double ss = 0.0;
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            x[m][e] = __fmul_rn(x[m][e], t[m][e]);
            const double xd = double(x[m][e]);
            ss = fma(xd, xd, ss);
        }
    fwht_regs<LOG2B_T>(x, g.log2b, lane_in_block);
    ss = warp_sum(ss);
    const int n_warps = g.tg >> 5;
    double* slot = red + parity * 32;
    if ((tid_g & 31) == 0) slot[tid_g >> 5] = ss;
    group_barrier(group, g.tg);
    double total = 0.0;
    for (int w = 0; w < n_warps; ++w) total += slot[w];
    return float(sqrt(total));
}

// g = f32(1 / (r * sqrt(b))), computed in double.
__device__ __forceinline__ float inv_norm_factor(float r, int log2b) {
    return float(1.0 / (double(r) * sqrt(double(1 << log2b))));
}

// ---------------------------------------------------------------------------------------------
// nearest-codeword search
// ---------------------------------------------------------------------------------------------

struct SearchSmem {
    const float2* cb;         // K codewords
    const uint2* cells;       // grid*grid records
    const uint16_t* overflow;
    const uint8_t* lut;       // 4096 bytes
    int grid;
    int K;
};

__device__ __forceinline__ void consider(const float2* cb, int k, float zx, float zy, float& best, int& arg) {
    const float2 c = cb[k];
    const float dx = __fsub_rn(zx, c.x), dy = __fsub_rn(zy, c.y);
    const float d = __fmaf_rn(dy, dy, __fmul_rn(dx, dx));
    if (d < best) {
        best = d;
        arg = k;
    }
}

__device__ __noinline__ int search_exhaustive(const float2* cb, int K, float zx, float zy) {
    float best = INFINITY;
    int arg = 0;
    for (int k = 0; k < K; ++k) consider(cb, k, zx, zy, best, arg);
    return arg;
}

__device__ __noinline__ int search_overflow(const SearchSmem& s, uint2 rec, float zx, float zy) {
    const int off = int(rec.x >> 16), cnt = int(rec.y & 0xffffu);
    float best = INFINITY;
    int arg = 0;
    for (int i = 0; i < cnt; ++i) consider(s.cb, int(s.overflow[off + i]), zx, zy, best, arg);
    return arg;
}

__device__ __forceinline__ int search_table(const SearchSmem& s, float zx, float zy) {
    // beyond the table's reach (or NaN): exhaustive scan
    if (!(fabsf(zx) < 16000.0f && fabsf(zy) < 16000.0f)) return search_exhaustive(s.cb, s.K, zx, zy);
    const float fx = __fmaf_rn(zx, 256.0f, 2048.0f), fy = __fmaf_rn(zy, 256.0f, 2048.0f);
    const int bx = min(max(int(fx), 0), 4095), by = min(max(int(fy), 0), 4095);
    const int ix = s.lut[bx], iy = s.lut[by];
    const uint2 rec = s.cells[iy * s.grid + ix];
    if ((rec.x & 0xffffu) == 0xffffu) return search_overflow(s, rec, zx, zy);
    float best = INFINITY;
    int arg = 0;
    consider(s.cb, int(rec.x & 0xffffu), zx, zy, best, arg);
    consider(s.cb, int(rec.x >> 16), zx, zy, best, arg);
    consider(s.cb, int(rec.y & 0xffffu), zx, zy, best, arg);
    consider(s.cb, int(rec.y >> 16), zx, zy, best, arg);
    return arg;
}

// ---------------------------------------------------------------------------------------------
// encode kernel
// ---------------------------------------------------------------------------------------------

struct EncodeArgs {
    RowGeom g;
    const void* W;
    const float* chan_scale;
    const int8_t* signs;
    const float* sigma;
    const uint4* blob;       // codebook + table, as laid out by qamw_codebook_create
    int blob_bytes;
    int off_cells, off_overflow, off_lut;
    int K, log2K, grid;
    int brute;
    uint8_t* packed;
    long long packed_row_stride;  // bytes
    int row_words;           // 32-bit words per packed row (stride / 4)
    float* row_norm;
    int32_t* status;
    int idx_stride;          // u16 entries of index staging per group
};

template <bool BF16, int LOG2B_T>
__global__ void __launch_bounds__(kMaxThreads, 1) encode_kernel(const EncodeArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    const RowGeom& g = a.g;
    // shared memory: [blob][red: groups x 64 doubles][idx: groups x idx_stride u16]
    {
        uint4* dst = reinterpret_cast<uint4*>(smem);
        for (int i = threadIdx.x; i < a.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(a.blob + i);
    }
    const int blob_pad = (a.blob_bytes + 15) & ~15;
    double* red_all = reinterpret_cast<double*>(smem + blob_pad);
    uint16_t* idx_all = reinterpret_cast<uint16_t*>(smem + blob_pad + g.groups * 64 * sizeof(double));
    __syncthreads();

    SearchSmem s;
    s.cb = reinterpret_cast<const float2*>(smem);
    s.cells = reinterpret_cast<const uint2*>(smem + a.off_cells);
    s.overflow = reinterpret_cast<const uint16_t*>(smem + a.off_overflow);
    s.lut = smem + a.off_lut;
    s.grid = a.grid;
    s.K = a.K;

    const int group = threadIdx.x / g.tg;
    const int tid_g = threadIdx.x - group * g.tg;
    const int lane_in_block = (LOG2B_T >= 5) ? (tid_g & ((1 << (LOG2B_T >= 5 ? LOG2B_T - 5 : 0)) - 1)) : 0;
    double* red = red_all + group * 64;
    uint16_t* idx_s = idx_all + size_t(group) * a.idx_stride;
    const int n_pairs = g.d_in >> 1;

    float t[4][8];
    load_col_factors<LOG2B_T>(t, a.chan_scale, a.signs, g.d_in, tid_g);
    float q[4][4];
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int k0 = octet_offset<LOG2B_T>(tid_g, m) >> 1;
#pragma unroll
        for (int p = 0; p < 4; ++p) q[m][p] = (k0 + p < n_pairs) ? float(1.0 / double(a.sigma[k0 + p])) : 0.f;
    }

    const long long row_step = (long long)gridDim.x * g.groups;
    long long row = (long long)blockIdx.x * g.groups + group;
    const unsigned div_magic = 0xffffffffu / unsigned(a.log2K) + 1u;  // ceil(2^32 / B)

    RawRow<BF16> raw;
    if (row < g.d_out) load_row<BF16, LOG2B_T>(raw, a.W, row, g, tid_g);
    int parity = 0;
    for (; row < g.d_out; row += row_step, parity ^= 1) {
        RawRow<BF16> nxt;
        const long long next_row = row + row_step;
        if (next_row < g.d_out) load_row<BF16, LOG2B_T>(nxt, a.W, next_row, g, tid_g);

        float x[4][8];
        const float r = front_half<BF16, LOG2B_T>(raw, t, x, g, group, tid_g, lane_in_block, red, parity);
        const bool finite = isfinite(r);
        if (tid_g == 0) {
            a.row_norm[row] = r;
            if (!finite && a.status) atomicOr(a.status, 1);
        }
        const float gn = (finite && r > 0.f) ? inv_norm_factor(r, g.log2b) : 0.f;

#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int k0 = octet_offset<LOG2B_T>(tid_g, m) >> 1;
            if (k0 < n_pairs) {
                uint32_t id[4];
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    float zx = 0.f, zy = 0.f;
                    if (gn != 0.f) {  // zero or non-finite rows are encoded as the origin
                        zx = __fmul_rn(__fmul_rn(x[m][2 * p], gn), q[m][p]);
                        zy = __fmul_rn(__fmul_rn(x[m][2 * p + 1], gn), q[m][p]);
                    }
                    id[p] = uint32_t(a.brute ? search_exhaustive(s.cb, s.K, zx, zy) : search_table(s, zx, zy));
                }
                *reinterpret_cast<uint2*>(idx_s + k0) = make_uint2(id[0] | (id[1] << 16), id[2] | (id[3] << 16));
            }
        }
        group_barrier(group, g.tg);

        // bit packing: index k occupies bits [k*B, (k+1)*B) of the row stream (LSB first)
        uint32_t* out = reinterpret_cast<uint32_t*>(a.packed + row * a.packed_row_stride);
        const int B = a.log2K;
        for (int w = tid_g; w < a.row_words; w += g.tg) {
            const unsigned bit0 = unsigned(w) * 32u;
            int k = int(__umulhi(bit0, div_magic));  // floor(bit0 / B)
            uint32_t word = 0;
            for (; k < n_pairs; ++k) {
                const int sh = k * B - int(bit0);
                if (sh >= 32) break;
                const uint32_t v = idx_s[k];
                word |= sh >= 0 ? (v << sh) : (v >> (-sh));
            }
            out[w] = word;
        }
        raw = nxt;
    }
}

// ---------------------------------------------------------------------------------------------
// auxiliary row kernel: rotate (mode 0: write y) or calibrate (mode 1: per-group |z_k| sums)
// ---------------------------------------------------------------------------------------------

struct AuxArgs {
    RowGeom g;
    const void* W;
    const float* chan_scale;
    const int8_t* signs;
    int mode;
    // rotate
    float* y_out;
    float* row_norm;
    // calibrate
    int n_calib_rows;        // rows visited: floor(t * d_out / n_calib_rows)
    double* partial;         // [total_groups][n_pairs_padded] sums, then [total_groups] used-row counts
    int pair_stride;
    int32_t* status;
};

template <bool BF16, int LOG2B_T>
__global__ void __launch_bounds__(kMaxThreads, 1) aux_kernel(const AuxArgs a) {
    __shared__ double red_all[kMaxGroups * 64];
    const RowGeom& g = a.g;
    const int group = threadIdx.x / g.tg;
    const int tid_g = threadIdx.x - group * g.tg;
    const int lane_in_block = (LOG2B_T >= 5) ? (tid_g & ((1 << (LOG2B_T >= 5 ? LOG2B_T - 5 : 0)) - 1)) : 0;
    double* red = red_all + group * 64;
    const int n_pairs = g.d_in >> 1;

    float t[4][8];
    load_col_factors<LOG2B_T>(t, a.chan_scale, a.signs, g.d_in, tid_g);

    const int n_rows = a.mode == 1 ? a.n_calib_rows : g.d_out;
    const long long total_groups = (long long)gridDim.x * g.groups;
    const long long my_group = (long long)blockIdx.x * g.groups + group;
    double acc[4][4];
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[m][p] = 0.0;
    int used = 0;

    int parity = 0;
    for (long long it = my_group; it < n_rows; it += total_groups, parity ^= 1) {
        const long long row = a.mode == 1 ? (it * g.d_out) / a.n_calib_rows : it;
        RawRow<BF16> raw;
        load_row<BF16, LOG2B_T>(raw, a.W, row, g, tid_g);
        float x[4][8];
        const float r = front_half<BF16, LOG2B_T>(raw, t, x, g, group, tid_g, lane_in_block, red, parity);
        const bool finite = isfinite(r);
        if (!finite && a.status && tid_g == 0) atomicOr(a.status, 1);
        const float gn = (finite && r > 0.f) ? inv_norm_factor(r, g.log2b) : 0.f;
        if (a.mode == 0) {
            if (tid_g == 0) a.row_norm[row] = r;
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const int e0 = octet_offset<LOG2B_T>(tid_g, m);
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e0 + e < g.d_in) a.y_out[row * g.d_in + e0 + e] = __fmul_rn(x[m][e], gn);
            }
        } else if (gn != 0.f) {
            ++used;
#pragma unroll
            for (int m = 0; m < 4; ++m)
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const float y0 = __fmul_rn(x[m][2 * p], gn), y1 = __fmul_rn(x[m][2 * p + 1], gn);
                    acc[m][p] += double(sqrtf(__fmaf_rn(y1, y1, __fmul_rn(y0, y0))));
                }
        }
    }
    if (a.mode == 1) {
        double* mine = a.partial + my_group * a.pair_stride;
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int k0 = octet_offset<LOG2B_T>(tid_g, m) >> 1;
#pragma unroll
            for (int p = 0; p < 4; ++p)
                if (k0 + p < n_pairs) mine[k0 + p] = acc[m][p];
        }
        if (tid_g == 0) a.partial[total_groups * a.pair_stride + my_group] = double(used);
    }
}

// sigma_k from the per-group partial sums, added in group order (reproducible).
__global__ void calibrate_finish_kernel(const double* partial, int total_groups, int pair_stride, int n_pairs,
                                        int d_in, float* sigma_out) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n_pairs) return;
    double used = 0.0, sum = 0.0;
    for (int gidx = 0; gidx < total_groups; ++gidx) {
        used += partial[size_t(total_groups) * pair_stride + gidx];
        sum += partial[size_t(gidx) * pair_stride + k];
    }
    const double inv_sqrt_d = 1.0 / sqrt(double(d_in));
    double sg = used > 0.0 ? (sum / used) / sqrt(1.5707963267948966) : inv_sqrt_d;
    sg = fmax(sg, 1e-4 * inv_sqrt_d);
    sigma_out[k] = float(sg);
}

// ---------------------------------------------------------------------------------------------
// decode kernel
// ---------------------------------------------------------------------------------------------

struct DecodeArgs {
    RowGeom g;               // d_out, d_in, log2b, tg, groups; vec = output rows 16-byte aligned
    const uint8_t* packed;
    long long packed_row_stride;
    int row_words;           // readable 32-bit words per packed row
    const float* row_norm;
    const float* chan_scale;
    const int8_t* signs;
    const float* sigma;
    const float2* codebook;  // device, K entries
    int K, log2K;
    __nv_bfloat16* out;
};

template <int LOG2B_T>
__global__ void __launch_bounds__(kMaxThreads, 1) decode_kernel(const DecodeArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    float2* cb = reinterpret_cast<float2*>(smem);
    for (int i = threadIdx.x; i < a.K; i += blockDim.x) cb[i] = a.codebook[i];
    __syncthreads();

    const RowGeom& g = a.g;
    const int group = threadIdx.x / g.tg;
    const int tid_g = threadIdx.x - group * g.tg;
    const int lane_in_block = (LOG2B_T >= 5) ? (tid_g & ((1 << (LOG2B_T >= 5 ? LOG2B_T - 5 : 0)) - 1)) : 0;
    const int n_pairs = g.d_in >> 1;
    const int B = a.log2K;
    const uint32_t mask = (1u << B) - 1u;

    // per-column output factor sign_j / (s_j sqrt(b)) and per-pair sigma
    float mcol[4][8], sg[4][4];
    const double inv_sqrt_b = 1.0 / sqrt(double(1 << g.log2b));
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int e0 = octet_offset<LOG2B_T>(tid_g, m);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = e0 + e;
            float v = 0.f;
            if (j < g.d_in) v = float(double(a.signs[j]) * inv_sqrt_b / double(a.chan_scale ? a.chan_scale[j] : 1.0f));
            mcol[m][e] = v;
        }
#pragma unroll
        for (int p = 0; p < 4; ++p) sg[m][p] = ((e0 >> 1) + p < n_pairs) ? a.sigma[(e0 >> 1) + p] : 0.f;
    }

    const long long row_step = (long long)gridDim.x * g.groups;
    for (long long row = (long long)blockIdx.x * g.groups + group; row < g.d_out; row += row_step) {
        const uint32_t* in = reinterpret_cast<const uint32_t*>(a.packed + row * a.packed_row_stride);
        const float r = a.row_norm[row];
        float x[4][8];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int e0 = octet_offset<LOG2B_T>(tid_g, m);
            const int k0 = e0 >> 1;
            if (k0 < n_pairs) {
                const unsigned bit0 = unsigned(k0) * unsigned(B);
                const int w0 = int(bit0 >> 5), sh = int(bit0 & 31u);
                const uint32_t lo = __ldg(in + w0);
                const uint32_t mid = (w0 + 1 < a.row_words) ? __ldg(in + w0 + 1) : 0u;
                const uint32_t hi = (w0 + 2 < a.row_words) ? __ldg(in + w0 + 2) : 0u;
                // 64-bit window starting at bit `sh` of (hi:mid:lo); 4*B <= 48 bits are needed
                unsigned long long win = ((unsigned long long)mid << 32 | lo) >> sh;
                if (sh) win |= (unsigned long long)hi << (64 - sh);
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const bool valid = k0 + p < n_pairs;
                    const uint32_t id = uint32_t(win >> (p * B)) & mask;
                    const float2 c = cb[valid ? id : 0u];
                    x[m][2 * p] = c.x * sg[m][p];
                    x[m][2 * p + 1] = c.y * sg[m][p];
                }
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) x[m][e] = 0.f;
            }
        }
        fwht_regs<LOG2B_T>(x, g.log2b, lane_in_block);
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int e0 = octet_offset<LOG2B_T>(tid_g, m);
            if (e0 >= g.d_in) continue;
            __nv_bfloat16* dst = a.out + row * g.d_in + e0;
            if (g.vec) {
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(x[m][2 * i] * (mcol[m][2 * i] * r),
                                                              x[m][2 * i + 1] * (mcol[m][2 * i + 1] * r));
                    w[i] = *reinterpret_cast<uint32_t*>(&h2);
                }
                *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e0 + e < g.d_in) dst[e] = __float2bfloat16_rn(x[m][e] * (mcol[m][e] * r));
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// distortion kernel
// ---------------------------------------------------------------------------------------------

template <bool BF16>
__global__ void __launch_bounds__(256) distortion_kernel(const void* W, long long w_row_stride, const __nv_bfloat16* What,
                                                         const float* act_rms, int d_out, int d_in, double* out4) {
    double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    for (long long row = blockIdx.x; row < d_out; row += gridDim.x) {
        const char* wrow = static_cast<const char*>(W) + row * w_row_stride * (BF16 ? 2 : 4);
        const __nv_bfloat16* hrow = What + row * d_in;
        for (int j = threadIdx.x; j < d_in; j += blockDim.x) {
            const float w = BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(wrow)[j])
                                 : reinterpret_cast<const float*>(wrow)[j];
            const double wd = double(w), e = wd - double(__bfloat162float(hrow[j]));
            const double r2 = act_rms ? double(act_rms[j]) * double(act_rms[j]) : 1.0;
            s0 += e * e;
            s1 += wd * wd;
            s2 += r2 * e * e;
            s3 += r2 * wd * wd;
        }
    }
    __shared__ double sh[4][8];
    s0 = warp_sum(s0); s1 = warp_sum(s1); s2 = warp_sum(s2); s3 = warp_sum(s3);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { sh[0][warp] = s0; sh[1][warp] = s1; sh[2][warp] = s2; sh[3][warp] = s3; }
    __syncthreads();
    if (threadIdx.x < 4) {
        double v = 0;
        for (int w = 0; w < int(blockDim.x >> 5); ++w) v += sh[threadIdx.x][w];
        atomicAdd(out4 + threadIdx.x, v);
    }
}

// ---------------------------------------------------------------------------------------------
// host-side launch helpers
// ---------------------------------------------------------------------------------------------

int check_params(const qamw_params* p) {
    if (!p) return QAMW_ERR_ARG;
    if (p->d_out < 0 || p->d_in <= 0) return QAMW_ERR_ARG;
    if (p->d_in % 2) return QAMW_ERR_SHAPE;
    if (p->block < 2 || p->block > QAMW_MAX_BLOCK || !is_pow2(p->block) || p->d_in % p->block) return QAMW_ERR_SHAPE;
    if (p->K < 2 || p->K > QAMW_MAX_K || !is_pow2(p->K)) return QAMW_ERR_SHAPE;
    if (p->d_in > 32 * kMaxThreads) return QAMW_ERR_SHAPE;
    if (p->w_dtype != QAMW_DTYPE_F32 && p->w_dtype != QAMW_DTYPE_BF16) return QAMW_ERR_ARG;
    if (p->w_row_stride < p->d_in) return QAMW_ERR_ARG;
    return QAMW_OK;
}

RowGeom make_geom(const qamw_params* p, const void* W) {
    RowGeom g;
    g.d_out = p->d_out;
    g.d_in = p->d_in;
    g.log2b = ilog2(p->block);
    const int threads = (p->d_in + 31) / 32;
    g.tg = ((threads + 31) / 32) * 32;
    g.groups = std::max(1, std::min(kMaxGroups, kMaxThreads / g.tg));
    g.w_bf16 = p->w_dtype == QAMW_DTYPE_BF16;
    const size_t esz = g.w_bf16 ? 2 : 4;
    g.vec = (p->d_in % 8 == 0) && (reinterpret_cast<uintptr_t>(W) % 16 == 0) && ((size_t(p->w_row_stride) * esz) % 16 == 0);
    g.w_row_stride = p->w_row_stride;
    return g;
}

int sm_count() {
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        cudaDeviceGetAttribute(&cached, cudaDevAttrMultiProcessorCount, dev);
        cached_dev = dev;
    }
    return cached > 0 ? cached : 148;
}

int finish_launch(const char* what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_cuda_error(what, int(e));
        return QAMW_ERR_CUDA;
    }
    return QAMW_OK;
}

template <class Kernel>
int set_smem(Kernel k, size_t bytes) {
    if (bytes > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes));
        if (e != cudaSuccess) {
            set_cuda_error("cudaFuncSetAttribute", int(e));
            return QAMW_ERR_NOMEM;
        }
    }
    return QAMW_OK;
}

template <bool BF16, int LOG2B_T>
int launch_encode(const EncodeArgs& a, int blocks, size_t smem, cudaStream_t st) {
    int rc = set_smem(encode_kernel<BF16, LOG2B_T>, smem);
    if (rc) return rc;
    encode_kernel<BF16, LOG2B_T><<<blocks, a.g.tg * a.g.groups, smem, st>>>(a);
    return finish_launch("encode_kernel");
}

template <bool BF16, int LOG2B_T>
int launch_aux(const AuxArgs& a, int blocks, cudaStream_t st) {
    aux_kernel<BF16, LOG2B_T><<<blocks, a.g.tg * a.g.groups, 0, st>>>(a);
    return finish_launch("aux_kernel");
}

template <int LOG2B_T>
int launch_decode(const DecodeArgs& a, int blocks, size_t smem, cudaStream_t st) {
    int rc = set_smem(decode_kernel<LOG2B_T>, smem);
    if (rc) return rc;
    decode_kernel<LOG2B_T><<<blocks, a.g.tg * a.g.groups, smem, st>>>(a);
    return finish_launch("decode_kernel");
}

#define QAMW_DISPATCH_LOG2B(log2b, CALL)            \
    switch ((log2b) >= 5 ? (log2b) : 0) {           \
        case 0: CALL(0); break;                     \
        case 5: CALL(5); break;                     \
        case 6: CALL(6); break;                     \
        case 7: CALL(7); break;                     \
        case 8: CALL(8); break;                     \
        case 9: CALL(9); break;                     \
        default: CALL(10); break;                   \
    }

}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------

extern "C" const char* qamw_last_cuda_error(void) { return g_last_error; }

extern "C" int qamw_codebook_create(const float* codebook_host, int K, int grid, qamw_codebook** out) {
    if (!codebook_host || !out) return QAMW_ERR_ARG;
    if (K < 2 || K > QAMW_MAX_K || !is_pow2(K)) return QAMW_ERR_SHAPE;
    if (grid < 0 || grid > 255) return QAMW_ERR_ARG;
    *out = nullptr;
    SearchTable t;
    // leave room for the per-group scratch of the encoder inside the 227 KB of one SM
    const size_t budget = size_t(200) * 1024 - size_t(K) * 8;
    if (!choose_search_table(codebook_host, K, grid, budget, &t)) return QAMW_ERR_NOMEM;
    qamw_codebook* cb = new (std::nothrow) qamw_codebook();
    if (!cb) return QAMW_ERR_NOMEM;
    cb->K = K;
    cb->grid = t.grid;
    cb->n_candidates = t.n_candidates;
    cb->max_list = t.max_list;
    cb->n_overflow_cells = t.n_overflow_cells;
    cb->h_codebook.assign(codebook_host, codebook_host + 2 * K);
    cb->off_cells = size_t(K) * 8;
    cb->off_overflow = cb->off_cells + t.cells.size() * 2;
    cb->off_lut = cb->off_overflow + t.overflow.size() * 2;
    cb->blob_bytes = cb->off_lut + t.lut.size();
    std::vector<unsigned char> blob(cb->blob_bytes, 0);
    std::memcpy(blob.data(), codebook_host, size_t(K) * 8);
    std::memcpy(blob.data() + cb->off_cells, t.cells.data(), t.cells.size() * 2);
    if (!t.overflow.empty()) std::memcpy(blob.data() + cb->off_overflow, t.overflow.data(), t.overflow.size() * 2);
    std::memcpy(blob.data() + cb->off_lut, t.lut.data(), t.lut.size());
    cudaError_t e = cudaGetDevice(&cb->device);
    if (e == cudaSuccess) e = cudaMalloc(&cb->d_blob, cb->blob_bytes);
    if (e == cudaSuccess) e = cudaMemcpy(cb->d_blob, blob.data(), cb->blob_bytes, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        set_cuda_error("qamw_codebook_create", int(e));
        if (cb->d_blob) cudaFree(cb->d_blob);
        delete cb;
        return QAMW_ERR_CUDA;
    }
    *out = cb;
    return QAMW_OK;
}

extern "C" void qamw_codebook_destroy(qamw_codebook* cb) {
    if (!cb) return;
    if (cb->d_blob) cudaFree(cb->d_blob);
    delete cb;
}

extern "C" int qamw_codebook_table_info(const qamw_codebook* cb, int32_t* info_out) {
    if (!cb || !info_out) return QAMW_ERR_ARG;
    info_out[0] = cb->grid;
    info_out[1] = cb->n_candidates;
    info_out[2] = cb->max_list;
    info_out[3] = cb->n_overflow_cells;
    info_out[4] = int32_t((cb->off_lut - cb->off_overflow) / 2);
    info_out[5] = int32_t(cb->blob_bytes - size_t(cb->K) * 8);
    return QAMW_OK;
}

extern "C" int qamw_encode(const void* W, const qamw_params* p, const float* chan_scale, const int8_t* signs,
                           const float* sigma, const qamw_codebook* cb, uint8_t* packed_out, float* row_norm_out,
                           int32_t* status_out, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!W || !signs || !sigma || !cb || !packed_out || !row_norm_out) return QAMW_ERR_ARG;
    if (cb->K != p->K) return QAMW_ERR_ARG;
    const size_t row_bytes = qamw_packed_row_bytes(p->d_in, p->K);
    if (p->packed_row_stride < (long long)row_bytes || p->packed_row_stride % 4) return QAMW_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(packed_out) % 4) return QAMW_ERR_ALIGN;
    if (p->d_out == 0) return QAMW_OK;
    EncodeArgs a;
    a.g = make_geom(p, W);
    a.W = W;
    a.chan_scale = chan_scale;
    a.signs = signs;
    a.sigma = sigma;
    a.blob = static_cast<const uint4*>(cb->d_blob);
    a.blob_bytes = int(cb->blob_bytes);
    a.off_cells = int(cb->off_cells);
    a.off_overflow = int(cb->off_overflow);
    a.off_lut = int(cb->off_lut);
    a.K = p->K;
    a.log2K = ilog2(p->K);
    a.grid = cb->grid;
    a.brute = (p->flags & QAMW_FLAG_BRUTE_FORCE) ? 1 : 0;
    a.packed = packed_out;
    a.packed_row_stride = p->packed_row_stride;
    a.row_words = int(p->packed_row_stride / 4);
    a.row_norm = row_norm_out;
    a.status = status_out;
    a.idx_stride = ((p->d_in / 2 + 7) / 8) * 8 + 8;
    const size_t smem = ((cb->blob_bytes + 15) & ~size_t(15)) + size_t(a.g.groups) * 64 * sizeof(double) +
                        size_t(a.g.groups) * a.idx_stride * 2;
    if (smem > 227 * 1024) return QAMW_ERR_NOMEM;
    const int blocks = std::max(1, std::min(sm_count(), (p->d_out + a.g.groups - 1) / a.g.groups));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define CALL(LB)                                                                  \
    rc = a.g.w_bf16 ? launch_encode<true, LB>(a, blocks, smem, st) : launch_encode<false, LB>(a, blocks, smem, st)
    QAMW_DISPATCH_LOG2B(a.g.log2b, CALL)
#undef CALL
    return rc;
}

extern "C" int qamw_rotate(const void* W, const qamw_params* p, const float* chan_scale, const int8_t* signs,
                           float* y_out, float* row_norm_out, int32_t* status_out, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!W || !signs || !y_out || !row_norm_out) return QAMW_ERR_ARG;
    if (p->d_out == 0) return QAMW_OK;
    AuxArgs a{};
    a.g = make_geom(p, W);
    a.W = W;
    a.chan_scale = chan_scale;
    a.signs = signs;
    a.mode = 0;
    a.y_out = y_out;
    a.row_norm = row_norm_out;
    a.status = status_out;
    const int blocks = std::max(1, std::min(sm_count(), (p->d_out + a.g.groups - 1) / a.g.groups));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define CALL(LB) rc = a.g.w_bf16 ? launch_aux<true, LB>(a, blocks, st) : launch_aux<false, LB>(a, blocks, st)
    QAMW_DISPATCH_LOG2B(a.g.log2b, CALL)
#undef CALL
    return rc;
}

namespace {
struct CalibPlan {
    int n_rows, blocks, total_groups, pair_stride;
    size_t bytes;
};
CalibPlan calib_plan(const qamw_params* p, const RowGeom& g) {
    CalibPlan c;
    c.n_rows = std::min(p->d_out, QAMW_CALIB_MAX_ROWS);
    c.blocks = std::max(1, std::min(148, (c.n_rows + g.groups - 1) / g.groups));
    c.total_groups = c.blocks * g.groups;
    c.pair_stride = ((p->d_in / 2 + 3) / 4) * 4;
    c.bytes = (size_t(c.total_groups) * c.pair_stride + size_t(c.total_groups)) * sizeof(double);
    return c;
}
}  // namespace

extern "C" size_t qamw_calibrate_workspace_bytes(const qamw_params* p) {
    if (check_params(p)) return 0;
    RowGeom g = make_geom(p, nullptr);
    return calib_plan(p, g).bytes;
}

extern "C" int qamw_calibrate(const void* W, const qamw_params* p, const float* chan_scale, const int8_t* signs,
                              float* sigma_out, void* workspace, size_t workspace_bytes, int32_t* status_out,
                              void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!W || !signs || !sigma_out || !workspace) return QAMW_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % 8) return QAMW_ERR_ALIGN;
    AuxArgs a{};
    a.g = make_geom(p, W);
    const CalibPlan c = calib_plan(p, a.g);
    if (workspace_bytes < c.bytes) return QAMW_ERR_NOMEM;
    a.W = W;
    a.chan_scale = chan_scale;
    a.signs = signs;
    a.mode = 1;
    a.n_calib_rows = c.n_rows;
    a.partial = static_cast<double*>(workspace);
    a.pair_stride = c.pair_stride;
    a.status = status_out;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define CALL(LB) rc = a.g.w_bf16 ? launch_aux<true, LB>(a, c.blocks, st) : launch_aux<false, LB>(a, c.blocks, st)
    QAMW_DISPATCH_LOG2B(a.g.log2b, CALL)
#undef CALL
    if (rc) return rc;
    const int n_pairs = p->d_in / 2;
    calibrate_finish_kernel<<<(n_pairs + 127) / 128, 128, 0, st>>>(a.partial, c.total_groups, c.pair_stride, n_pairs,
                                                                    p->d_in, sigma_out);
    return finish_launch("calibrate_finish_kernel");
}

// ---------------------------------------------------------------------------------------------
// calibration for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------------

// Scratch of qamw_calibrate_static.  It is part of the library image: every device that loads the
// library holds these bytes until the process exits.  In host code the name below is only a handle
// for cudaGetSymbolAddress; it is never passed to a kernel as if it were a device address.
static __device__ __align__(256) unsigned char g_static_calib_scratch[QAMW_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_scratch_mutex;
void* g_static_scratch_ptr[kMaxDevices] = {};  // device address of the array, per device ordinal
}  // namespace

extern "C" int qamw_calibrate_static(const void* W, const qamw_params* p, const float* chan_scale,
                                     const int8_t* signs, float* sigma_out, int32_t* status_out, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    const size_t need = qamw_calibrate_workspace_bytes(p);
    if (need > size_t(QAMW_STATIC_SCRATCH_BYTES)) {
        std::snprintf(g_last_error, sizeof(g_last_error),
                      "qamw_calibrate_static: this shape needs %zu bytes of scratch, the built-in array holds %zu",
                      need, size_t(QAMW_STATIC_SCRATCH_BYTES));
        return QAMW_ERR_NOMEM;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_cuda_error("qamw_calibrate_static: cudaGetDevice", int(e == cudaSuccess ? cudaErrorInvalidDevice : e));
        return QAMW_ERR_CUDA;
    }
    void* scratch = nullptr;
    {
        // first call on this device: look up where the array lives in this device's memory
        std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
        if (!g_static_scratch_ptr[dev]) {
            void* ptr = nullptr;
            e = cudaGetSymbolAddress(&ptr, g_static_calib_scratch);
            if (e != cudaSuccess || !ptr) {
                set_cuda_error("qamw_calibrate_static: cudaGetSymbolAddress", int(e));
                return QAMW_ERR_CUDA;
            }
            g_static_scratch_ptr[dev] = ptr;
        }
        scratch = g_static_scratch_ptr[dev];
    }
    // Nothing in the scratch has to start at zero: every word the reduction reads is written
    // earlier in the same call, so the previous call's contents are simply overwritten.
    return qamw_calibrate(W, p, chan_scale, signs, sigma_out, scratch, size_t(QAMW_STATIC_SCRATCH_BYTES), status_out,
                          stream);
}

extern "C" int qamw_decode(const uint8_t* packed, const float* row_norm, const float* chan_scale, const int8_t* signs,
                           const float* sigma, const qamw_codebook* cb, const qamw_params* p, void* w_hat_bf16_out,
                           void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!packed || !row_norm || !signs || !sigma || !cb || !w_hat_bf16_out) return QAMW_ERR_ARG;
    if (cb->K != p->K) return QAMW_ERR_ARG;
    const size_t row_bytes = qamw_packed_row_bytes(p->d_in, p->K);
    if (p->packed_row_stride < (long long)row_bytes || p->packed_row_stride % 4) return QAMW_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(packed) % 4 || reinterpret_cast<uintptr_t>(w_hat_bf16_out) % 2) return QAMW_ERR_ALIGN;
    if (p->d_out == 0) return QAMW_OK;
    DecodeArgs a;
    a.g = make_geom(p, nullptr);
    a.g.vec = (p->d_in % 8 == 0) && (reinterpret_cast<uintptr_t>(w_hat_bf16_out) % 16 == 0);
    a.packed = packed;
    a.packed_row_stride = p->packed_row_stride;
    a.row_words = int(p->packed_row_stride / 4);
    a.row_norm = row_norm;
    a.chan_scale = chan_scale;
    a.signs = signs;
    a.sigma = sigma;
    a.codebook = static_cast<const float2*>(cb->d_blob);
    a.K = p->K;
    a.log2K = ilog2(p->K);
    a.out = static_cast<__nv_bfloat16*>(w_hat_bf16_out);
    const size_t smem = size_t(p->K) * 8;
    const int blocks = std::max(1, std::min(sm_count(), (p->d_out + a.g.groups - 1) / a.g.groups));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define CALL(LB) rc = launch_decode<LB>(a, blocks, smem, st)
    QAMW_DISPATCH_LOG2B(a.g.log2b, CALL)
#undef CALL
    return rc;
}

extern "C" int qamw_distortion(const void* W, const void* w_hat_bf16, const float* act_rms, const qamw_params* p,
                               double* out4, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!W || !w_hat_bf16 || !out4) return QAMW_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(out4, 0, 4 * sizeof(double), st);
    if (e != cudaSuccess) {
        set_cuda_error("cudaMemsetAsync", int(e));
        return QAMW_ERR_CUDA;
    }
    if (p->d_out == 0) return QAMW_OK;
    const int blocks = std::max(1, std::min(4 * sm_count(), p->d_out));
    if (p->w_dtype == QAMW_DTYPE_BF16)
        distortion_kernel<true><<<blocks, 256, 0, st>>>(W, p->w_row_stride, static_cast<const __nv_bfloat16*>(w_hat_bf16),
                                                        act_rms, p->d_out, p->d_in, out4);
    else
        distortion_kernel<false><<<blocks, 256, 0, st>>>(W, p->w_row_stride, static_cast<const __nv_bfloat16*>(w_hat_bf16),
                                                         act_rms, p->d_out, p->d_in, out4);
    return finish_launch("distortion_kernel");
}
