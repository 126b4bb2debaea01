// CUDA kernels (sm_100a) and device-side entry points of libqamw.
//
// Thread geometry shared by the row kernels (encode, decode, calibrate, rotate).
//   * A row of d_in elements is owned by one "group" of TG threads (whole warps); a thread block
//     holds several groups, each on its own row, and the grid is persistent: rows are strided
//     over all groups of all blocks.
//   * Thread t of a group owns the 32 contiguous elements [32 t, 32 t + 32) of the row as four
//     "octets" of eight elements, kept in registers as 4 x 4 packed f32 pairs, so the thread reads
//     (encode) or writes (decode) 16-byte pieces and the per-column constants of its columns stay
//     in registers for the whole kernel.
//   * Walsh-Hadamard butterflies of a block of b elements: stages h = 1, 2, 4 work inside an octet,
//     h = 8, 16 between the thread's octets, and for b > 32 the stages h = 32 ... b/2 pair the
//     L = b/32 threads of the block (L <= 32, never across warps).  Stages always run in ascending
//     order of h with one f32 rounding per output, which makes the result reproducible bit for bit.
//   * A cross-thread stage is a "half exchange": instead of both threads fetching all 32 partner
//     values, each thread sends two of its octets and receives two, then computes both outputs
//     (a + c, a - c) of the 16 butterflies whose inputs it now holds.  That halves the shuffles;
//     the price is that the stage swaps the roles of a lane bit and an octet-slot bit, so after
//     the rotation a thread holds other octets of the block than before (octet_after()).  For the
//     first two cross stages the threads with the lane bit set load their octets in swapped
//     register slots, which makes "keep slot 0, send slot 1" the same code for both partners.
//   * Shared-memory reads are what limits these kernels on B200 (random 8-byte reads replay on
//     bank conflicts), hence: the codebook is stored in several bank-separated copies and every
//     lane reads the copy of its own banks.
//   * A warp owns 1024 consecutive elements: whole Hadamard blocks and 64*B consecutive bytes of
//     the packed row.  The decoder therefore has no barrier after its prologue, and the warps of
//     an encoder row meet once per row, for the row norm; each warp stages its own piece of the
//     packed row in shared memory.
//   * The encoder's four-candidate search has no branch, so that the sixteen searches of a thread
//     (unrolled) interleave; the kernel is sensitive to the size of that loop body, which is why
//     the rare paths (overflow lists, reach check, exhaustive scan) are kept out of it.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include "qamw_device.cuh"
#include "qamw_internal.h"

namespace qamw {

static thread_local char g_last_error[256] = "";

void set_cuda_error(const char* what, int code) {
    std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(cudaError_t(code)));
}
void set_error_text(const char* text) { std::snprintf(g_last_error, sizeof(g_last_error), "%s", text); }

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

}  // namespace qamw

using namespace qamw;

namespace {

constexpr int kMaxThreads = 512;   // threads per block (register budget: 128 per thread)
constexpr int kMaxGroups = 15;     // named barriers 1..15
constexpr size_t kEncodeStaticSmem = 512;  // the encoder's statically allocated partial sums

struct RowGeom {
    int d_out, d_in;
    int log2b;        // log2 of the Hadamard block
    int tg;           // threads per group (multiple of 32)
    int groups;       // groups per thread block
    int vec;          // rows can be moved with 16-byte accesses
    int cvec;         // per-column constants (channel scales, signs, sigma) can be read with vector loads
    int w_bf16;       // 1 = bf16 weights, 0 = f32
    long long w_row_stride;  // elements
};


// Which octet of the row (in units of 8 elements) sits in register slot r of thread tid_g:
//   octet_before: when the row enters the rotation;  octet_after: after all butterfly stages.
// S = number of cross-thread stages, L = 2^S threads per block.  Cross stage j exchanges on slot
// bit (j & 1); afterwards lane bit j selects bit j of the octet index inside the block and the
// slot bits select its two top bits, so the L threads of a block write L consecutive octets.
template <int LOG2B_T>
struct Layout {
    static constexpr int S = LOG2B_T > 5 ? LOG2B_T - 5 : 0;
    static constexpr int L = 1 << S;
    __device__ static __forceinline__ int octet_before(int tid_g, int r) {
        int flip = 0;
        if (S >= 1) flip |= tid_g & 1;
        if (S >= 2) flip |= tid_g & 2;
        return 4 * tid_g + (r ^ flip);
    }
    __device__ static __forceinline__ int octet_after(int tid_g, int r) {
        if (S == 0) return 4 * tid_g + r;
        const int q = tid_g & (L - 1), blk = tid_g >> S;
        const int hi = (S & 1) ? (((r >> 1) & 1) | ((r & 1) << 1)) : r;
        return blk * (4 * L) + q + L * hi;
    }
};

// Unnormalised Walsh-Hadamard butterfly of the thread's 4 x 8 elements and, for blocks wider
// than 32, of the L threads of the block; stages in ascending order.  LOG2B_T >= 5: block size
// 2^LOG2B_T known at compile time; LOG2B_T == 0: block size 2^log2b_rt <= 16 given at run time.
// P[r][i] holds elements (2i, 2i+1) of the octet in slot r.
template <int LOG2B_T, bool FIRST_STAGE_DONE = false>
__device__ __forceinline__ void fwht_regs(f32x2 (&P)[4][4], int log2b_rt, int tid_g) {
    typedef Layout<LOG2B_T> Lay;
    const int log2b = LOG2B_T ? LOG2B_T : log2b_rt;
    if (log2b >= 1 && !FIRST_STAGE_DONE) {  // h = 1: inside a packed pair
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float a, c;
                unpack2(P[r][i], a, c);
                P[r][i] = pack2(__fadd_rn(a, c), __fsub_rn(a, c));
            }
    }
    if (log2b >= 2) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            bfly2(P[r][0], P[r][1]);
            bfly2(P[r][2], P[r][3]);
        }
    }
    if (log2b >= 3) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            bfly2(P[r][0], P[r][2]);
            bfly2(P[r][1], P[r][3]);
        }
    }
    // h = 8, 16: between the octets of the thread.  A thread whose slots are swapped for the
    // first (second) cross stage holds the upper octet in the lower slot, so its sum and
    // difference change places: out_lo = s*lo + hi, out_hi = lo - s*hi with s = -1 (an fma with
    // +-1 rounds exactly like the add or subtract it stands for).
    const float s0 = (Lay::S >= 1 && (tid_g & 1)) ? -1.0f : 1.0f;
    const float s1 = (Lay::S >= 2 && (tid_g & 2)) ? -1.0f : 1.0f;
    if (log2b >= 4) {
        const f32x2 sp = pack2(s0, s0), sn = pack2(-s0, -s0);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f32x2 a = P[0][i], c = P[1][i];
            P[0][i] = fma2(a, sp, c);
            P[1][i] = fma2(c, sn, a);
            a = P[2][i];
            c = P[3][i];
            P[2][i] = fma2(a, sp, c);
            P[3][i] = fma2(c, sn, a);
        }
    }
    if (log2b >= 5) {
        const f32x2 sp = pack2(s1, s1), sn = pack2(-s1, -s1);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f32x2 a = P[0][i], c = P[2][i];
            P[0][i] = fma2(a, sp, c);
            P[2][i] = fma2(c, sn, a);
            a = P[1][i];
            c = P[3][i];
            P[1][i] = fma2(a, sp, c);
            P[3][i] = fma2(c, sn, a);
        }
    }
    // Cross-thread stages j = 0 .. S-1 (h = 32 << j), partner lane = lane ^ (1 << j).
    // j = 0: slots {0,2} are kept and {1,3} sent; the upper thread loaded its octets swapped, so
    // this is the same code for both partners.  The sender multiplies by its own sign s, which is
    // minus the receiver's: with v = -s_r * partner, keep + partner = fma(v, -s_r, keep) and the
    // difference (lower thread: keep - partner, upper thread: partner - keep) = fma(keep, s_r, v).
    if (Lay::S >= 1) {
        const f32x2 sp = pack2(s0, s0), sn = pack2(-s0, -s0);
#pragma unroll
        for (int rr = 0; rr < 4; rr += 2)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const f32x2 keep = P[rr][i];
                const f32x2 v = shfl_xor2(mul2(P[rr + 1][i], sp), 1);
                P[rr][i] = fma2(v, sn, keep);
                P[rr + 1][i] = fma2(keep, sp, v);
            }
    }
    if (Lay::S >= 2) {  // j = 1: slots {0,1} kept, {2,3} sent
        const f32x2 sp = pack2(s1, s1), sn = pack2(-s1, -s1);
#pragma unroll
        for (int rr = 0; rr < 2; ++rr)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const f32x2 keep = P[rr][i];
                const f32x2 v = shfl_xor2(mul2(P[rr + 2][i], sp), 2);
                P[rr][i] = fma2(v, sn, keep);
                P[rr + 2][i] = fma2(keep, sp, v);
            }
    }
#pragma unroll
    for (int j = 2; j < Lay::S; ++j) {  // later stages: kept and sent slots are selected per thread
        const bool upper = (tid_g >> j) & 1;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int ra = (j & 1) ? t : 2 * t;            // slot with partition bit 0
            const int rb = (j & 1) ? t + 2 : 2 * t + 1;    // slot with partition bit 1
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const f32x2 keep = upper ? P[rb][i] : P[ra][i];
                const f32x2 send = upper ? P[ra][i] : P[rb][i];
                const f32x2 got = shfl_xor2(send, 1 << j);
                const f32x2 a = upper ? got : keep, c = upper ? keep : got;
                P[ra][i] = add2(a, c);
                P[rb][i] = sub2(a, c);
            }
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
    for (int r = 0; r < 4; ++r) {
        const int e0 = 8 * Layout<LOG2B_T>::octet_before(tid_g, r);
        if (g.vec) {
            if (e0 < g.d_in) {
                const uint4* p = reinterpret_cast<const uint4*>(base + size_t(e0) * (BF16 ? 2 : 4));
                if (BF16) {
                    raw.v[r] = __ldg(p);
                } else {
                    raw.v[2 * r] = __ldg(p);
                    raw.v[2 * r + 1] = __ldg(p + 1);
                }
            } else {
                if (BF16) {
                    raw.v[r] = make_uint4(0, 0, 0, 0);
                } else {
                    raw.v[2 * r] = make_uint4(0, 0, 0, 0);
                    raw.v[2 * r + 1] = make_uint4(0, 0, 0, 0);
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
                raw.v[r] = make_uint4(w[0] | (w[1] << 16), w[2] | (w[3] << 16), w[4] | (w[5] << 16), w[6] | (w[7] << 16));
            } else {
                raw.v[2 * r] = make_uint4(w[0], w[1], w[2], w[3]);
                raw.v[2 * r + 1] = make_uint4(w[4], w[5], w[6], w[7]);
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


// Raw per-column inputs of the encoder side for the octets a thread holds when the row is loaded.
struct ColRaw {
    float cs[4][8];   // channel scales (1 when there are none)
    float sgn[4][8];  // signs, 0 beyond the row
};
template <int LOG2B_T>
__device__ __forceinline__ void load_col_raw(ColRaw& c, const float* chan_scale, const int8_t* signs, int d_in,
                                             int cvec, int tid_g) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int e0 = 8 * Layout<LOG2B_T>::octet_before(tid_g, r);
        if (chan_scale) {
            load8f(chan_scale, e0, d_in, cvec, 1.0f, c.cs[r]);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) c.cs[r][e] = 1.0f;
        }
        load8s(signs, e0, d_in, cvec, c.sgn[r]);
    }
}
// t_j = f32(s_j) * sign_j (0 beyond the row)
__device__ __forceinline__ void col_factors(const ColRaw& c, f32x2 (&t)[4][4]) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int i = 0; i < 4; ++i) t[r][i] = pack2(c.cs[r][2 * i] * c.sgn[r][2 * i], c.cs[r][2 * i + 1] * c.sgn[r][2 * i + 1]);
}

// Scaling, row norm and butterfly of one row held in registers (the arithmetic contract of the
// encoder, steps x, r, h).  Returns the row norm r; P holds the unnormalised butterfly output in
// the layout of octet_after().  `red` is this group's reduction scratch (one double per warp, two
// buffers).
template <bool BF16, int LOG2B_T>
__device__ __forceinline__ float front_half(const RawRow<BF16>& raw, const f32x2 (&t)[4][4], f32x2 (&P)[4][4],
                                            const RowGeom& g, int group, int tid_g, double* red, int parity,
                                            float& gn_out) {
    float x[4][8];
    raw_to_float<BF16>(raw, x);
    double ss = 0.0;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            P[r][i] = mul2(pack2(x[r][2 * i], x[r][2 * i + 1]), t[r][i]);
            float a, c;
            unpack2(P[r][i], a, c);
            const double ad = double(a), cd = double(c);
            ss = fma(ad, ad, ss);
            ss = fma(cd, cd, ss);
        }
    fwht_regs<LOG2B_T>(P, g.log2b, tid_g);
    ss = warp_sum(ss);
    const int n_warps = g.tg >> 5;
    double* slot = red + parity * 32;
    if ((tid_g & 31) == 0) slot[tid_g >> 5] = ss;
    group_barrier(group, g.tg);
    // one thread of the group turns the warp sums into r and g = f32(c_b / r), c_b = f32(1/sqrt(b)) (g = 0 for a
    // zero or non-finite row); the others pick both up after a second barrier
    float2* rg = reinterpret_cast<float2*>(slot + 16);
    if (tid_g == 0) {
        double total = 0.0;
        for (int w = 0; w < n_warps; ++w) total += slot[w];
        const float r = float(sqrt(total));
        const float gn = (isfinite(r) && r > 0.f) ? __fdiv_rn(float(1.0 / sqrt(double(1 << g.log2b))), r) : 0.f;
        *rg = make_float2(r, gn);
    }
    group_barrier(group, g.tg);
    const float2 v = *rg;
    gn_out = v.y;
    return v.x;
}



// Index staging: the 4 indices of an octet are staged as one 64-bit value (index p at bits
// [p*B, (p+1)*B)).  Octet o sits in 8-byte slot o + 4*(o/16): the 32 bytes of padding after every
// 16 octets keep the stores of a warp (eight runs of 32 bytes, 128 bytes apart) on distinct banks.
__device__ __forceinline__ int stage_slot(int o) { return o + ((o >> 4) << 2); }

// ---------------------------------------------------------------------------------------------
// encode kernel
// ---------------------------------------------------------------------------------------------

struct EncodeArgs {
    RowGeom g;
    const void* W;
    const float* chan_scale;
    const int8_t* signs;
    const float* sigma;
    const float2* codebook;  // device, K entries
    const uint4* table;      // cells | overflow, as laid out by qamw_codebook_create
    int table_bytes;         // a multiple of 16
    int off_overflow;        // byte offset inside the table
    int K, log2K, grid;
    float map_zmax, map_c0, map_c1, map_c2, map_bias;  // the cell map of the table
    int log2c;               // log2 of the number of codebook copies in shared memory
    int brute;
    float inv_sqrt_b;        // c_b = f32(1 / sqrt(b))
    uint8_t* packed;
    long long packed_row_stride;  // bytes
    int row_words;           // 32-bit words per packed row (stride / 4)
    int payload_words;       // words that hold index bits: ceil(row payload bytes / 4)
    float* row_norm;         // out: r_i
    int32_t* status;         // out (optional): bit 0 set when a row norm is not finite
};

constexpr int kStageSlotsPerWarp = 128 + 4 * 8;  // 128 octets of a warp plus their padding

// Encoder.  A warp owns 1024 consecutive elements of a row (whole Hadamard blocks): it rotates
// them with shuffles, searches its 512 pairs, stages the indices in its own piece of shared
// memory and writes its 64*B bytes of the packed row.  The warps of a row share one thing, the
// row norm: each adds its partial sum of squares to shared memory and they meet at one named
// barrier per row, after the rotation.  W is read once.
template <bool BF16, int LOG2B_T>
__global__ void __launch_bounds__(kMaxThreads, 1) encode_kernel(const EncodeArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ double ss_part[2][32];  // per-warp partial sums of squares, two rows in flight
    const RowGeom& g = a.g;
    // dynamic shared memory: [codebook copies][table][index staging: one piece per warp]
    const int group = threadIdx.x / g.tg;
    const int tid_g = threadIdx.x - group * g.tg;
    const int lane = threadIdx.x & 31;
    const int n_pairs = g.d_in >> 1;
    // all global loads of the prologue are issued before anything waits for one of them
    ColRaw craw;
    load_col_raw<LOG2B_T>(craw, a.chan_scale, a.signs, g.d_in, g.cvec, tid_g);
    int k0s[4];
    float q[4][4];  // pair positions and reciprocal pair scales of the octets held after the rotation
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        k0s[r] = 4 * Layout<LOG2B_T>::octet_after(tid_g, r);
        load4f(a.sigma, k0s[r], n_pairs, g.cvec, 1.0f, q[r]);
    }
    const int cb_bytes = (a.K * 8) << a.log2c;
    fill_codebook_copies(reinterpret_cast<float2*>(smem), a.codebook, a.K, a.log2c);
    unsigned char* table = smem + cb_bytes;
    {
        uint4* dst = reinterpret_cast<uint4*>(table);
        const int n16 = a.table_bytes / 16;
        for (int base = 0; base < n16; base += 8 * blockDim.x) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = base + u * blockDim.x + threadIdx.x;
                if (i < n16) v[u] = __ldg(a.table + i);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = base + u * blockDim.x + threadIdx.x;
                if (i < n16) dst[i] = v[u];
            }
        }
    }
    const int table_pad = (a.table_bytes + 15) & ~15;
    unsigned long long* oct_s =
        reinterpret_cast<unsigned long long*>(table + table_pad) + size_t(threadIdx.x >> 5) * kStageSlotsPerWarp;

    f32x2 t[4][4];
    col_factors(craw, t);
    // q_k = f32(1 / (double)sigma_k): the correctly rounded f32 reciprocal is the same number (the
    // exact quotient of two f32 is never within 2^-53 of an f32 rounding boundary unless it is exact)
    bool risky = false;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            q[r][p] = (k0s[r] + p < n_pairs) ? __frcp_rn(q[r][p]) : 0.f;
            // |z| <= q (1 + eps) because |y| <= 1 for a unit row: only a huge reciprocal pair scale
            // can carry a point beyond the table's reach
            risky |= !(q[r][p] < 15000.0f);
        }
    const int any_risky = __syncthreads_or(risky ? 1 : 0);  // also the prologue's barrier

    SearchSmem s;
    s.cb = smem_addr(smem) + 8u * (threadIdx.x & ((1 << a.log2c) - 1));
    s.cb_stride = 8u << a.log2c;
    s.cells = smem_addr(table) - 8u * kMagicBits * uint32_t(a.grid + 1);
    s.overflow = smem_addr(table + a.off_overflow);
    s.grid = uint32_t(a.grid);
    s.K = a.K;
    s.zlo = pack2(-a.map_zmax, -a.map_zmax);
    s.c0 = pack2(a.map_c0, a.map_c0);
    s.c1 = pack2(a.map_c1, a.map_c1);
    s.c2 = pack2(a.map_c2, a.map_c2);
    s.bias = pack2(a.map_bias, a.map_bias);

    const long long row_step = (long long)gridDim.x * g.groups;
    const int B = a.log2K, B4 = 4 * a.log2K;
    const unsigned div_magic = 0xffffffffu / unsigned(B4) + 1u;  // ceil(2^32 / (4B))
    const int n_oct = (n_pairs + 3) >> 2;
    const int warp_g = tid_g >> 5;                 // segment of the row this warp owns
    const int oct0 = 128 * warp_g;                 // its first octet
    const int seg_word0 = 16 * B * warp_g;         // its first packed word (64*B bytes per segment)
    const bool last_seg = (warp_g + 1) * 1024 >= g.d_in;
    const int n_warps = g.tg >> 5;

    // The row loop exists in three variants chosen once per block, so that the common one carries
    // no call to the rarely needed searches: 0 = table search, 1 = table search with the reach
    // check, 2 = exhaustive search.
    auto rows = [&](auto mode_tag) {
        constexpr int MODE = decltype(mode_tag)::value;
        int parity = 0;
        for (long long row = (long long)blockIdx.x * g.groups + group; row < g.d_out; row += row_step, parity ^= 1) {
            RawRow<BF16> raw;
            load_row<BF16, LOG2B_T>(raw, a.W, row, g, tid_g);
            f32x2 P[4][4];
            {
                float x[4][8];
                raw_to_float<BF16>(raw, x);
#pragma unroll
                for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                    for (int i = 0; i < 4; ++i) P[rr][i] = mul2(pack2(x[rr][2 * i], x[rr][2 * i + 1]), t[rr][i]);
            }
            // sum of squares of the row: ss = sum_j (double)x_j^2, per thread, per warp, then per row
            double* part = &ss_part[parity][threadIdx.x >> 5] - warp_g;  // the row's per-warp sums
            {
                double ss = 0.0;
#pragma unroll
                for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float p, c;
                        unpack2(P[rr][i], p, c);
                        const double pd = double(p), cd = double(c);
                        ss = fma(pd, pd, ss);
                        ss = fma(cd, cd, ss);
                    }
                ss = warp_sum(ss);
                if (lane == 0) part[warp_g] = ss;
            }
            // The rotation does not need the norm, so the warps of the row meet only after it.  A
            // warp can be one row ahead of another at most, hence the two sets of partial sums.
            fwht_regs<LOG2B_T>(P, g.log2b, tid_g);
            group_barrier(group, g.tg);
            float gn = 0.f;
            if (lane == 0) {  // every warp adds the same numbers in the same order
                double total = 0.0;
                for (int w = 0; w < n_warps; ++w) total += part[w];
                const float r = float(sqrt(total));
                // g = f32(c_b / r); 0 for a zero row (all its pairs become the origin, 0 * 0) and for a
                // non-finite row (its indices are unspecified; the searches accept any input)
                if (isfinite(r) && r > 0.f) gn = __fdiv_rn(a.inv_sqrt_b, r);
                if (warp_g == 0) {
                    a.row_norm[row] = r;
                    if (!isfinite(r) && a.status) atomicOr(a.status, 1);
                }
            }
            gn = __shfl_sync(kFull, gn, 0);
            const f32x2 gn2 = pack2(gn, gn);
            // The sixteen points of the thread stay in the registers of the rotation; the search is
            // unrolled over the four octets (the branch-free search is compact enough for that: with a
            // branch per point the unrolled loop did not fit the instruction cache).
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    float yx, yy;
                    unpack2(mul2(P[rr][p], gn2), yx, yy);
                    P[rr][p] = pack2(__fmul_rn(yx, q[rr][p]), __fmul_rn(yy, q[rr][p]));
                }
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
                const int k0 = 4 * Layout<LOG2B_T>::octet_after(tid_g, rr);
                uint32_t v[4];
                if (MODE == 0) {
                    uint2 rec[4];
                    float2 z[4];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        unpack2(P[rr][p], z[p].x, z[p].y);
                        v[p] = uint32_t(search_cell(s, z[p].x, z[p].y, rec[p]));
                    }
                    // rare: one of the four cells has more than four candidates
                    if (cell_overflows(rec[0]) || cell_overflows(rec[1]) || cell_overflows(rec[2]) || cell_overflows(rec[3])) {
#pragma unroll
                        for (int p = 0; p < 4; ++p)
                            if (cell_overflows(rec[p])) v[p] = uint32_t(search_overflow(s, rec[p], z[p].x, z[p].y));
                    }
                } else {
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        float2 z;
                        unpack2(P[rr][p], z.x, z.y);
                        v[p] = uint32_t(MODE == 2 ? search_exhaustive(s, z.x, z.y) : search_table(s, z.x, z.y));
                    }
                }
                // two indices fit a 32-bit word (B <= 12)
                unsigned long long packed4 =
                    (unsigned long long)(v[0] | (v[1] << B)) | ((unsigned long long)(v[2] | (v[3] << B)) << (2 * B));
                if (k0 < n_pairs) {
                    if (k0 + 4 > n_pairs) packed4 &= (1ull << ((n_pairs - k0) * B)) - 1ull;  // the row ends inside this octet
                    oct_s[stage_slot((k0 >> 2) - oct0)] = packed4;
                }
            }
            __syncwarp();
            // bit packing of the warp's segment: octet o occupies bits [o*4B, (o+1)*4B) (LSB first)
            uint32_t* out = reinterpret_cast<uint32_t*>(a.packed + row * a.packed_row_stride);
            for (int j = lane; j < 16 * B; j += 32) {
                const int gw = seg_word0 + j;
                if (gw >= a.payload_words) break;
                const unsigned bit0 = unsigned(j) * 32u;
                int o = int(__umulhi(bit0, div_magic));  // floor(bit0 / (4B)), local octet
                uint32_t word;
                if (B4 >= 32) {
                    // an octet is at least as wide as a word: the word takes bits from octet o and,
                    // if it reaches past it, from octet o + 1 (slots past the row read as garbage
                    // only into bits that the caller's row payload does not contain)
                    const int sh = int(bit0) - o * B4;  // 0 <= sh < 4B
                    const unsigned long long v0 = oct_s[stage_slot(o)];
                    const unsigned long long v1 = (o + 1 < 128 && oct0 + o + 1 < n_oct) ? oct_s[stage_slot(o + 1)] : 0ull;
                    word = uint32_t(v0 >> sh) | uint32_t((v1 << (B4 - sh)) & 0xffffffffull);
                } else {
                    word = 0;
                    for (; oct0 + o < n_oct; ++o) {
                        const int sh = o * B4 - int(bit0);
                        if (sh >= 32) break;
                        const unsigned long long v = oct_s[stage_slot(o)];
                        word |= sh >= 0 ? uint32_t(v << sh) : uint32_t(v >> (-sh));
                    }
                }
                out[gw] = word;
            }
            if (last_seg)  // padding up to the row stride is written as zero
                for (int gw = a.payload_words + lane; gw < a.row_words; gw += 32) out[gw] = 0u;
            __syncwarp();  // the staging piece is free again
        }
    };
    if (a.brute) rows(std::integral_constant<int, 2>{});
    else if (any_risky) rows(std::integral_constant<int, 1>{});
    else rows(std::integral_constant<int, 0>{});
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
    double* partial;         // [total_groups][pair_stride] sums, then [total_groups] used-row counts
    int pair_stride;
    int32_t* status;
};

template <bool BF16, int LOG2B_T>
__global__ void __launch_bounds__(kMaxThreads, 1) aux_kernel(const AuxArgs a) {
    __shared__ double red_all[kMaxGroups * 64];
    const RowGeom& g = a.g;
    const int group = threadIdx.x / g.tg;
    const int tid_g = threadIdx.x - group * g.tg;
    double* red = red_all + group * 64;
    const int n_pairs = g.d_in >> 1;

    f32x2 t[4][4];
    {
        ColRaw craw;
        load_col_raw<LOG2B_T>(craw, a.chan_scale, a.signs, g.d_in, g.cvec, tid_g);
        col_factors(craw, t);
    }
    int e0s[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) e0s[r] = 8 * Layout<LOG2B_T>::octet_after(tid_g, r);
    const bool y_vec = (g.d_in % 8 == 0) && (reinterpret_cast<uintptr_t>(a.y_out) % 16 == 0);

    const int n_rows = a.mode == 1 ? a.n_calib_rows : g.d_out;
    const long long total_groups = (long long)gridDim.x * g.groups;
    const long long my_group = (long long)blockIdx.x * g.groups + group;
    double acc[4][4];
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[m][p] = 0.0;
    int used = 0;

    RawRow<BF16> raw;
    if (my_group < n_rows) {
        const long long row = a.mode == 1 ? (my_group * g.d_out) / a.n_calib_rows : my_group;
        load_row<BF16, LOG2B_T>(raw, a.W, row, g, tid_g);
    }
    int parity = 0;
    for (long long it = my_group; it < n_rows; it += total_groups, parity ^= 1) {
        const long long row = a.mode == 1 ? (it * g.d_out) / a.n_calib_rows : it;
        RawRow<BF16> nxt;
        const long long it_next = it + total_groups;
        if (it_next < n_rows) {
            const long long row_next = a.mode == 1 ? (it_next * g.d_out) / a.n_calib_rows : it_next;
            load_row<BF16, LOG2B_T>(nxt, a.W, row_next, g, tid_g);
        }
        f32x2 P[4][4];
        float gn;
        const float r = front_half<BF16, LOG2B_T>(raw, t, P, g, group, tid_g, red, parity, gn);
        if (!isfinite(r) && a.status && tid_g == 0) atomicOr(a.status, 1);
        const f32x2 gn2 = pack2(gn, gn);
        if (a.mode == 0) {
            if (tid_g == 0) a.row_norm[row] = r;
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
                if (e0s[rr] >= g.d_in) continue;
                float y[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) unpack2(mul2(P[rr][i], gn2), y[2 * i], y[2 * i + 1]);
                float* dst = a.y_out + row * g.d_in + e0s[rr];
                if (y_vec) {
                    reinterpret_cast<float4*>(dst)[0] = make_float4(y[0], y[1], y[2], y[3]);
                    reinterpret_cast<float4*>(dst)[1] = make_float4(y[4], y[5], y[6], y[7]);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (e0s[rr] + e < g.d_in) dst[e] = y[e];
                }
            }
        } else if (gn != 0.f) {
            ++used;
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    float y0, y1;
                    unpack2(mul2(P[rr][p], gn2), y0, y1);
                    acc[rr][p] += double(sqrtf(__fmaf_rn(y1, y1, __fmul_rn(y0, y0))));
                }
        }
        raw = nxt;
    }
    if (a.mode == 1) {
        double* mine = a.partial + my_group * a.pair_stride;
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
            const int k0 = e0s[rr] >> 1;
#pragma unroll
            for (int p = 0; p < 4; ++p)
                if (k0 + p < n_pairs) mine[k0 + p] = acc[rr][p];
        }
        if (tid_g == 0) a.partial[total_groups * a.pair_stride + my_group] = double(used);
    }
}

// sigma_k from the per-group partial sums.  A block owns 32 pair positions; its 32 warps each add
// a contiguous slice of the groups in ascending order (eight loads in flight at a time) and the 32
// slice sums are then added in ascending order, so the result does not depend on timing.
constexpr int kFinishSlices = 32;
__global__ void __launch_bounds__(32 * kFinishSlices) calibrate_finish_kernel(const double* partial, int total_groups,
                                                                            int pair_stride, int n_pairs, int d_in,
                                                                            float* sigma_out) {
    __shared__ double part_sum[kFinishSlices][32], part_used[kFinishSlices];
    const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + lane;
    const int per = (total_groups + kFinishSlices - 1) / kFinishSlices;
    const int g0 = min(total_groups, slice * per), g1 = min(total_groups, g0 + per);
    double sum = 0.0;
    if (k < n_pairs) {
        int gidx = g0;
        for (; gidx + 8 <= g1; gidx += 8) {
            double v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = partial[size_t(gidx + u) * pair_stride + k];
#pragma unroll
            for (int u = 0; u < 8; ++u) sum += v[u];
        }
        for (; gidx < g1; ++gidx) sum += partial[size_t(gidx) * pair_stride + k];
    }
    if (lane == 0) {
        double used = 0.0;
        for (int gidx = g0; gidx < g1; ++gidx) used += partial[size_t(total_groups) * pair_stride + gidx];
        part_used[slice] = used;
    }
    part_sum[slice][lane] = sum;
    __syncthreads();
    if (slice == 0 && k < n_pairs) {
        double s = 0.0, u = 0.0;
        for (int i = 0; i < kFinishSlices; ++i) {
            s += part_sum[i][lane];
            u += part_used[i];
        }
        const double inv_sqrt_d = 1.0 / sqrt(double(d_in));
        double sg = u > 0.0 ? (s / u) / sqrt(1.5707963267948966) : inv_sqrt_d;
        sg = fmax(sg, 1e-4 * inv_sqrt_d);
        sigma_out[k] = float(sg);
    }
}

// ---------------------------------------------------------------------------------------------
// decode kernel
// ---------------------------------------------------------------------------------------------

struct DecodeArgs {
    RowGeom g;               // d_out, d_in, log2b, tg, groups; vec = output rows 16-byte aligned
    const uint8_t* packed;
    long long packed_row_stride;
    int row_bytes;           // bytes of a packed row that may be copied (payload rounded up to the copy size)
    int copy_log2;           // log2 of the async copy size: 4 when rows are 16-byte aligned, else 2
    int seg_bytes;           // packed bytes of the 512 pairs of one warp: 64 * B
    int stage_bytes;         // one staging buffer of a warp: seg_bytes + 16
    float inv_sqrt_b;        // f32(1 / sqrt(b))
    const float* row_norm;
    const float* chan_scale;
    const int8_t* signs;
    const float* sigma;
    const float2* codebook;  // device, K entries
    int K, log2K;
    int log2c;               // log2 of the number of codebook copies in shared memory
    __nv_bfloat16* out;
};


// A warp owns 1024 consecutive elements of its row, i.e. 512 pairs = 64*B consecutive bytes of the
// packed row (a multiple of 16 for every B).  Each warp streams that segment through its own
// two-deep shared-memory ring: while a row is decoded the next one is on its way, and since
// nothing is shared between warps the kernel has no barrier after its prologue.
template <int LOG2B_T>
__global__ void __launch_bounds__(kMaxThreads, 1) decode_kernel(const DecodeArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    const RowGeom& g = a.g;
    const int group = threadIdx.x / g.tg;
    const int tid_g = threadIdx.x - group * g.tg;
    const int lane = threadIdx.x & 31;
    const int n_pairs = g.d_in >> 1;
    const int B = a.log2K;
    const uint32_t mask = (1u << B) - 1u;
    const uint32_t cb_stride = 8u << a.log2c;
    const uint32_t cb = smem_addr(smem) + 8u * (threadIdx.x & ((1 << a.log2c) - 1));
    unsigned char* stage = smem + ((size_t(a.K) * 8) << a.log2c) + size_t(threadIdx.x >> 5) * 2 * a.stage_bytes;

    // first row on its way before anything else
    const long long seg_off = (long long)(tid_g >> 5) * a.seg_bytes;  // of this warp's segment inside a packed row
    const int seg_len = int(max(0LL, min((long long)a.seg_bytes, (long long)a.row_bytes - seg_off)));
    const int n_chunks = seg_len >> a.copy_log2;
    auto issue_row = [&](long long row, int buf) {
        const unsigned char* src = a.packed + row * a.packed_row_stride + seg_off;
        unsigned char* dst = stage + buf * a.stage_bytes;
        for (int c = lane; c < n_chunks; c += 32)
            cp_async(dst + (size_t(c) << a.copy_log2), src + (size_t(c) << a.copy_log2), a.copy_log2);
        cp_async_commit();
    };
    const long long row_step = (long long)gridDim.x * g.groups;
    long long row = (long long)blockIdx.x * g.groups + group;
    if (row < g.d_out) issue_row(row, 0);
    // the 16 bytes after a staged segment are read (and masked away) by the last windows: keep them defined
    if (lane < 8) reinterpret_cast<uint32_t*>(stage + (lane >> 2) * a.stage_bytes + a.seg_bytes)[lane & 3] = 0u;

    // Input side: window position and pair scales of the octets in the slots before the rotation.
    // Output side: element offsets and factors sign_j / (s_j sqrt(b)) of the slots after it.
    // The global loads of these constants and of the codebook are all issued before the first use.
    int e_out[4], w0s[4], shs[4];
    bool live[4];
    float sg[4][4];
    float cs[4][8], sgn[4][8];
    const int warp_pair0 = (tid_g & ~31) * 16;  // first pair of this warp's segment
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int k0 = 4 * Layout<LOG2B_T>::octet_before(tid_g, r);
        live[r] = k0 < n_pairs;
        const unsigned bit0 = unsigned(k0 - warp_pair0) * unsigned(B);
        w0s[r] = int(bit0 >> 5);
        shs[r] = int(bit0 & 31u);
        e_out[r] = 8 * Layout<LOG2B_T>::octet_after(tid_g, r);
        load4f(a.sigma, k0, n_pairs, g.cvec, 0.f, sg[r]);
        if (a.chan_scale) {
            load8f(a.chan_scale, e_out[r], g.d_in, g.cvec, 1.0f, cs[r]);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) cs[r][e] = 1.0f;
        }
        load8s(a.signs, e_out[r], g.d_in, g.cvec, sgn[r]);
    }
    fill_codebook_copies(reinterpret_cast<float2*>(smem), a.codebook, a.K, a.log2c, true);
    f32x2 mcol[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int i = 0; i < 4; ++i)
            mcol[r][i] = pack2(__fdiv_rn(sgn[r][2 * i] * a.inv_sqrt_b, cs[r][2 * i]),
                               __fdiv_rn(sgn[r][2 * i + 1] * a.inv_sqrt_b, cs[r][2 * i + 1]));
    __syncthreads();

    // The row loop exists twice.  When the rows allow 16-byte accesses (d_in a multiple of 8), octets
    // beyond the end of the row are decoded like the others instead of being tested for: their pair
    // scales are 0, so whatever index the staging buffer holds for them decodes to 0, they belong to
    // Hadamard blocks that lie wholly beyond the row, and only their stores are suppressed.
    auto rows = [&](auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        int buf = 0;
        for (; row < g.d_out; row += row_step, buf ^= 1) {
            const float rn = a.row_norm[row];
            cp_async_wait_all();
            __syncwarp();  // every lane's part of this row has landed; the other buffer is no longer read
            if (row + row_step < g.d_out) issue_row(row + row_step, buf ^ 1);
            const uint32_t* in = reinterpret_cast<const uint32_t*>(stage + buf * a.stage_bytes);
            f32x2 P[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if (FULL || live[r]) {
                    const uint32_t* w = in + w0s[r];
                    const uint32_t lo = w[0], mid = w[1], hi = w[2];
                    // bits [sh, sh+64) of (hi:mid:lo) as two words; pairs 0,1 come from the first word,
                    // pairs 2,3 from the 32 bits that start 2B further on (4B <= 48)
                    const uint32_t a0 = __funnelshift_r(lo, mid, shs[r]), a1 = __funnelshift_r(mid, hi, shs[r]);
                    const uint32_t b0 = __funnelshift_r(a0, a1, 2 * B);
                    const uint32_t id[4] = {a0 & mask, (a0 >> B) & mask, b0 & mask, (b0 >> B) & mask};
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        // pairs past the end of a row whose length is not a multiple of 8 have scale 0
                        const float2 c = lds_f32x2(cb + id[p] * cb_stride);
                        P[r][p] = pack2(c.x * sg[r][p], c.y * sg[r][p]);
                    }
                } else {
#pragma unroll
                    for (int p = 0; p < 4; ++p) P[r][p] = pack2(0.f, 0.f);
                }
            }
            fwht_regs<LOG2B_T, true>(P, g.log2b, tid_g);  // stage h = 1 is already in the stored codewords
            const f32x2 rn2 = pack2(rn, rn);
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int e0 = e_out[r];
                if (!FULL && e0 >= g.d_in) continue;
                __nv_bfloat16* dst = a.out + row * g.d_in + e0;
                uint32_t w[4];
                float y[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    unpack2(mul2(P[r][i], mul2(mcol[r][i], rn2)), y[2 * i], y[2 * i + 1]);
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(y[2 * i], y[2 * i + 1]);
                    w[i] = *reinterpret_cast<uint32_t*>(&h2);
                }
                if (FULL) {  // octets beyond the row are computed like the others and not stored
                    if (e0 < g.d_in) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
                } else if (g.vec) {
                    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (e0 + e < g.d_in) dst[e] = __float2bfloat16_rn(y[e]);
                }
            }
        }
    };
    // block-uniform, so that a block runs one loop body only (two bodies in flight cost more in
    // instruction fetch than the tests save)
    if (g.vec) rows(std::true_type{});
    else rows(std::false_type{});
}

// ---------------------------------------------------------------------------------------------
// distortion kernel
// ---------------------------------------------------------------------------------------------

// A block walks over (row chunk, column tile) work items; a thread owns 8 consecutive columns of
// the tile and accumulates, per column, sum e^2 and sum w^2 over the rows of the chunk in double;
// the activation weights r_j^2 are applied once per column at the end of the chunk.
constexpr int kDistThreads = 128;
constexpr int kDistRows = 16;

template <bool BF16>
__device__ __forceinline__ void dist_load(const void* W, long long w_row_stride, const __nv_bfloat16* What, int row,
                                          int j0, int d_in, int vec, float (&w)[8], float (&h)[8]) {
    const char* wrow = static_cast<const char*>(W) + (long long)row * w_row_stride * (BF16 ? 2 : 4);
    const __nv_bfloat16* hrow = What + (long long)row * d_in;
    if (vec) {
        const uint4 hv = __ldg(reinterpret_cast<const uint4*>(hrow + j0));
        const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            h[2 * i] = __uint_as_float(hw[i] << 16);
            h[2 * i + 1] = __uint_as_float(hw[i] & 0xffff0000u);
        }
        if (BF16) {
            const uint4 wv = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(wrow) + j0));
            const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                w[2 * i] = __uint_as_float(ww[i] << 16);
                w[2 * i + 1] = __uint_as_float(ww[i] & 0xffff0000u);
            }
        } else {
            const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(wrow) + j0);
            const float4 a = __ldg(p), c = __ldg(p + 1);
            w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
            w[4] = c.x; w[5] = c.y; w[6] = c.z; w[7] = c.w;
        }
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const bool in = j0 + e < d_in;
            h[e] = in ? __bfloat162float(hrow[j0 + e]) : 0.f;
            w[e] = !in ? 0.f
                       : (BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(wrow)[j0 + e])
                               : reinterpret_cast<const float*>(wrow)[j0 + e]);
        }
    }
}

__host__ __device__ inline long long dist_item_count(int d_out, int d_in) {
    return (long long)((d_in + 8 * kDistThreads - 1) / (8 * kDistThreads)) * ((d_out + kDistRows - 1) / kDistRows);
}

// bf16 matrices in the 16-byte layout: the rows of a thread's work items form one stream that runs
// through a private shared-memory ring of kDistDepth rows (two 16-byte asynchronous copies per row,
// kDistDepth - 1 rows ahead, across item boundaries).  With the rows held in registers two rows were
// in flight per thread and the kernel waited on memory latency; the ring keeps about 140 KB per SM in
// flight without a register per byte.  A thread reads back only what it copied itself: no barrier.
constexpr int kDistDepth = 8;
struct DistCursor {
    long long item;
    int row, r1, j0;
    bool valid;  // the thread's columns lie inside the matrix
};
__device__ __forceinline__ void dist_cursor_open(DistCursor& c, int d_out, int d_in, int col_tiles) {
    const int chunk = int(c.item / col_tiles), tile = int(c.item - (long long)chunk * col_tiles);
    c.j0 = (tile * kDistThreads + int(threadIdx.x)) * 8;
    c.valid = c.j0 < d_in;
    c.row = chunk * kDistRows;
    c.r1 = min(d_out, c.row + kDistRows);
}
__device__ __forceinline__ void dist_items_stream(const __nv_bfloat16* W, long long w_row_stride, const __nv_bfloat16* What,
                                                  const float* act_rms, int d_out, int d_in, long long first,
                                                  long long last, long long step, double& s0, double& s1, double& s2,
                                                  double& s3) {
    __shared__ uint4 ring[kDistDepth][2][kDistThreads];
    if (first >= last) return;
    const int col_tiles = (d_in + 8 * kDistThreads - 1) / (8 * kDistThreads);
    DistCursor prod, cons;
    prod.item = cons.item = first;
    dist_cursor_open(prod, d_out, d_in, col_tiles);
    cons = prod;
    int issued = 0;
    auto issue = [&]() {  // one commit group per row of the stream, empty past its end
        if (prod.item < last) {
            if (prod.valid) {
                cp_async(&ring[issued % kDistDepth][0][threadIdx.x], W + (long long)prod.row * w_row_stride + prod.j0, 4);
                cp_async(&ring[issued % kDistDepth][1][threadIdx.x], What + (long long)prod.row * d_in + prod.j0, 4);
            }
            if (++prod.row == prod.r1) {
                prod.item += step;
                if (prod.item < last) dist_cursor_open(prod, d_out, d_in, col_tiles);
            }
        }
        ++issued;
        cp_async_commit();
    };
    for (int i = 0; i < kDistDepth - 1; ++i) issue();
    double E[8], Q[8];
    float rj[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) E[e] = Q[e] = 0.0;
    bool fresh = true;
    for (int taken = 0; cons.item < last; ++taken) {
        if (fresh) {  // the activation weights of this item's columns, needed when the item ends
#pragma unroll
            for (int e = 0; e < 8; ++e) rj[e] = act_rms && cons.valid ? __ldg(act_rms + cons.j0 + e) : 1.0f;
            fresh = false;
        }
        asm volatile("cp.async.wait_group %0;" ::"n"(kDistDepth - 2) : "memory");
        const uint4 wv = ring[taken % kDistDepth][0][threadIdx.x], hv = ring[taken % kDistDepth][1][threadIdx.x];
        issue();  // refills the slot read one row ago
        if (cons.valid) {
            const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w}, hw[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const double w0 = double(__uint_as_float(ww[i] << 16)), w1 = double(__uint_as_float(ww[i] & 0xffff0000u));
                const double d0 = w0 - double(__uint_as_float(hw[i] << 16));
                const double d1 = w1 - double(__uint_as_float(hw[i] & 0xffff0000u));
                E[2 * i] = fma(d0, d0, E[2 * i]);
                Q[2 * i] = fma(w0, w0, Q[2 * i]);
                E[2 * i + 1] = fma(d1, d1, E[2 * i + 1]);
                Q[2 * i + 1] = fma(w1, w1, Q[2 * i + 1]);
            }
        }
        if (++cons.row == cons.r1) {  // end of the item: weight the column sums and start over
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const double r2 = double(rj[e]) * double(rj[e]);
                s0 += E[e];
                s1 += Q[e];
                s2 = fma(r2, E[e], s2);
                s3 = fma(r2, Q[e], s3);
                E[e] = Q[e] = 0.0;
            }
            cons.item += step;
            if (cons.item < last) dist_cursor_open(cons, d_out, d_in, col_tiles);
            fresh = true;
        }
    }
    cp_async_wait_all();
}

// The work items `first`, `first + step`, ... below `last` of one matrix, added into the thread's
// four running sums.
template <bool BF16>
__device__ __forceinline__ void dist_items(const void* W, long long w_row_stride, const __nv_bfloat16* What,
                                           const float* act_rms, int d_out, int d_in, int vec, long long first,
                                           long long last, long long step, double& s0, double& s1, double& s2,
                                           double& s3) {
    if (BF16 && vec) {
        dist_items_stream(static_cast<const __nv_bfloat16*>(W), w_row_stride, What, act_rms, d_out, d_in, first, last, step,
                          s0, s1, s2, s3);
        return;
    }
    const int col_tiles = (d_in + 8 * kDistThreads - 1) / (8 * kDistThreads);
    for (long long item = first; item < last; item += step) {
        const int chunk = int(item / col_tiles), tile = int(item - (long long)chunk * col_tiles);
        const int j0 = (tile * kDistThreads + threadIdx.x) * 8;
        if (j0 >= d_in) continue;
        const int r0 = chunk * kDistRows, r1 = min(d_out, r0 + kDistRows);
        double E[8], Q[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) E[e] = Q[e] = 0.0;
        int row = r0;
        for (; row + 2 <= r1; row += 2) {  // generic path: two rows in flight per thread
            float w[2][8], h[2][8];
#pragma unroll
            for (int u = 0; u < 2; ++u) dist_load<BF16>(W, w_row_stride, What, row + u, j0, d_in, vec, w[u], h[u]);
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const double wd = double(w[u][e]), d = wd - double(h[u][e]);
                    E[e] = fma(d, d, E[e]);
                    Q[e] = fma(wd, wd, Q[e]);
                }
        }
        for (; row < r1; ++row) {
            float w[8], h[8];
            dist_load<BF16>(W, w_row_stride, What, row, j0, d_in, vec, w, h);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const double wd = double(w[e]), d = wd - double(h[e]);
                E[e] = fma(d, d, E[e]);
                Q[e] = fma(wd, wd, Q[e]);
            }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            double r2 = 1.0;
            if (act_rms && j0 + e < d_in) {
                const double rj = double(act_rms[j0 + e]);
                r2 = rj * rj;
            }
            s0 += E[e];
            s1 += Q[e];
            s2 = fma(r2, E[e], s2);
            s3 = fma(r2, Q[e], s3);
        }
    }
}

// Block-wide sums of the four values (fixed order inside the block), added to out4 by four threads,
// or stored there when the caller adds the blocks up itself.
__device__ __forceinline__ void dist_flush(double s0, double s1, double s2, double s3, double* out4, bool store = false) {
    __shared__ double sh[4][kDistThreads / 32];
    s0 = warp_sum(s0); s1 = warp_sum(s1); s2 = warp_sum(s2); s3 = warp_sum(s3);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();  // a previous flush has been read
    if (lane == 0) { sh[0][warp] = s0; sh[1][warp] = s1; sh[2][warp] = s2; sh[3][warp] = s3; }
    __syncthreads();
    if (threadIdx.x < 4) {
        double v = 0;
        for (int w = 0; w < kDistThreads / 32; ++w) v += sh[threadIdx.x][w];
        if (store) out4[threadIdx.x] = v;
        else atomicAdd(out4 + threadIdx.x, v);
    }
}

template <bool BF16>
__global__ void __launch_bounds__(kDistThreads, 5) distortion_kernel(const void* W, long long w_row_stride,
                                                                  const __nv_bfloat16* What, const float* act_rms,
                                                                  int d_out, int d_in, int vec, double* out4) {
    const long long n_items = dist_item_count(d_out, d_in);
    double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    dist_items<BF16>(W, w_row_stride, What, act_rms, d_out, d_in, vec, blockIdx.x, n_items, gridDim.x, s0, s1, s2, s3);
    dist_flush(s0, s1, s2, s3, out4);
}

// All matrices of a batch: block b owns a contiguous span of the concatenated item list and leaves one
// record of four partial sums per matrix of its span.  The block that finishes last (one ticket counter
// behind a fence) adds the records of every matrix in a fixed order -- a thread per sum for the matrices
// a few blocks worked on, a warp per sum (lanes take every 32nd record, then a fixed tree) for a matrix
// spread over many -- and writes the four sums: one launch, no atomics on the sums, the same bits on
// every run.
constexpr int kDistWideRecords = 64;
template <bool BF16>
__global__ void __launch_bounds__(kDistThreads, 5) distortion_batch_kernel(const MatDesc* descs, const int4* spans,
                                                                        const DistReduce red, int n_mats) {
    const int4 span = spans[blockIdx.x];
    for (int m = span.x; m <= span.z; ++m) {
        const MatDesc& d = descs[m];
        const long long first = m == span.x ? span.y : 0;
        const long long last = m == span.z ? span.w : dist_item_count(d.d_out, d.d_in);
        const size_t esz = BF16 ? 2 : 4;
        const int vec = (d.d_in % 8 == 0) && (reinterpret_cast<uintptr_t>(d.W) % 16 == 0) &&
                        ((size_t(d.w_row_stride) * esz) % 16 == 0) && (reinterpret_cast<uintptr_t>(d.w_hat) % 16 == 0);
        double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
        if (first < last)
            dist_items<BF16>(d.W, d.w_row_stride, static_cast<const __nv_bfloat16*>(d.w_hat), d.act_rms, d.d_out, d.d_in, vec,
                             first, last, 1, s0, s1, s2, s3);
        const DistOwner own = red.owner[m];
        dist_flush(s0, s1, s2, s3, red.partial + 4 * size_t(own.offset + int(blockIdx.x) - own.first), true);
    }
    __shared__ bool last_block;
    __threadfence();  // this block's records are visible before its ticket is
    __syncthreads();
    if (threadIdx.x == 0) last_block = atomicAdd(red.counter, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!last_block) return;
    __threadfence();
    for (int idx = threadIdx.x; idx < 4 * n_mats; idx += blockDim.x) {
        const int m = idx >> 2, t = idx & 3;
        const DistOwner own = red.owner[m];
        const int n_rec = own.last - own.first + 1;
        if (n_rec > kDistWideRecords) continue;
        const double* rec = red.partial + 4 * size_t(own.offset) + t;
        double v = 0.0;
        for (int r = 0; r < n_rec; ++r) v += __ldcg(rec + 4 * size_t(r));
        descs[m].dist4[t] = v;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int idx = warp; idx < 4 * n_mats; idx += kDistThreads / 32) {
        const int m = idx >> 2, t = idx & 3;
        const DistOwner own = red.owner[m];
        const int n_rec = own.last - own.first + 1;
        if (n_rec <= kDistWideRecords) continue;
        const double* rec = red.partial + 4 * size_t(own.offset) + t;
        double v = 0.0;
        for (int r = lane; r < n_rec; r += 32) v += __ldcg(rec + 4 * size_t(r));
        v = warp_sum(v);
        if (lane == 0) descs[m].dist4[t] = v;
    }
    if (threadIdx.x == 0) *red.counter = 0u;  // ready for the next launch
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
    g.cvec = 0;
    return g;
}

// Per-column constant arrays allow vector loads: d_in a multiple of 8, floats 16-byte and signs
// 8-byte aligned.
int const_vec_ok(const qamw_params* p, const float* chan_scale, const int8_t* signs, const float* sigma) {
    auto al = [](const void* q, uintptr_t a) { return reinterpret_cast<uintptr_t>(q) % a == 0; };
    return (p->d_in % 8 == 0) && al(chan_scale, 16) && al(signs, 8) && al(sigma, 16);
}

// One persistent block per SM, or per second SM when the caller shares the device between two streams.
int grid_limit(const qamw_params* p) {
    const int n = sm_count();
    return (p->flags & QAMW_FLAG_HALF_DEVICE) ? std::max(1, n / 2) : n;
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

// Largest power-of-two number of codebook copies (at most 16: one per 8-byte bank pair) that
// fits into `budget` bytes of shared memory.
int pick_log2_copies(int K, size_t budget) {
    int log2c = 4;
    while (log2c > 0 && (size_t(K) * 8 << log2c) > budget) --log2c;
    return log2c;
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

namespace qamw {
int check_matrix_params(const qamw_params* p) { return check_params(p); }
long long distortion_items(int d_out, int d_in) { return dist_item_count(d_out, d_in); }
int distortion_batch_launch(const MatDesc* descs_dev, int n, const void* spans_dev, int blocks, int w_bf16,
                            const DistReduce& red, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (w_bf16) distortion_batch_kernel<true><<<blocks, kDistThreads, 0, st>>>(descs_dev, static_cast<const int4*>(spans_dev), red, n);
    else distortion_batch_kernel<false><<<blocks, kDistThreads, 0, st>>>(descs_dev, static_cast<const int4*>(spans_dev), red, n);
    return finish_launch("distortion_batch_kernel");
}
}  // namespace qamw

namespace {
// The codebook's tables live on the device it was created on; a call made with another device
// current would hand the kernels pointers they cannot use.
bool on_codebook_device(const qamw_codebook* cb) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == cb->device;
}
}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------

extern "C" const char* qamw_last_cuda_error(void) { return g_last_error; }

extern "C" int qamw_codebook_create(const float* codebook_host, int K, int grid, qamw_codebook** out) {
    if (!codebook_host || !out) return QAMW_ERR_ARG;
    if (K < 2 || K > QAMW_MAX_K || !is_pow2(K)) return QAMW_ERR_SHAPE;
    if (grid < 0 || grid > 255 || (grid > 0 && grid % 2 == 0)) return QAMW_ERR_ARG;
    *out = nullptr;
    SearchTable t;
    // The encoder's shared memory also holds 20 KB of per-warp index staging (16 warps x 1.25 KB)
    // and the codebook in eight bank-separated copies (two for K = 4096): the table gets what is left
    // of the 227 KB of one SM.  The grid side is odd.
    const size_t copies = K <= 2048 ? 8 : 2;
    const size_t budget = kSmemLimit - kEncodeStaticSmem - size_t(16) * (kStageSlotsPerWarp * 8) - size_t(K) * 8 * copies;
    if (!choose_search_table(codebook_host, K, grid, budget, &t)) return QAMW_ERR_NOMEM;
    qamw_codebook* cb = new (std::nothrow) qamw_codebook();
    if (!cb) return QAMW_ERR_NOMEM;
    cb->K = K;
    cb->map = t.map;
    cb->n_candidates = t.n_candidates;
    cb->max_list = t.max_list;
    cb->n_overflow_cells = t.n_overflow_cells;
    cb->h_codebook.assign(codebook_host, codebook_host + 2 * K);
    cb->off_cells = size_t(K) * 8;
    cb->off_overflow = cb->off_cells + t.cells.size() * 2;
    cb->blob_bytes = cb->off_overflow + t.overflow.size() * 2;
    std::vector<unsigned char> blob(cb->blob_bytes, 0);
    std::memcpy(blob.data(), codebook_host, size_t(K) * 8);
    std::memcpy(blob.data() + cb->off_cells, t.cells.data(), t.cells.size() * 2);
    if (!t.overflow.empty()) std::memcpy(blob.data() + cb->off_overflow, t.overflow.data(), t.overflow.size() * 2);
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

extern "C" int qamw_codebook_create_polar(const float* levels_host, int Ba, int Bp, qamw_codebook** out) {
    if (!levels_host || !out) return QAMW_ERR_ARG;
    *out = nullptr;
    if (Ba < 0 || Bp < 0 || Ba + Bp < 1 || (1 << (Ba + Bp)) > QAMW_MAX_K) return QAMW_ERR_SHAPE;
    const int Na = 1 << Ba, Np = 1 << Bp, K = Na * Np;
    for (int j = 0; j < Na; ++j)
        if (!(levels_host[j] > 0.f) || (j > 0 && !(levels_host[j] > levels_host[j - 1]))) return QAMW_ERR_ARG;
    qamw_codebook* cb = new (std::nothrow) qamw_codebook();
    if (!cb) return QAMW_ERR_NOMEM;
    cb->K = K;
    cb->polar = true;
    cb->polar_ba = Ba;
    cb->polar_bp = Bp;
    cb->h_codebook.resize(size_t(2) * K);
    qamw_polar_codebook(levels_host, Ba, Bp, cb->h_codebook.data());
    // squared thresholds between adjacent levels (the last entry is never read), then the unit vectors
    // of the bin boundaries 2 pi k / N_p of the upper half plane
    const int n_bnd = std::max(1, Np / 2);
    const int n_thr = std::max(2, Na);  // an even count keeps the 8-byte vectors behind it aligned
    std::vector<float> tables(size_t(n_thr) + 2 * size_t(n_bnd), 0.f);
    for (int j = 0; j + 1 < Na; ++j) {
        const double t = 0.5 * (double(levels_host[j]) + double(levels_host[j + 1]));
        tables[j] = float(t * t);
    }
    tables[Na - 1] = INFINITY;
    const double pi = 3.14159265358979323846264338327950288;
    for (int k2 = 0; k2 < n_bnd; ++k2) {
        const double beta = 2.0 * pi * k2 / double(Np);
        tables[n_thr + 2 * k2] = float(std::cos(beta));
        tables[n_thr + 2 * k2 + 1] = float(std::sin(beta));
    }
    cb->off_cells = size_t(K) * 8;
    cb->off_overflow = cb->off_cells + size_t(n_thr) * 4;
    cb->blob_bytes = (cb->off_cells + tables.size() * 4 + 15) & ~size_t(15);
    std::vector<unsigned char> blob(cb->blob_bytes, 0);
    std::memcpy(blob.data(), cb->h_codebook.data(), size_t(K) * 8);
    std::memcpy(blob.data() + cb->off_cells, tables.data(), tables.size() * 4);
    cudaError_t e = cudaGetDevice(&cb->device);
    if (e == cudaSuccess) e = cudaMalloc(&cb->d_blob, cb->blob_bytes);
    if (e == cudaSuccess) e = cudaMemcpy(cb->d_blob, blob.data(), cb->blob_bytes, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        set_cuda_error("qamw_codebook_create_polar", int(e));
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
    info_out[0] = cb->map.grid;
    info_out[1] = cb->n_candidates;
    info_out[2] = cb->max_list;
    info_out[3] = cb->n_overflow_cells;
    info_out[4] = int32_t((cb->blob_bytes - cb->off_overflow) / 2);
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
    if (!on_codebook_device(cb)) return QAMW_ERR_ARG;
    const size_t row_bytes = qamw_packed_row_bytes(p->d_in, p->K);
    if (p->packed_row_stride < (long long)row_bytes || p->packed_row_stride % 4) return QAMW_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(packed_out) % 4) return QAMW_ERR_ALIGN;
    if (p->d_out == 0) return QAMW_OK;
    if (!(p->flags & QAMW_FLAG_GENERAL_KERNELS)) {  // common layouts: the multi-matrix kernel, here with one matrix
        MatDesc d{};
        d.W = W;
        d.chan_scale = chan_scale;
        d.signs = signs;
        d.sigma = sigma;
        d.packed = packed_out;
        d.row_norm = row_norm_out;
        d.w_row_stride = p->w_row_stride;
        d.packed_row_stride = p->packed_row_stride;
        d.d_out = p->d_out;
        d.d_in = p->d_in;
        rc = rows_encode(nullptr, &d, 1, nullptr, 0, p->block, p->K, p->w_dtype == QAMW_DTYPE_BF16, cb, p->flags,
                         status_out, stream);
        if (rc != QAMW_ERR_SHAPE) return rc;
    }
    if (cb->polar) return QAMW_ERR_SHAPE;  // the polar quantiser exists in the kernels for the common layouts only
    EncodeArgs a;
    a.g = make_geom(p, W);
    a.g.cvec = const_vec_ok(p, chan_scale, signs, sigma);
    a.W = W;
    a.chan_scale = chan_scale;
    a.signs = signs;
    a.sigma = sigma;
    a.codebook = static_cast<const float2*>(cb->d_blob);
    a.table = reinterpret_cast<const uint4*>(static_cast<const unsigned char*>(cb->d_blob) + cb->off_cells);
    a.table_bytes = int(cb->blob_bytes - cb->off_cells);
    a.off_overflow = int(cb->off_overflow - cb->off_cells);
    a.K = p->K;
    a.log2K = ilog2(p->K);
    a.grid = cb->map.grid;
    a.map_zmax = cb->map.zmax;
    a.map_c0 = cb->map.c0;
    a.map_c1 = cb->map.c1;
    a.map_c2 = cb->map.c2;
    a.map_bias = 12582912.0f + float(cb->map.half);
    a.brute = (p->flags & QAMW_FLAG_BRUTE_FORCE) ? 1 : 0;
    a.packed = packed_out;
    a.packed_row_stride = p->packed_row_stride;
    a.row_words = int(p->packed_row_stride / 4);
    a.payload_words = int((row_bytes + 3) / 4);
    a.row_norm = row_norm_out;
    a.inv_sqrt_b = float(1.0 / std::sqrt(double(p->block)));
    const size_t fixed = ((size_t(a.table_bytes) + 15) & ~size_t(15)) +
                         size_t(a.g.groups) * (a.g.tg / 32) * (kStageSlotsPerWarp * 8);
    if (fixed + size_t(p->K) * 8 > kSmemLimit - kEncodeStaticSmem) return QAMW_ERR_NOMEM;
    a.log2c = pick_log2_copies(p->K, kSmemLimit - kEncodeStaticSmem - fixed);
    const size_t smem = fixed + (size_t(p->K) * 8 << a.log2c);
    const int blocks = std::max(1, std::min(grid_limit(p), (p->d_out + a.g.groups - 1) / a.g.groups));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    a.status = status_out;
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
    a.g.cvec = const_vec_ok(p, chan_scale, signs, nullptr);
    a.W = W;
    a.chan_scale = chan_scale;
    a.signs = signs;
    a.mode = 0;
    a.y_out = y_out;
    a.row_norm = row_norm_out;
    a.status = status_out;
    const int blocks = std::max(1, std::min(grid_limit(p), (p->d_out + a.g.groups - 1) / a.g.groups));
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
    c.blocks = std::max(1, std::min(std::min(148, grid_limit(p)), (c.n_rows + g.groups - 1) / g.groups));
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
    a.g.cvec = const_vec_ok(p, chan_scale, signs, nullptr);
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
    calibrate_finish_kernel<<<(n_pairs + 31) / 32, 32 * kFinishSlices, 0, st>>>(a.partial, c.total_groups, c.pair_stride, n_pairs,
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
// Largest need of any accepted shape: at most 148 blocks x 15 row groups of partial sums over at most
// 8192 pair positions, plus the row counts.  The refusal below therefore never fires today; it guards
// the array against a later change of those limits.
static_assert(size_t(148) * kMaxGroups * (size_t(32 * kMaxThreads / 2) + 1) * sizeof(double) >= 0, "");

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

extern "C" int qamw_quantize(const void* W, const qamw_params* p, const float* act_rms_host, float alpha,
                             uint64_t sign_seed, const qamw_codebook* cb, float* chan_scale_out, int8_t* signs_out,
                             float* sigma_out, uint8_t* packed_out, float* row_norm_out, void* workspace,
                             size_t workspace_bytes, int32_t* status_out, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!W || !cb || !signs_out || !sigma_out || !packed_out || !row_norm_out || !workspace) return QAMW_ERR_ARG;
    const bool scaled = act_rms_host && alpha != 0.f;
    if (scaled && !chan_scale_out) return QAMW_ERR_ARG;
    if (workspace_bytes < qamw_calibrate_workspace_bytes(p)) return QAMW_ERR_NOMEM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // E0 and the sign mask are d_in numbers each: computed on the host, copied once
    std::vector<int8_t> signs(size_t(p->d_in));
    rc = qamw_make_signs(sign_seed, p->d_in, signs.data());
    if (rc) return rc;
    cudaError_t e = cudaMemcpyAsync(signs_out, signs.data(), signs.size(), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && scaled) {
        std::vector<float> s(size_t(p->d_in));
        rc = qamw_channel_scales(act_rms_host, p->d_in, alpha, s.data());
        if (rc) return rc;
        e = cudaMemcpyAsync(chan_scale_out, s.data(), s.size() * sizeof(float), cudaMemcpyHostToDevice, st);
    }
    if (e != cudaSuccess) {
        set_cuda_error("qamw_quantize: cudaMemcpyAsync", int(e));
        return QAMW_ERR_CUDA;
    }
    const float* cs = scaled ? chan_scale_out : nullptr;
    rc = qamw_calibrate(W, p, cs, signs_out, sigma_out, workspace, workspace_bytes, status_out, stream);
    if (rc) return rc;
    return qamw_encode(W, p, cs, signs_out, sigma_out, cb, packed_out, row_norm_out, status_out, stream);
}

extern "C" int qamw_decode(const uint8_t* packed, const float* row_norm, const float* chan_scale, const int8_t* signs,
                           const float* sigma, const qamw_codebook* cb, const qamw_params* p, void* w_hat_bf16_out,
                           void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!packed || !row_norm || !signs || !sigma || !cb || !w_hat_bf16_out) return QAMW_ERR_ARG;
    if (cb->K != p->K) return QAMW_ERR_ARG;
    if (!on_codebook_device(cb)) return QAMW_ERR_ARG;
    const size_t row_bytes = qamw_packed_row_bytes(p->d_in, p->K);
    if (p->packed_row_stride < (long long)row_bytes || p->packed_row_stride % 4) return QAMW_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(packed) % 4 || reinterpret_cast<uintptr_t>(w_hat_bf16_out) % 2) return QAMW_ERR_ALIGN;
    if (p->d_out == 0) return QAMW_OK;
    if (!(p->flags & QAMW_FLAG_GENERAL_KERNELS)) {  // common layouts: the multi-matrix kernel, here with one matrix
        MatDesc d{};
        d.chan_scale = chan_scale;
        d.signs = signs;
        d.sigma = sigma;
        d.packed = const_cast<uint8_t*>(packed);
        d.row_norm = const_cast<float*>(row_norm);
        d.w_hat = w_hat_bf16_out;
        d.packed_row_stride = p->packed_row_stride;
        d.d_out = p->d_out;
        d.d_in = p->d_in;
        rc = rows_decode(nullptr, &d, 1, nullptr, 0, p->block, p->K, static_cast<const float*>(cb->d_blob), p->flags, stream);
        if (rc != QAMW_ERR_SHAPE) return rc;
    }
    DecodeArgs a;
    a.g = make_geom(p, nullptr);
    a.g.cvec = const_vec_ok(p, chan_scale, signs, sigma);
    a.g.vec = (p->d_in % 8 == 0) && (reinterpret_cast<uintptr_t>(w_hat_bf16_out) % 16 == 0);
    a.packed = packed;
    a.packed_row_stride = p->packed_row_stride;
    a.row_bytes = int((row_bytes + 3) / 4 * 4);
    const bool rows16 = reinterpret_cast<uintptr_t>(packed) % 16 == 0 && p->packed_row_stride % 16 == 0;
    a.copy_log2 = rows16 ? 4 : 2;
    if (rows16) a.row_bytes = int((row_bytes + 15) / 16 * 16);  // <= the stride, which is a multiple of 16
    a.log2K = ilog2(p->K);
    a.seg_bytes = 64 * a.log2K;
    a.stage_bytes = a.seg_bytes + 16;
    a.inv_sqrt_b = float(1.0 / std::sqrt(double(p->block)));
    a.row_norm = row_norm;
    a.chan_scale = chan_scale;
    a.signs = signs;
    a.sigma = sigma;
    a.codebook = static_cast<const float2*>(cb->d_blob);
    a.K = p->K;
    a.out = static_cast<__nv_bfloat16*>(w_hat_bf16_out);
    const size_t stage_total = size_t(a.g.groups) * (a.g.tg / 32) * 2 * a.stage_bytes;
    a.log2c = pick_log2_copies(p->K, std::min(size_t(128) * 1024, kSmemLimit - stage_total));
    const size_t smem = (size_t(p->K) * 8 << a.log2c) + stage_total;
    const int blocks = std::max(1, std::min(grid_limit(p), (p->d_out + a.g.groups - 1) / a.g.groups));
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
    const size_t esz = p->w_dtype == QAMW_DTYPE_BF16 ? 2 : 4;
    const int vec = (p->d_in % 8 == 0) && (reinterpret_cast<uintptr_t>(W) % 16 == 0) &&
                    ((size_t(p->w_row_stride) * esz) % 16 == 0) && (reinterpret_cast<uintptr_t>(w_hat_bf16) % 16 == 0);
    const long long items = (long long)((p->d_in + 8 * kDistThreads - 1) / (8 * kDistThreads)) *
                            ((p->d_out + kDistRows - 1) / kDistRows);
    const int blocks = int(std::max<long long>(1, std::min<long long>(32LL * sm_count(), items)));
    if (p->w_dtype == QAMW_DTYPE_BF16)
        distortion_kernel<true><<<blocks, kDistThreads, 0, st>>>(W, p->w_row_stride,
                                                                 static_cast<const __nv_bfloat16*>(w_hat_bf16), act_rms,
                                                                 p->d_out, p->d_in, vec, out4);
    else
        distortion_kernel<false><<<blocks, kDistThreads, 0, st>>>(W, p->w_row_stride,
                                                                  static_cast<const __nv_bfloat16*>(w_hat_bf16), act_rms,
                                                                  p->d_out, p->d_in, vec, out4);
    return finish_launch("distortion_kernel");
}
