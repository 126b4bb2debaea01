// Row kernels of libqamw for the common layouts (32-byte aligned rows, d_in a multiple of 16,
// Hadamard blocks of 32 elements or more): one persistent launch walks any number of matrices.
//
// Geometry.
//   * A warp owns a "segment" of 256 * NS consecutive elements of a row: NS = 4 octets (32 elements)
//     per thread in the decoder, NS = 2 (16 elements) in the encoder, whose register budget then
//     allows 20 to 28 resident warps per SM instead of 15.  A row is owned by a group of
//     ceil(d_in / (256 NS)) warps; a block holds as many groups as fit and the grid is persistent.
//   * A launch takes an array of matrix descriptors.  The rows of all matrices form one list, cut
//     into one contiguous span per block with (nearly) equal numbers of weights, so a block meets one
//     or two matrices; the tables in shared memory (codebook copies, cell records) are filled once
//     per launch and only the per-column constants of a warp's segment are reloaded when the matrix
//     changes.
//   * Walsh-Hadamard butterflies of a block of b elements: stages h = 1, 2, 4 inside an octet, then
//     one stage per octet slot bit inside the thread, then one "half exchange" per lane bit: a thread
//     keeps the slots whose top slot bit is 0, sends the others to its partner (lane ^ 2^j), and
//     computes both outputs (K + R, K - R) of the butterflies whose inputs it then holds.  Every
//     exchange uses the top slot bit, so after the last stage a thread holds runs of NS/2 adjacent
//     octets and the threads of a block cover consecutive runs: 32-byte stores that tile full
//     128-byte lines (decoder).  A thread starts with NS consecutive octets.  Which physical slot
//     receives the sum and which the difference of a stage is chosen so that the next stage can again
//     keep the lower slots and send the upper ones without moving registers: a thread whose next lane
//     bit is set multiplies the received value by -1 first (K - R, K + R), and the last in-thread
//     stage does the same for odd lanes.  An upper partner then holds R - K as K - R: some slots end
//     up negated, by a pattern that depends on the lane only and is folded into the per-column
//     constants.  Stages run in ascending order of h with one f32 rounding per output, and a
//     multiplication by +-1 is exact, so the result is bit-identical to the plain butterfly.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <new>
#include <type_traits>
#include <unordered_map>
#include <vector>

#include "qamw_device.cuh"
#include "qamw_internal.h"

using namespace qamw;

namespace {

// ---------------------------------------------------------------------------------------------
// layout of a Hadamard block over NS slots and L = 2^S lanes
// ---------------------------------------------------------------------------------------------
template <int NS, int LOG2B>
struct Lay2 {
    static_assert(NS == 2 || NS == 4, "two or four octets per thread");
    static constexpr int LS = NS == 4 ? 2 : 1;          // slot bits
    static constexpr int TOP = NS / 2;                  // value of the top slot bit
    static constexpr int S = LOG2B - 3 - LS;            // cross-lane stages
    static_assert(S >= 0 && S <= 5, "block size out of range for this geometry");
    static constexpr int L = 1 << S;
    // octet (units of 8 elements, relative to the warp's segment) in physical slot p before the
    // butterflies: NS consecutive octets per lane
    __device__ static __forceinline__ int octet_before(int lane, int p) { return NS * lane + p; }
    // ... and after them
    __device__ static __forceinline__ int octet_after(int lane, int p) {
        if (S == 0) return NS * lane + p;
        const int q = lane & (L - 1), blk = lane >> S;
        const int o = (p & (TOP - 1)) | ((q & 1) << (LS - 1)) | ((q >> 1) << LS) | ((p >> (LS - 1)) << (LS + S - 1));
        return blk * (NS * L) + o;
    }
    // true if physical slot p of this lane holds minus the butterfly output
    __device__ static __forceinline__ bool negated(int lane, int p) {
        bool neg_k = false, neg_x = false;
#pragma unroll
        for (int j = 0; j < S; ++j) {
            const bool upper = (lane >> j) & 1;
            const bool normal = (j == S - 1) || !((lane >> (j + 1)) & 1);
            if (normal) {
                neg_x = neg_k ^ upper;
            } else {
                const bool old = neg_k;
                neg_k = old ^ upper;
                neg_x = old;
            }
        }
        return (p & TOP) ? neg_x : neg_k;
    }
};

// Unnormalised Walsh-Hadamard butterfly of the NS x 8 elements of a thread and, for wider blocks, of
// the L lanes of the block.  P[p][i] holds elements (2i, 2i+1) of the octet in physical slot p.
// FIRST_STAGE_DONE: the caller's inputs already went through stage h = 1.
template <int NS, int LOG2B, bool FIRST_STAGE_DONE>
__device__ __forceinline__ void fwht2(f32x2 (&P)[NS][4], int lane) {
    typedef Lay2<NS, LOG2B> Lay;
    constexpr int TOP = Lay::TOP;
    if (!FIRST_STAGE_DONE) {
#pragma unroll
        for (int p = 0; p < NS; ++p)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float a, c;
                unpack2(P[p][i], a, c);
                P[p][i] = pack2(__fadd_rn(a, c), __fsub_rn(a, c));
            }
    }
#pragma unroll
    for (int p = 0; p < NS; ++p) {  // h = 2, 4
        bfly2(P[p][0], P[p][1]);
        bfly2(P[p][2], P[p][3]);
        bfly2(P[p][0], P[p][2]);
        bfly2(P[p][1], P[p][3]);
    }
    if (NS == 4) {  // h = 8: slot bit 0
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            bfly2(P[0][i], P[1][i]);
            bfly2(P[2 % NS][i], P[3 % NS][i]);
        }
    }
    // top slot bit (h = 8 for NS = 2, h = 16 for NS = 4).  The first half exchange wants the two
    // halves of an odd lane in swapped places, so an odd lane writes its difference into the lower
    // slots and its sum into the upper ones: out_lo = a + s c, out_hi = a - s c with s = -1.
    if (Lay::S >= 1) {
        const float s0 = (lane & 1) ? -1.0f : 1.0f;
        const f32x2 sp = pack2(s0, s0), sn = pack2(-s0, -s0);
#pragma unroll
        for (int p = 0; p < TOP; ++p)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const f32x2 a = P[p][i], c = P[p + TOP][i];
                P[p][i] = fma2(c, sp, a);
                P[p + TOP][i] = fma2(c, sn, a);
            }
    } else {
#pragma unroll
        for (int p = 0; p < TOP; ++p)
#pragma unroll
            for (int i = 0; i < 4; ++i) bfly2(P[p][i], P[p + TOP][i]);
    }
    // cross-lane stages
#pragma unroll
    for (int j = 0; j < Lay::S; ++j) {
        if (j == Lay::S - 1) {
#pragma unroll
            for (int p = 0; p < TOP; ++p)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const f32x2 keep = P[p][i];
                    const f32x2 got = shfl_xor2(P[p + TOP][i], 1 << j);
                    P[p][i] = add2(keep, got);
                    P[p + TOP][i] = sub2(keep, got);
                }
        } else {
            const float al = ((lane >> (j + 1)) & 1) ? -1.0f : 1.0f;
            const f32x2 ap = pack2(al, al), an = pack2(-al, -al);
#pragma unroll
            for (int p = 0; p < TOP; ++p)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const f32x2 keep = P[p][i];
                    const f32x2 got = shfl_xor2(P[p + TOP][i], 1 << j);
                    P[p][i] = fma2(got, ap, keep);
                    P[p + TOP][i] = fma2(got, an, keep);
                }
        }
    }
}

__device__ __forceinline__ void st_global_256(void* p, const uint32_t (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]),
                 "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}
__device__ __forceinline__ void ld_global_256(const void* p, uint32_t (&w)[8]) {
    asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// The span of the concatenated row list that this block works on: first matrix, first row in it,
// last matrix, end row in it.  Without a span table there is one matrix, split evenly.
__device__ __forceinline__ int4 block_span(const int4* spans, int d_out_single) {
    if (spans) return spans[blockIdx.x];
    const long long n = d_out_single;
    return make_int4(0, int(n * blockIdx.x / gridDim.x), 0, int(n * (blockIdx.x + 1) / gridDim.x));
}

// ---------------------------------------------------------------------------------------------
// decoder
// ---------------------------------------------------------------------------------------------
constexpr int kDecodeDepth = 4;
template <int N>
__device__ __forceinline__ void cp_async_wait_pending() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

struct Decode2Args {
    const MatDesc* descs;    // device array, or NULL: `one` is the only matrix
    MatDesc one;
    const int4* spans;       // per block (see block_span), or NULL
    const float2* codebook;  // device, K entries
    int K, log2K, log2c;
    int seg_bytes;           // packed bytes of one warp segment: 16 * NS * B
    int stage_bytes;         // one staging buffer of a warp (128-byte aligned, at least seg_bytes + 16)
    float inv_sqrt_b;
};

// A warp streams its segment of the packed row through its own shared-memory ring of kDecodeDepth rows
// (16-byte asynchronous copies, kDecodeDepth - 1 rows ahead: with one row in flight per warp the reads
// are bound by memory latency); nothing is shared between warps after the prologue, so there is no
// barrier.
// Per row a thread reads its 4 NS B index bits as two runs of 32-bit words, gathers the codewords
// (stored as (x + y, x - y): butterfly stage h = 1) from its own bank-separated copy, scales them by
// the pair scales, runs the remaining butterflies and writes bf16.
template <int NS, int LOG2B>
__global__ void __launch_bounds__(NS == 4 ? 512 : 896, 1) decode2_kernel(const Decode2Args a) {
    typedef Lay2<NS, LOG2B> Lay;
    constexpr int TOP = Lay::TOP;
    constexpr int WE = 256 * NS;  // elements of a warp segment
    extern __shared__ __align__(16) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int B = a.log2K;
    const uint32_t mask = (1u << B) - 1u;
    const uint32_t cb_stride = 8u << a.log2c;
    const uint32_t cb = smem_addr(smem) + 8u * (threadIdx.x & ((1 << a.log2c) - 1));
    unsigned char* stage = smem + ((size_t(a.K) * 8) << a.log2c) + size_t(warp) * kDecodeDepth * a.stage_bytes;
    const uint32_t stage_addr = smem_addr(stage);

    fill_codebook_copies(reinterpret_cast<float2*>(smem), a.codebook, a.K, a.log2c, true);
    // the 16 bytes after a staged segment are read (and masked away) by the last threads: keep them defined
    if (lane < 4 * kDecodeDepth) reinterpret_cast<uint32_t*>(stage + (lane >> 2) * a.stage_bytes + a.seg_bytes)[lane & 3] = 0u;
    __syncthreads();

    // where this thread's index bits sit inside a staged segment: two runs (the lower and the upper
    // physical slots), each 4 B TOP bits long
    uint32_t run_word[2], run_shift[2];
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        const unsigned bit0 = unsigned(4 * Lay::octet_before(lane, x * TOP)) * unsigned(B);
        run_word[x] = 4u * (bit0 >> 5);
        run_shift[x] = bit0 & 31u;
    }

    const int4 span = block_span(a.spans, a.one.d_out);
    for (int m = span.x; m <= span.z; ++m) {
        const MatDesc& d = a.descs ? a.descs[m] : a.one;
        const int d_in = d.d_in, n_pairs = d_in >> 1;
        const int row_begin = m == span.x ? span.y : 0;
        const int row_end = m == span.z ? span.w : d.d_out;
        const int n_seg = (d_in + WE - 1) / WE;
        const int groups = n_warps / n_seg;  // >= 1 (checked on the host)
        const int group = warp / n_seg, seg = warp - group * n_seg;
        const int row0 = row_begin + group;
        if (group >= groups || row0 >= row_end) continue;  // this warp has no work in this matrix
        const int row_step = groups;
        const int n_rows = (row_end - row0 + row_step - 1) / row_step;
        const long long pstride = d.packed_row_stride;
        const int row_bytes = int((((long long)n_pairs * B + 7) / 8 + 15) & ~15LL);  // <= stride (a multiple of 16)
        const long long seg_off = (long long)seg * a.seg_bytes;
        const int n_chunks = max(0, min(a.seg_bytes, row_bytes - int(seg_off))) >> 4;
        // at most 48 chunks of 16 bytes per segment: two predicated copies per lane, no loop
        const bool copy0 = lane < n_chunks, copy1 = lane + 32 < n_chunks;
        const unsigned char* src = d.packed + (long long)row0 * pstride + seg_off;  // next row to fetch
        const long long src_step = (long long)row_step * pstride;
        int issued = 0;
        auto issue_row = [&]() {  // one commit group per row, empty past the end
            if (issued < n_rows) {
                unsigned char* dst = stage + (issued % kDecodeDepth) * a.stage_bytes;
                if (copy0) cp_async(dst + (lane << 4), src + (lane << 4), 4);
                if (copy1) cp_async(dst + ((lane + 32) << 4), src + ((lane + 32) << 4), 4);
                src += src_step;
            }
            ++issued;
            cp_async_commit();
        };
        __syncwarp();  // the previous matrix's last row has been read by every lane
        for (int i = 0; i < kDecodeDepth - 1; ++i) issue_row();

        // per-column constants of this warp's segment
        const int oct0 = seg * (WE / 8);  // first octet of the segment
        float sg[NS][4];
        f32x2 mcol[NS][4];
        bool store_ok[NS];
        int e_out[NS];
#pragma unroll
        for (int p = 0; p < NS; ++p) {
            const int k0 = 4 * (oct0 + Lay::octet_before(lane, p));
            load4f(d.sigma, k0, n_pairs, 1, 0.f, sg[p]);
            const int e0 = 8 * (oct0 + Lay::octet_after(lane, p));
            e_out[p] = e0;
            store_ok[p] = e0 < d_in;
            float cs[8], sgn[8];
            if (d.chan_scale) {
                load8f(d.chan_scale, e0, d_in, 1, 1.0f, cs);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) cs[e] = 1.0f;
            }
            load8s(d.signs, e0, d_in, 1, sgn);
            const float fl = Lay::negated(lane, p) ? -1.0f : 1.0f;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                mcol[p][i] = pack2(fl * __fdiv_rn(sgn[2 * i] * a.inv_sqrt_b, cs[2 * i]),
                                   fl * __fdiv_rn(sgn[2 * i + 1] * a.inv_sqrt_b, cs[2 * i + 1]));
        }
        __nv_bfloat16* orow = static_cast<__nv_bfloat16*>(d.w_hat) + (long long)row0 * d_in;
        const long long out_step = (long long)row_step * d_in;
        const float* rnp = d.row_norm + row0;

        for (int it = 0; it < n_rows; ++it, orow += out_step, rnp += row_step) {
            const float rn = __ldg(rnp);
            cp_async_wait_pending<kDecodeDepth - 2>();
            __syncwarp();  // every lane's part of this row has landed; the buffer refilled next is no longer read
            issue_row();
            const uint32_t in = stage_addr + uint32_t((it % kDecodeDepth) * a.stage_bytes);
            f32x2 P[NS][4];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const uint32_t w = in + run_word[x];
                const uint32_t sh = run_shift[x];
                uint32_t id[4 * TOP];
                if (NS == 4) {
                    // 8 indices = 8 B bits <= 96: four words, shifted down to three, then cut in steps of 2 B bits
                    const uint32_t w0 = lds_u32(w), w1 = lds_u32(w + 4), w2 = lds_u32(w + 8), w3 = lds_u32(w + 12);
                    uint32_t v0 = __funnelshift_r(w0, w1, sh), v1 = __funnelshift_r(w1, w2, sh), v2 = __funnelshift_r(w2, w3, sh);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        id[2 * t] = v0 & mask;
                        id[2 * t + 1] = (v0 >> B) & mask;
                        if (t < 3) {
                            v0 = __funnelshift_r(v0, v1, 2 * B);
                            v1 = __funnelshift_r(v1, v2, 2 * B);
                            v2 >>= 2 * B;
                        }
                    }
                } else {
                    const uint32_t w0 = lds_u32(w), w1 = lds_u32(w + 4), w2 = lds_u32(w + 8);
                    const uint32_t a0 = __funnelshift_r(w0, w1, sh), a1 = __funnelshift_r(w1, w2, sh);
                    const uint32_t b0 = __funnelshift_r(a0, a1, 2 * B);
                    id[0] = a0 & mask;
                    id[1] = (a0 >> B) & mask;
                    id[2] = b0 & mask;
                    id[3] = (b0 >> B) & mask;
                }
#pragma unroll
                for (int t = 0; t < TOP; ++t) {
                    const int p = x * TOP + t;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        // pairs beyond the end of the row have scale 0 and decode to 0 whatever their bits are
                        const float2 c = lds_f32x2(cb + id[4 * t + i] * cb_stride);
                        P[p][i] = pack2(c.x * sg[p][i], c.y * sg[p][i]);
                    }
                }
            }
            fwht2<NS, LOG2B, true>(P, lane);
            const f32x2 rn2 = pack2(rn, rn);
#pragma unroll
            for (int p = 0; p < NS; p += (NS == 4 ? 2 : 1)) {
                constexpr int NP = NS == 4 ? 2 : 1;  // adjacent octets written by one store
                uint32_t w[4 * NP];
#pragma unroll
                for (int t = 0; t < NP; ++t)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float y0, y1;
                        unpack2(mul2(P[p + t][i], mul2(mcol[p + t][i], rn2)), y0, y1);
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(y0, y1);
                        w[4 * t + i] = *reinterpret_cast<uint32_t*>(&h2);
                    }
                if (store_ok[p]) {
                    if constexpr (NS == 4) {
                        st_global_256(orow + e_out[p], w);
                    } else {
                        *reinterpret_cast<uint4*>(orow + e_out[p]) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
        cp_async_wait_all();
    }
}

// ---------------------------------------------------------------------------------------------
// encoder
// ---------------------------------------------------------------------------------------------
struct Encode2Args {
    const MatDesc* descs;
    MatDesc one;
    const int4* spans;
    const float2* codebook;  // device, K entries
    const uint4* table;      // cells | overflow, as laid out by qamw_codebook_create
    int table_bytes;         // a multiple of 16
    int off_overflow;        // byte offset inside the table
    int K, log2K, grid;
    float map_zmax, map_c0, map_c1, map_c2, map_bias;  // the cell map of the table
    int log2c;               // log2 of the number of codebook copies in shared memory
    int brute;
    float inv_sqrt_b;        // c_b = f32(1 / sqrt(b))
    int32_t* status;         // out (optional): bit 0 set when a row norm is not finite
    unsigned char* calib_base;  // calibration mode: base of the partial-sum workspace (MatDesc::calib_offset)
    int polar_ba, polar_bp;  // polar quantiser: amplitude and phase bits; `table` then holds the squared
                             // amplitude thresholds (2^Ba floats) and, from off_overflow on, the unit vectors
                             // of the phase bin boundaries of the upper half plane (2^Bp / 2 float2)
};

// Polar quantiser (Section 3.5): amplitude |z| to the nearest of 2^Ba levels, phase to one of 2^Bp
// uniform bins, index = (phase << Ba) | amplitude.  Both are binary searches over small tables in
// shared memory: squared thresholds (midpoints of adjacent levels) for the amplitude, and for the
// phase the sign of the cross product with the boundary directions after folding the lower half plane
// onto the upper one.  A point on a threshold takes the lower level, a point on a boundary the bin
// that starts there, the origin bin 0 -- the oracle's rules; within f32 rounding of a threshold or a
// boundary either neighbour may come out.
struct PolarSmem {
    uint32_t thr2;  // shared-memory address of the squared thresholds
    uint32_t bnd;   // ... of the boundary unit vectors
    int Ba, Bp;
};
__device__ __forceinline__ int search_polar(const PolarSmem& s, float zx, float zy) {
    const float r2 = __fmaf_rn(zy, zy, __fmul_rn(zx, zx));
    int a = 0;
    for (int step = (1 << s.Ba) >> 1; step > 0; step >>= 1) {
        float t;
        asm("ld.shared.f32 %0, [%1];" : "=f"(t) : "r"(s.thr2 + 4u * uint32_t(a + step - 1)));
        if (r2 > t) a += step;
    }
    int p = 0;
    if (s.Bp > 0) {
        const bool lower = zy < 0.f || (zy == 0.f && zx < 0.f);
        const float x = lower ? -zx : zx, y = lower ? -zy : zy;
        for (int step = (1 << s.Bp) >> 2; step > 0; step >>= 1) {
            const float2 b = lds_f32x2(s.bnd + 8u * uint32_t(p + step));
            if (__fmaf_rn(b.x, y, -__fmul_rn(b.y, x)) >= 0.f) p += step;
        }
        if (lower) p += (1 << s.Bp) >> 1;
        if (r2 == 0.f) p = 0;
    }
    return (p << s.Ba) | a;
}

// Index staging of a warp: its 64 octets as one 64-bit value each (index p of the octet at bits
// [p B, (p+1) B)); 8 slots of padding after every 16 keep the two stores of a warp on distinct banks
// for the common block sizes.
template <int NS>
struct Stage2 {
    static constexpr int kSlots = NS == 2 ? 96 : 160;  // 32 NS octets plus their padding
    __device__ static __forceinline__ int slot(int o) { return NS == 2 ? o + ((o >> 4) << 3) : o + ((o >> 4) << 2); }
};

// Encoder, two octets per thread.  A warp owns 512 consecutive elements of a row: it scales them,
// adds up its part of the row norm, rotates (shuffles only), and after the one meeting point of the
// row's warps -- a named barrier for the norm -- searches its 256 pairs, stages the indices and
// writes its 32 B bytes of the packed row.  W is read once.
// QUANT: 0 = nearest codeword through the cell table, 1 = polar quantiser, 2 = no quantiser at all:
// the kernel then is the calibration pass of Section 3.4, which visits n = min(d_out, 1024) rows
// floor(t d_out / n) and adds up the pair moduli |(y_2k, y_2k+1)| per pair position.  Every row group
// of every block owns one slot of partial sums in the workspace; calibrate_finish2_kernel adds the
// slots in ascending order, so the result does not depend on timing.
template <bool BF16, int LOG2B, int NS, int MAXT, int QUANT>
__global__ void __launch_bounds__(MAXT, 1) encode2_kernel(const Encode2Args a) {
    constexpr bool POLAR = QUANT == 1, CALIB = QUANT == 2;
    constexpr int WE = 256 * NS;
    typedef Lay2<NS, LOG2B> Lay;
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ double ss_part[2][32];  // per-warp partial sums of squares, two rows in flight
    __shared__ MatDesc cur;            // the matrix the block is working on (re-read per row: saves registers)
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;

    const int cb_bytes = QUANT != 0 ? 0 : (a.K * 8) << a.log2c;  // only the table search reads codewords
    if (QUANT == 0) fill_codebook_copies(reinterpret_cast<float2*>(smem), a.codebook, a.K, a.log2c);
    unsigned char* table = smem + cb_bytes;
    if (!CALIB) {
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
    unsigned long long* oct_s = reinterpret_cast<unsigned long long*>(table + table_pad) + size_t(warp) * Stage2<NS>::kSlots;

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
    PolarSmem ps;
    ps.thr2 = smem_addr(table);
    ps.bnd = smem_addr(table + a.off_overflow);
    ps.Ba = a.polar_ba;
    ps.Bp = a.polar_bp;

    const int B = a.log2K, B4 = 4 * a.log2K;
    const unsigned div_magic = 0xffffffffu / unsigned(B4) + 1u;  // ceil(2^32 / (4B))
    constexpr int kEsz = BF16 ? 2 : 4;

    const int4 span = block_span(a.spans, a.one.d_out);
    for (int m = span.x; m <= span.z; ++m) {
        // The warps regroup when the row length changes: nobody may still be inside the previous
        // matrix (its named barriers and partial sums) when the first warp enters the next one.  The
        // first pass also waits for the tables.
        __syncthreads();
        if (threadIdx.x == 0) cur = a.descs ? a.descs[m] : a.one;
        __syncthreads();
        const MatDesc& d = cur;
        const int d_in = d.d_in, n_pairs = d_in >> 1;
        const int row_begin = m == span.x ? span.y : 0;
        const int n_cal = min(d.d_out, QAMW_CALIB_MAX_ROWS);  // calibration walks this many rows
        const int row_end = m == span.z ? span.w : (CALIB ? n_cal : d.d_out);
        const int n_seg = (d_in + WE - 1) / WE;
        const int groups = min(15, n_warps / n_seg);  // named barriers 1..15
        const int group = warp / n_seg, seg = warp - group * n_seg;
        const int row0 = row_begin + group;
        if (group >= groups || row0 >= row_end) continue;
        const int row_step = groups;
        const int tg = n_seg * 32;
        const int oct0 = seg * (WE / 8);

        // per-column constants: t_j = s_j sign_j of the columns the thread loads; reciprocal pair scales
        // (with the butterfly's sign pattern folded in) of the pairs it holds after the rotation
        f32x2 t[NS][4];
        float q[NS][4];
        bool live[NS];
        bool risky = false;
#pragma unroll
        for (int p = 0; p < NS; ++p) {
            const int e0 = 8 * (oct0 + Lay::octet_before(lane, p));
            float cs[8], sgn[8];
            if (d.chan_scale) {
                load8f(d.chan_scale, e0, d_in, 1, 1.0f, cs);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) cs[e] = 1.0f;
            }
            load8s(d.signs, e0, d_in, 1, sgn);
#pragma unroll
            for (int i = 0; i < 4; ++i) t[p][i] = pack2(cs[2 * i] * sgn[2 * i], cs[2 * i + 1] * sgn[2 * i + 1]);
            const int k0 = 4 * (oct0 + Lay::octet_after(lane, p));
            live[p] = k0 < n_pairs;
            if (!CALIB) {
                load4f(d.sigma, k0, n_pairs, 1, 1.0f, q[p]);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) q[p][i] = 1.0f;
            }
            const float fl = Lay::negated(lane, p) ? -1.0f : 1.0f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                // q_k = f32(1 / (double)sigma_k): the correctly rounded f32 reciprocal is the same number
                const float r = live[p] ? __frcp_rn(q[p][i]) : 0.f;
                // |z| <= q (1 + eps) because |y| <= 1 for a unit row: only a huge reciprocal pair scale can
                // carry a point beyond the table's reach
                risky |= !(r < 15000.0f);
                q[p][i] = fl * r;
            }
        }
        const bool any_risky = __any_sync(kFull, risky);

        const int col0 = seg * WE + 8 * NS * lane;  // first column of this thread
        const bool have_w = col0 < d_in;            // the fast path needs d_in to be a multiple of 8 NS: all or none
        const int seg_word0 = 4 * NS * B * seg;     // first packed word of this warp's segment (16 NS B bytes per segment)
        const bool last_seg = seg == n_seg - 1;
        double* part_base = &ss_part[0][group * n_seg];

        auto rows = [&](auto mode_tag) {
            constexpr int MODE = decltype(mode_tag)::value;  // 0 = table, 1 = table with reach check, 2 = exhaustive, 3 = polar, 4 = calibrate
            int parity = 0;
            double acc[NS][4];
            int used = 0;
#pragma unroll
            for (int p = 0; p < NS; ++p)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[p][i] = 0.0;
            // raw bits of the thread's elements of one row; the next row is fetched as soon as this one
            // has been converted, so its latency hides behind the rotation and the search
            constexpr int kRaw = BF16 ? 4 * NS : 8 * NS;
            uint32_t raw[kRaw];
            auto fetch = [&](int t) {
                const long long row = CALIB ? (long long)t * cur.d_out / n_cal : t;
                const char* wp = static_cast<const char*>(cur.W) + (row * cur.w_row_stride + col0) * kEsz;
#pragma unroll
                for (int h = 0; h < kRaw / 8; ++h) {
                    uint32_t w[8];
                    ld_global_256(wp + 32 * h, w);
#pragma unroll
                    for (int i = 0; i < 8; ++i) raw[8 * h + i] = w[i];
                }
            };
#pragma unroll
            for (int i = 0; i < kRaw; ++i) raw[i] = 0u;
            if (have_w) fetch(row0);
            for (int row = row0; row < row_end; row += row_step, parity ^= 1) {
                f32x2 P[NS][4];
                if (BF16) {
#pragma unroll
                    for (int i = 0; i < 4 * NS; ++i)
                        P[i >> 2][i & 3] = mul2(pack2(__uint_as_float(raw[i] << 16), __uint_as_float(raw[i] & 0xffff0000u)),
                                                t[i >> 2][i & 3]);
                } else {
#pragma unroll
                    for (int i = 0; i < 4 * NS; ++i)
                        P[i >> 2][i & 3] = mul2(pack2(__uint_as_float(raw[2 * i]), __uint_as_float(raw[2 * i + 1])), t[i >> 2][i & 3]);
                }
                if (have_w && row + row_step < row_end) fetch(row + row_step);
                // sum of squares of the row: ss = sum_j (double)x_j^2, per thread, per warp, then per row
                double* part = part_base + parity * 32;
                {
                    double ss = 0.0;
#pragma unroll
                    for (int p = 0; p < NS; ++p)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float x0, x1;
                            unpack2(P[p][i], x0, x1);
                            const double d0 = double(x0), d1 = double(x1);
                            ss = fma(d0, d0, ss);
                            ss = fma(d1, d1, ss);
                        }
                    ss = warp_sum(ss);
                    if (lane == 0) part[seg] = ss;
                }
                // The rotation does not need the norm, so the warps of the row meet only after it.  A
                // warp can be one row ahead of another at most, hence the two sets of partial sums.
                fwht2<NS, LOG2B, false>(P, lane);
                group_barrier(group, tg);
                float gn = 0.f;
                if (lane == 0) {  // every warp adds the same numbers in the same order
                    double total = 0.0;
                    for (int w = 0; w < n_seg; ++w) total += part[w];
                    const float r = float(sqrt(total));
                    // g = f32(c_b / r); 0 for a zero row (all its pairs become the origin) and for a non-finite
                    // row (its indices are unspecified; the searches accept any input)
                    if (isfinite(r) && r > 0.f) gn = __fdiv_rn(a.inv_sqrt_b, r);
                    if (seg == 0) {
                        if (!CALIB) cur.row_norm[row] = r;
                        if (!isfinite(r) && a.status) atomicOr(a.status, 1);
                    }
                }
                gn = __shfl_sync(kFull, gn, 0);
                const f32x2 gn2 = pack2(gn, gn);
                if constexpr (MODE == 4) {  // calibration: rows of zero (or non-finite) norm are skipped
                    if (gn != 0.f) {
                        ++used;
#pragma unroll
                        for (int p = 0; p < NS; ++p)
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                float y0, y1;
                                unpack2(mul2(P[p][i], gn2), y0, y1);
                                acc[p][i] += double(sqrtf(__fmaf_rn(y1, y1, __fmul_rn(y0, y0))));
                            }
                    }
                } else {
#pragma unroll
                for (int p = 0; p < NS; ++p) {
                    uint32_t v[4];
                    float2 z[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float yx, yy;
                        unpack2(mul2(P[p][i], gn2), yx, yy);
                        z[i] = make_float2(__fmul_rn(yx, q[p][i]), __fmul_rn(yy, q[p][i]));
                    }
                    if (MODE == 3) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) v[i] = uint32_t(search_polar(ps, z[i].x, z[i].y));
                    } else if (MODE == 0) {
                        uint2 rec[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) v[i] = uint32_t(search_cell(s, z[i].x, z[i].y, rec[i]));
                        // rare: one of the four cells has more than four candidates
                        if (int(cell_overflows(rec[0])) | int(cell_overflows(rec[1])) | int(cell_overflows(rec[2])) | int(cell_overflows(rec[3]))) {
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                if (cell_overflows(rec[i])) v[i] = uint32_t(search_overflow(s, rec[i], z[i].x, z[i].y));
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            v[i] = uint32_t(MODE == 2 ? search_exhaustive(s, z[i].x, z[i].y) : search_table(s, z[i].x, z[i].y));
                    }
                    // two indices fit a 32-bit word (B <= 12); octets beyond the row are staged as zero
                    unsigned long long packed4 =
                        (unsigned long long)(v[0] | (v[1] << B)) | ((unsigned long long)(v[2] | (v[3] << B)) << (2 * B));
                    if (!live[p]) packed4 = 0ull;
                    oct_s[Stage2<NS>::slot(Lay::octet_after(lane, p))] = packed4;
                }
                __syncwarp();
                // bit packing of the warp's segment: octet o occupies bits [o*4B, (o+1)*4B) (LSB first)
                const long long pstride = cur.packed_row_stride;
                uint32_t* out = reinterpret_cast<uint32_t*>(cur.packed + (long long)row * pstride);
                const int row_words = int(pstride >> 2);
                const int payload_words = int((((long long)(cur.d_in >> 1) * B + 7) / 8 + 3) / 4);
                for (int j = lane; j < 4 * NS * B; j += 32) {
                    const int gw = seg_word0 + j;
                    if (gw >= payload_words) break;
                    const unsigned bit0 = unsigned(j) * 32u;
                    int o = int(__umulhi(bit0, div_magic));  // floor(bit0 / (4B)), octet inside the segment
                    uint32_t word;
                    if (B4 >= 32) {
                        // an octet is at least as wide as a word: bits from octet o and, past its end, from o + 1
                        const int sh = int(bit0) - o * B4;  // 0 <= sh < 4B
                        const unsigned long long v0 = oct_s[Stage2<NS>::slot(o)];
                        const unsigned long long v1 = o + 1 < WE / 8 ? oct_s[Stage2<NS>::slot(o + 1)] : 0ull;
                        word = uint32_t(v0 >> sh) | uint32_t((v1 << (B4 - sh)) & 0xffffffffull);
                    } else {
                        word = 0;
                        for (; o < WE / 8; ++o) {
                            const int sh = o * B4 - int(bit0);
                            if (sh >= 32) break;
                            const unsigned long long v = oct_s[Stage2<NS>::slot(o)];
                            word |= sh >= 0 ? uint32_t(v << sh) : uint32_t(v >> (-sh));
                        }
                    }
                    out[gw] = word;
                }
                if (last_seg)  // padding up to the row stride is written as zero
                    for (int gw = payload_words + lane; gw < row_words; gw += 32) out[gw] = 0u;
                __syncwarp();  // the staging piece is free again
                }  // MODE != 4
            }
            if constexpr (MODE == 4) {  // this row group's sums go to its own slot of the matrix's workspace
                const int pair_stride = (n_pairs + 3) & ~3;
                const int slot = (int(blockIdx.x) - cur.calib_first_block) * groups + group;
                double* ws = reinterpret_cast<double*>(a.calib_base + cur.calib_offset);
                double* mine = ws + size_t(slot) * pair_stride;
#pragma unroll
                for (int p = 0; p < NS; ++p)
                    if (live[p]) {
                        const int k0 = 4 * (oct0 + Lay::octet_after(lane, p));
#pragma unroll
                        for (int i = 0; i < 4; ++i) mine[k0 + i] = acc[p][i];
                    }
                if (lane == 0 && seg == 0) ws[size_t(cur.calib_slots) * pair_stride + slot] = double(used);
            }
        };
        if constexpr (CALIB) {
            rows(std::integral_constant<int, 4>{});
        } else if constexpr (POLAR) {
            rows(std::integral_constant<int, 3>{});
        } else {
            if (a.brute) rows(std::integral_constant<int, 2>{});
            else if (any_risky) rows(std::integral_constant<int, 1>{});
            else rows(std::integral_constant<int, 0>{});
        }
    }
}

// sigma_k of every matrix from the slots of partial sums (zeroed before the calibration pass, so a
// slot nobody wrote counts as empty).  A block owns 32 pair positions of one matrix; its eight
// warps each add a contiguous slice of the slots in ascending order, and the eight slice sums are
// then added in ascending order: the result does not depend on timing.
constexpr int kFinishSlices = 8;
__global__ void __launch_bounds__(32 * kFinishSlices) calibrate_finish2_kernel(const MatDesc* descs,
                                                                             const unsigned char* calib_base) {
    __shared__ double part_sum[kFinishSlices][32], part_used[kFinishSlices];
    const MatDesc& d = descs[blockIdx.y];
    const int n_pairs = d.d_in >> 1, pair_stride = (n_pairs + 3) & ~3;
    if (int(blockIdx.x) * 32 >= n_pairs) return;
    const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + lane;
    const double* ws = reinterpret_cast<const double*>(calib_base + d.calib_offset);
    const int per = (d.calib_slots + kFinishSlices - 1) / kFinishSlices;
    const int s0 = min(d.calib_slots, slice * per), s1 = min(d.calib_slots, s0 + per);
    double sum = 0.0, used = 0.0;
    for (int slot = s0; slot < s1; ++slot) {
        if (k < n_pairs) sum += ws[size_t(slot) * pair_stride + k];
        if (lane == 0) used += ws[size_t(d.calib_slots) * pair_stride + slot];
    }
    part_sum[slice][lane] = sum;
    if (lane == 0) part_used[slice] = used;
    __syncthreads();
    if (slice == 0 && k < n_pairs) {
        double s = 0.0, u = 0.0;
        for (int i = 0; i < kFinishSlices; ++i) {
            s += part_sum[i][lane];
            u += part_used[i];
        }
        const double inv_sqrt_d = 1.0 / sqrt(double(d.d_in));
        double sg = u > 0.0 ? (s / u) / sqrt(1.5707963267948966) : inv_sqrt_d;  // Rayleigh mean = sigma sqrt(pi / 2)
        sg = fmax(sg, 1e-4 * inv_sqrt_d);
        const_cast<float*>(d.sigma)[k] = float(sg);
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
inline bool aligned(const void* p, uintptr_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; }

int pick_copies(int K, size_t budget) {
    int log2c = 4;
    while (log2c > 0 && (size_t(K) * 8 << log2c) > budget) --log2c;
    return log2c;
}

int launch_check(const char* what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_cuda_error(what, int(e));
        return QAMW_ERR_CUDA;
    }
    return QAMW_OK;
}

// cudaFuncSetAttribute once per kernel and device (the call is not free and the value never changes)
int raise_smem_limit(const void* kernel) {
    static std::mutex mu;
    static std::unordered_map<const void*, unsigned long long> done;  // kernel -> bit mask of devices
    int dev = 0;
    cudaGetDevice(&dev);
    const unsigned long long bit = 1ull << (dev & 63);
    std::lock_guard<std::mutex> lock(mu);
    unsigned long long& mask = done[kernel];
    if (mask & bit) return QAMW_OK;
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, kernel);
    if (e == cudaSuccess)  // the limit covers static and dynamic shared memory together
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemLimit - fa.sharedSizeBytes));
    if (e != cudaSuccess) {
        set_cuda_error("cudaFuncSetAttribute", int(e));
        return QAMW_ERR_NOMEM;
    }
    mask |= bit;
    return QAMW_OK;
}

template <int NS, int LOG2B>
int launch_decode2(const Decode2Args& a, int blocks, int threads, size_t smem, cudaStream_t st) {
    int rc = raise_smem_limit(reinterpret_cast<const void*>(&decode2_kernel<NS, LOG2B>));
    if (rc) return rc;
    decode2_kernel<NS, LOG2B><<<blocks, threads, smem, st>>>(a);
    return launch_check("decode2_kernel");
}

template <bool BF16, int LOG2B, int NS, int MAXT>
int launch_encode2(const Encode2Args& a, int blocks, int threads, size_t smem, cudaStream_t st) {
    if (a.calib_base) {
        int rc = raise_smem_limit(reinterpret_cast<const void*>(&encode2_kernel<BF16, LOG2B, NS, MAXT, 2>));
        if (rc) return rc;
        encode2_kernel<BF16, LOG2B, NS, MAXT, 2><<<blocks, threads, smem, st>>>(a);
        return launch_check("encode2_kernel (calibrate)");
    }
    if (a.polar_ba >= 0) {
        int rc = raise_smem_limit(reinterpret_cast<const void*>(&encode2_kernel<BF16, LOG2B, NS, MAXT, 1>));
        if (rc) return rc;
        encode2_kernel<BF16, LOG2B, NS, MAXT, 1><<<blocks, threads, smem, st>>>(a);
        return launch_check("encode2_kernel (polar)");
    }
    int rc = raise_smem_limit(reinterpret_cast<const void*>(&encode2_kernel<BF16, LOG2B, NS, MAXT, 0>));
    if (rc) return rc;
    encode2_kernel<BF16, LOG2B, NS, MAXT, 0><<<blocks, threads, smem, st>>>(a);
    return launch_check("encode2_kernel");
}

constexpr size_t kEncode2StaticSmem = 1024;  // ss_part and the current matrix descriptor, rounded up

}  // namespace

namespace qamw {

// Contiguous spans of the concatenated row list, one per block, of (nearly) equal cost.  A block works
// on `groups` rows at a time, each row step taking about the same time whatever the row length, so
// a row of matrix i costs 1 / groups_i: row_cost[i] = lcm / groups_i in integer units.
void make_spans(const MatDesc* descs, int n, int n_blocks, const int* row_cost, std::vector<int4>* out) {
    std::vector<long long> cum(n + 1, 0);
    for (int i = 0; i < n; ++i) cum[i + 1] = cum[i] + (long long)descs[i].d_out * row_cost[i];
    const long long total = cum[n];
    auto locate = [&](long long pos, int* m, int* row) {  // first row that starts at or after cost position `pos`
        int i = int(std::upper_bound(cum.begin(), cum.end(), pos) - cum.begin()) - 1;
        i = std::min(std::max(i, 0), n - 1);
        const long long r = (pos - cum[i] + row_cost[i] - 1) / row_cost[i];
        *m = i;
        *row = int(std::min<long long>(r, descs[i].d_out));
    };
    out->resize(n_blocks);
    int m0 = 0, r0 = 0;
    for (int k = 0; k < n_blocks; ++k) {
        int m1, r1;
        if (k == n_blocks - 1) {
            m1 = n - 1;
            r1 = descs[n - 1].d_out;
        } else {
            locate(total / n_blocks * (k + 1) + (total % n_blocks) * (k + 1) / n_blocks, &m1, &r1);
        }
        (*out)[k] = make_int4(m0, r0, m1, r1);
        m0 = m1;
        r0 = r1;
    }
}

int rows_decode(const MatDesc* descs_dev, const MatDesc* descs_host, int n, const void* spans_dev, int span_blocks,
                int block, int K, const float* codebook_dev, uint32_t flags, void* stream) {
    constexpr int NS = 4, WE = 256 * NS, kWarps = 16;
    const int log2b = ilog2(block);
    if (log2b < 5 || n <= 0) return QAMW_ERR_SHAPE;
    long long max_rows = 0;
    for (int i = 0; i < n; ++i) {
        const MatDesc& d = descs_host[i];
        if (d.d_in % 16 || d.d_in > WE * kWarps) return QAMW_ERR_SHAPE;
        if (!aligned(d.w_hat, 32) || !aligned(d.packed, 16) || d.packed_row_stride % 16) return QAMW_ERR_SHAPE;
        if (!aligned(d.chan_scale, 16) || !aligned(d.signs, 8) || !aligned(d.sigma, 16)) return QAMW_ERR_SHAPE;
        const int n_seg = (d.d_in + WE - 1) / WE;
        max_rows = std::max(max_rows, (long long)(d.d_out + kWarps / n_seg - 1) / (kWarps / n_seg));
    }
    if (max_rows == 0) return QAMW_OK;
    Decode2Args a;
    a.descs = descs_dev;
    a.one = descs_host[0];
    a.spans = static_cast<const int4*>(spans_dev);
    a.codebook = reinterpret_cast<const float2*>(codebook_dev);
    a.K = K;
    a.log2K = ilog2(K);
    a.seg_bytes = 16 * NS * a.log2K;
    a.stage_bytes = (a.seg_bytes + 16 + 127) & ~127;  // 128-byte aligned ring buffers
    a.inv_sqrt_b = float(1.0 / std::sqrt(double(block)));
    const size_t stage_total = size_t(kWarps) * kDecodeDepth * a.stage_bytes;
    a.log2c = pick_copies(K, std::min(size_t(128) * 1024, kSmemLimit - stage_total));
    const size_t smem = (size_t(K) * 8 << a.log2c) + stage_total;
    int grid = sm_count();
    if (flags & QAMW_FLAG_HALF_DEVICE) grid = std::max(1, grid / 2);
    const int blocks = spans_dev ? span_blocks : int(std::max<long long>(1, std::min<long long>(grid, max_rows)));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = QAMW_ERR_SHAPE;
    switch (log2b) {
        case 5: rc = launch_decode2<NS, 5>(a, blocks, kWarps * 32, smem, st); break;
        case 6: rc = launch_decode2<NS, 6>(a, blocks, kWarps * 32, smem, st); break;
        case 7: rc = launch_decode2<NS, 7>(a, blocks, kWarps * 32, smem, st); break;
        case 8: rc = launch_decode2<NS, 8>(a, blocks, kWarps * 32, smem, st); break;
        case 9: rc = launch_decode2<NS, 9>(a, blocks, kWarps * 32, smem, st); break;
        case 10: rc = launch_decode2<NS, 10>(a, blocks, kWarps * 32, smem, st); break;
        default: break;
    }
    return rc;
}

// Block sizes of the encoder: 20, 24 or 28 warps.  The register file is split over the four
// schedulers of an SM, 16384 registers each, so 5, 6 or 7 warps per scheduler leave 96, 80 or 72
// registers per thread.  A row of n_seg segments takes the size that keeps most warps busy (whole
// groups of n_seg warps, at most 15 groups), and among equals the smallest: 0 if the row is too long.
int encode_groups(int warps, int n_seg) { return std::min(15, warps / n_seg); }
int encode_warps(int n_seg) {
    int best = 0, best_busy = 0;
    for (int w = 20; w <= 28; w += 4) {
        const int busy = encode_groups(w, n_seg) * n_seg;
        if (busy > best_busy) {
            best = w;
            best_busy = busy;
        }
    }
    return best;
}
int decode_groups(int n_seg) { return 16 / n_seg; }
constexpr int kCostUnit = 360360;  // divisible by every group count 1..15

int rows_encode(const MatDesc* descs_dev, const MatDesc* descs_host, int n, const void* spans_dev, int span_blocks,
                int block, int K, int w_bf16, const ::qamw_codebook* cb, uint32_t flags, int32_t* status, void* stream,
                void* calib_base) {
    constexpr int NS = 2, WE = 256 * NS;
    const int log2b = ilog2(block);
    if (log2b < 5 || log2b > 9 || n <= 0) return QAMW_ERR_SHAPE;
    const size_t esz = w_bf16 ? 2 : 4;
    int max_seg = 1, warps = 0;
    long long rows = 0;
    for (int i = 0; i < n; ++i) {
        const MatDesc& d = descs_host[i];
        if (d.d_in % (8 * NS)) return QAMW_ERR_SHAPE;
        if (!aligned(d.W, 32) || (size_t(d.w_row_stride) * esz) % 32) return QAMW_ERR_SHAPE;
        if (!aligned(d.chan_scale, 16) || !aligned(d.signs, 8) || (!calib_base && !aligned(d.sigma, 16))) return QAMW_ERR_SHAPE;
        const int n_seg = (d.d_in + WE - 1) / WE;
        max_seg = std::max(max_seg, n_seg);
        warps = std::max(warps, encode_warps(n_seg));
        rows += d.d_out;
    }
    if (max_seg > warps) return QAMW_ERR_SHAPE;  // also: a row too long for any block size
    if (rows == 0) return QAMW_OK;
    Encode2Args a;
    a.descs = descs_dev;
    a.one = descs_host[0];
    a.spans = static_cast<const int4*>(spans_dev);
    a.calib_base = static_cast<unsigned char*>(calib_base);
    const bool calib = calib_base != nullptr;
    a.codebook = calib ? nullptr : static_cast<const float2*>(cb->d_blob);
    a.table = calib ? nullptr : reinterpret_cast<const uint4*>(static_cast<const unsigned char*>(cb->d_blob) + cb->off_cells);
    a.table_bytes = calib ? 0 : int(cb->blob_bytes - cb->off_cells);
    a.off_overflow = calib ? 0 : int(cb->off_overflow - cb->off_cells);
    a.K = K;
    a.log2K = ilog2(K);
    a.grid = calib ? 1 : cb->map.grid;
    a.map_zmax = calib ? 0.f : cb->map.zmax;
    a.map_c0 = calib ? 0.f : cb->map.c0;
    a.map_c1 = calib ? 0.f : cb->map.c1;
    a.map_c2 = calib ? 0.f : cb->map.c2;
    a.map_bias = calib ? 0.f : 12582912.0f + float(cb->map.half);
    a.brute = (flags & QAMW_FLAG_BRUTE_FORCE) ? 1 : 0;
    a.inv_sqrt_b = float(1.0 / std::sqrt(double(block)));
    a.status = status;
    const bool polar = !calib && cb->polar;
    a.polar_ba = polar ? cb->polar_ba : -1;
    a.polar_bp = polar ? cb->polar_bp : -1;
    const size_t fixed = ((size_t(a.table_bytes) + 15) & ~size_t(15)) + size_t(warps) * Stage2<NS>::kSlots * 8;
    if (!calib && fixed + size_t(K) * 8 > kSmemLimit - kEncode2StaticSmem) return QAMW_ERR_SHAPE;
    const bool tables = !calib && !polar;
    a.log2c = tables ? pick_copies(K, kSmemLimit - kEncode2StaticSmem - fixed) : 0;
    const size_t smem = fixed + (tables ? (size_t(K) * 8 << a.log2c) : 0);
    int grid = sm_count();
    if (flags & QAMW_FLAG_HALF_DEVICE) grid = std::max(1, grid / 2);
    const int blocks = spans_dev ? span_blocks : int(std::max<long long>(1, std::min<long long>(grid, rows)));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = QAMW_ERR_SHAPE;
#define QAMW_ENC2(LB)                                                                          \
    case LB:                                                                                   \
        if (warps == 28)                                                                       \
            rc = w_bf16 ? launch_encode2<true, LB, NS, 896>(a, blocks, 896, smem, st)          \
                        : launch_encode2<false, LB, NS, 896>(a, blocks, 896, smem, st);        \
        else if (warps == 24)                                                                  \
            rc = w_bf16 ? launch_encode2<true, LB, NS, 768>(a, blocks, 768, smem, st)          \
                        : launch_encode2<false, LB, NS, 768>(a, blocks, 768, smem, st);        \
        else                                                                                   \
            rc = w_bf16 ? launch_encode2<true, LB, NS, 640>(a, blocks, 640, smem, st)          \
                        : launch_encode2<false, LB, NS, 640>(a, blocks, 640, smem, st);        \
        break;
    switch (log2b) {
        QAMW_ENC2(5)
        QAMW_ENC2(6)
        QAMW_ENC2(7)
        QAMW_ENC2(8)
        QAMW_ENC2(9)
        default: break;
    }
#undef QAMW_ENC2
    return rc;
}

}  // namespace qamw

// ---------------------------------------------------------------------------------------------
// batches: all linear weights of a layer or a model behind one handle
// ---------------------------------------------------------------------------------------------
// A set of matrices that one launch of a row kernel walks: their descriptors on the device and one
// span of the concatenated row list per block.
struct RowSet {
    std::vector<int> index;         // positions in the batch
    std::vector<MatDesc> descs;     // host copy of the device array
    MatDesc* d_descs = nullptr;
    int4* d_spans = nullptr;
};

struct qamw_batch {
    int n = 0;
    int device = -1;
    int block = 0, K = 0, w_dtype = 0;
    const qamw_codebook* cb = nullptr;
    std::vector<qamw_matrix> items;
    int n_blocks = 0;
    RowSet dec;                     // all matrices, spans weighted for the decoder's geometry
    RowSet enc[3];                  // encoder: one set per block size (20, 24, 28 warps)
    int4* d_spans_dist = nullptr;   // distortion: spans of the concatenated work-item list, over dec.d_descs
    int n_blocks_dist = 0;
    double* d_dist_partial = nullptr;   // one record of four sums per (block, matrix of its span)
    DistOwner* d_dist_owner = nullptr;  // per matrix: first and last block whose span holds it, first record
    unsigned int* d_dist_counter = nullptr;  // ticket of the blocks; zero between launches
    MatDesc* d_cal_all = nullptr;       // calibration descriptors of all block-size classes, for the one finish launch
    int cal_all_n = 0, cal_all_max_pairs = 0;
    RowSet cal[3];                  // calibration: the encoder's sets again, spans over the calibration rows
    size_t cal_bytes = 0;           // partial-sum slots of all matrices (front of the caller's workspace)
    std::vector<size_t> ws_offset;  // calibration scratch of item i inside the caller's workspace
    size_t ws_bytes = 0;
};

namespace {
MatDesc make_desc(const qamw_matrix& it) {
    MatDesc d{};
    d.W = it.W;
    d.chan_scale = it.chan_scale;
    d.signs = it.signs;
    d.sigma = it.sigma;
    d.act_rms = it.act_rms;
    d.packed = it.packed;
    d.row_norm = it.row_norm;
    d.w_hat = it.w_hat_bf16;
    d.dist4 = it.dist4;
    d.w_row_stride = it.p.w_row_stride;
    d.packed_row_stride = it.p.packed_row_stride;
    d.d_out = it.p.d_out;
    d.d_in = it.p.d_in;
    return d;
}
}  // namespace

namespace {
void free_row_set(RowSet& r) {
    if (r.d_descs) cudaFree(r.d_descs);
    if (r.d_spans) cudaFree(r.d_spans);
    r.d_descs = nullptr;
    r.d_spans = nullptr;
}
cudaError_t upload_row_set(RowSet& r, int n_blocks, const std::vector<int>& row_cost) {
    if (r.descs.empty()) return cudaSuccess;
    std::vector<int4> spans;
    make_spans(r.descs.data(), int(r.descs.size()), n_blocks, row_cost.data(), &spans);
    cudaError_t e = cudaMalloc(&r.d_descs, sizeof(MatDesc) * r.descs.size());
    if (e == cudaSuccess) e = cudaMemcpy(r.d_descs, r.descs.data(), sizeof(MatDesc) * r.descs.size(), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMalloc(&r.d_spans, sizeof(int4) * spans.size());
    if (e == cudaSuccess) e = cudaMemcpy(r.d_spans, spans.data(), sizeof(int4) * spans.size(), cudaMemcpyHostToDevice);
    return e;
}
}  // namespace

extern "C" int qamw_batch_create(const qamw_matrix* items, int n, const qamw_codebook* cb, qamw_batch** out) {
    if (!items || n <= 0 || !cb || !out) return QAMW_ERR_ARG;
    *out = nullptr;
    for (int i = 0; i < n; ++i) {
        int rc = check_matrix_params(&items[i].p);
        if (rc) return rc;
        const qamw_params& p = items[i].p;
        if (p.block != items[0].p.block || p.K != items[0].p.K || p.w_dtype != items[0].p.w_dtype) return QAMW_ERR_ARG;
        if (p.K != cb->K || !items[i].signs) return QAMW_ERR_ARG;
        const size_t row_bytes = qamw_packed_row_bytes(p.d_in, p.K);
        if (p.packed_row_stride < (long long)row_bytes || p.packed_row_stride % 4) return QAMW_ERR_ALIGN;
        if (reinterpret_cast<uintptr_t>(items[i].packed) % 4) return QAMW_ERR_ALIGN;
    }
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) {
        set_cuda_error("qamw_batch_create", int(e));
        return QAMW_ERR_CUDA;
    }
    if (device != cb->device) return QAMW_ERR_ARG;  // the codebook lives on another device
    qamw_batch* b = new (std::nothrow) qamw_batch();
    if (!b) return QAMW_ERR_NOMEM;
    b->n = n;
    b->device = device;
    b->block = items[0].p.block;
    b->K = items[0].p.K;
    b->w_dtype = items[0].p.w_dtype;
    b->cb = cb;
    b->items.assign(items, items + n);
    b->n_blocks = sm_count();
    std::vector<int> dec_cost, enc_cost[3];
    for (int i = 0; i < n; ++i) {
        const MatDesc d = make_desc(items[i]);
        b->ws_offset.push_back(b->ws_bytes);
        b->ws_bytes += (qamw_calibrate_workspace_bytes(&items[i].p) + 255) & ~size_t(255);
        const int seg4 = (d.d_in + 1023) / 1024, seg2 = (d.d_in + 511) / 512;
        b->dec.index.push_back(i);
        b->dec.descs.push_back(d);
        dec_cost.push_back(kCostUnit / std::max(1, decode_groups(std::min(seg4, 16))));
        const int warps = encode_warps(seg2);
        const int c = warps == 20 ? 0 : (warps == 24 ? 1 : 2);  // rows too long for any size end up in the last set and fall back later
        b->enc[c].index.push_back(i);
        b->enc[c].descs.push_back(d);
        enc_cost[c].push_back(kCostUnit / std::max(1, encode_groups(warps ? warps : 28, std::min(seg2, 28))));
    }
    e = upload_row_set(b->dec, b->n_blocks, dec_cost);
    for (int c = 0; c < 3 && e == cudaSuccess; ++c) e = upload_row_set(b->enc[c], b->n_blocks, enc_cost[c]);
    for (int c = 0; c < 3 && e == cudaSuccess; ++c) {  // calibration: min(d_out, 1024) rows per matrix
        RowSet& r = b->cal[c];
        r.index = b->enc[c].index;
        r.descs = b->enc[c].descs;
        if (r.descs.empty()) continue;
        const int m = int(r.descs.size());
        std::vector<MatDesc> cal_rows(r.descs);
        for (MatDesc& d : cal_rows) d.d_out = std::min(d.d_out, QAMW_CALIB_MAX_ROWS);
        std::vector<int4> spans;
        make_spans(cal_rows.data(), m, b->n_blocks, enc_cost[c].data(), &spans);
        std::vector<int> first(size_t(m), b->n_blocks), last(size_t(m), -1);
        for (int k = 0; k < b->n_blocks; ++k)
            for (int i = spans[size_t(k)].x; i <= spans[size_t(k)].z; ++i) {
                first[size_t(i)] = std::min(first[size_t(i)], k);
                last[size_t(i)] = std::max(last[size_t(i)], k);
            }
        for (int i = 0; i < m; ++i) {
            MatDesc& d = r.descs[size_t(i)];
            const int groups = kCostUnit / enc_cost[c][size_t(i)];
            d.calib_first_block = first[size_t(i)];
            d.calib_slots = std::max(0, last[size_t(i)] - first[size_t(i)] + 1) * groups;
            d.calib_offset = (long long)b->cal_bytes;
            const size_t pair_stride = (size_t(d.d_in / 2) + 3) & ~size_t(3);
            b->cal_bytes += ((size_t(d.calib_slots) * (pair_stride + 1)) * sizeof(double) + 255) & ~size_t(255);
        }
        e = cudaMalloc(&r.d_descs, sizeof(MatDesc) * size_t(m));
        if (e == cudaSuccess) e = cudaMemcpy(r.d_descs, r.descs.data(), sizeof(MatDesc) * size_t(m), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMalloc(&r.d_spans, sizeof(int4) * spans.size());
        if (e == cudaSuccess) e = cudaMemcpy(r.d_spans, spans.data(), sizeof(int4) * spans.size(), cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) {  // all calibration descriptors in one array: one finish launch for every class
        std::vector<MatDesc> all;
        for (int c = 0; c < 3; ++c) all.insert(all.end(), b->cal[c].descs.begin(), b->cal[c].descs.end());
        b->cal_all_n = int(all.size());
        for (const MatDesc& d : all) b->cal_all_max_pairs = std::max(b->cal_all_max_pairs, d.d_in / 2);
        if (!all.empty()) {
            e = cudaMalloc(&b->d_cal_all, sizeof(MatDesc) * all.size());
            if (e == cudaSuccess) e = cudaMemcpy(b->d_cal_all, all.data(), sizeof(MatDesc) * all.size(), cudaMemcpyHostToDevice);
        }
    }
    if (e == cudaSuccess) {  // distortion: equal numbers of work items per block, sixteen blocks per SM
        std::vector<MatDesc> items_as_rows(b->dec.descs);
        std::vector<int> unit(size_t(n), 1);
        long long total = 0;
        for (int i = 0; i < n; ++i) {
            items_as_rows[size_t(i)].d_out = int(distortion_items(b->dec.descs[size_t(i)].d_out, b->dec.descs[size_t(i)].d_in));
            total += items_as_rows[size_t(i)].d_out;
        }
        b->n_blocks_dist = int(std::max<long long>(1, std::min<long long>(16LL * b->n_blocks, total)));
        std::vector<int4> spans;
        make_spans(items_as_rows.data(), n, b->n_blocks_dist, unit.data(), &spans);
        e = cudaMalloc(&b->d_spans_dist, sizeof(int4) * spans.size());
        if (e == cudaSuccess) e = cudaMemcpy(b->d_spans_dist, spans.data(), sizeof(int4) * spans.size(), cudaMemcpyHostToDevice);
        // per matrix: the blocks whose span holds it and where their records go
        std::vector<DistOwner> owner(size_t(n), DistOwner{int(spans.size()), -1, 0});
        for (size_t k = 0; k < spans.size(); ++k)
            for (int i = spans[k].x; i <= spans[k].z; ++i) {
                owner[size_t(i)].first = std::min(owner[size_t(i)].first, int(k));
                owner[size_t(i)].last = std::max(owner[size_t(i)].last, int(k));
            }
        int n_rec = 0;
        for (int i = 0; i < n; ++i) {
            owner[size_t(i)].offset = n_rec;
            n_rec += std::max(0, owner[size_t(i)].last - owner[size_t(i)].first + 1);
        }
        if (e == cudaSuccess) e = cudaMalloc(&b->d_dist_partial, sizeof(double) * 4 * size_t(std::max(1, n_rec)));
        if (e == cudaSuccess) e = cudaMalloc(&b->d_dist_owner, sizeof(DistOwner) * size_t(n));
        if (e == cudaSuccess) e = cudaMemcpy(b->d_dist_owner, owner.data(), sizeof(DistOwner) * size_t(n), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMalloc(&b->d_dist_counter, sizeof(unsigned int));
        if (e == cudaSuccess) e = cudaMemset(b->d_dist_counter, 0, sizeof(unsigned int));
    }
    if (e != cudaSuccess) {
        set_cuda_error("qamw_batch_create", int(e));
        qamw_batch_destroy(b);
        return QAMW_ERR_CUDA;
    }
    *out = b;
    return QAMW_OK;
}

extern "C" void qamw_batch_destroy(qamw_batch* b) {
    if (!b) return;
    free_row_set(b->dec);
    for (int c = 0; c < 3; ++c) {
        free_row_set(b->enc[c]);
        free_row_set(b->cal[c]);
    }
    if (b->d_spans_dist) cudaFree(b->d_spans_dist);
    if (b->d_dist_partial) cudaFree(b->d_dist_partial);
    if (b->d_dist_owner) cudaFree(b->d_dist_owner);
    if (b->d_dist_counter) cudaFree(b->d_dist_counter);
    if (b->d_cal_all) cudaFree(b->d_cal_all);
    delete b;
}

// The front of the workspace holds the slots of the batched pass, the rest the scratch of the
// single-matrix calls that matrices outside the common layout fall back to.
extern "C" size_t qamw_batch_workspace_bytes(const qamw_batch* b) { return b ? b->cal_bytes + b->ws_bytes : 0; }

extern "C" int qamw_calibrate_batch(const qamw_batch* b, void* workspace, size_t workspace_bytes, int32_t* status_out,
                                    void* stream) {
    if (!b || !workspace) return QAMW_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % 8) return QAMW_ERR_ALIGN;
    if (workspace_bytes < b->cal_bytes + b->ws_bytes) return QAMW_ERR_NOMEM;
    for (int i = 0; i < b->n; ++i)
        if (!b->items[i].W || !b->items[i].sigma) return QAMW_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t flags = b->items[0].p.flags;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    bool zeroed = false;
    // One pass per block size; the partial sums of all of them are finished by one launch, unless a class
    // had to go through the single-matrix kernels (then the classes that did not are finished one by one).
    bool fast[3] = {false, false, false}, any_general = false;
    for (int c = 0; c < 3; ++c) {
        const RowSet& set = b->cal[c];
        if (set.descs.empty()) continue;
        int rc = QAMW_ERR_SHAPE;
        if (!(flags & QAMW_FLAG_GENERAL_KERNELS)) {
            if (!zeroed) {  // a slot that no row group writes must read as empty
                cudaError_t e = cudaMemsetAsync(ws, 0, b->cal_bytes, st);
                if (e != cudaSuccess) {
                    set_cuda_error("cudaMemsetAsync", int(e));
                    return QAMW_ERR_CUDA;
                }
                zeroed = true;
            }
            rc = rows_encode(set.d_descs, set.descs.data(), int(set.descs.size()), set.d_spans, b->n_blocks, b->block, b->K,
                             b->w_dtype == QAMW_DTYPE_BF16, nullptr, flags, status_out, stream, ws);
            fast[c] = rc == QAMW_OK;
        }
        if (rc == QAMW_ERR_SHAPE) {  // some matrix of the set needs the general kernel: one call per matrix
            any_general = true;
            rc = QAMW_OK;
            for (size_t k = 0; k < set.index.size() && rc == QAMW_OK; ++k) {
                const int i = set.index[k];
                const qamw_matrix& it = b->items[i];
                rc = qamw_calibrate(it.W, &it.p, it.chan_scale, it.signs, it.sigma, ws + b->cal_bytes + b->ws_offset[i],
                                    workspace_bytes - b->cal_bytes - b->ws_offset[i], status_out, stream);
            }
        }
        if (rc) return rc;
    }
    if (!any_general && (fast[0] || fast[1] || fast[2])) {
        calibrate_finish2_kernel<<<dim3(unsigned((b->cal_all_max_pairs + 31) / 32), unsigned(b->cal_all_n)), 32 * kFinishSlices, 0,
                                   st>>>(b->d_cal_all, ws);
        return launch_check("calibrate_finish2_kernel");
    }
    for (int c = 0; c < 3; ++c) {
        if (!fast[c]) continue;
        const RowSet& set = b->cal[c];
        int max_pairs = 0;
        for (const MatDesc& d : set.descs) max_pairs = std::max(max_pairs, d.d_in / 2);
        calibrate_finish2_kernel<<<dim3(unsigned((max_pairs + 31) / 32), unsigned(set.descs.size())), 32 * kFinishSlices, 0,
                                   st>>>(set.d_descs, ws);
        const int rc = launch_check("calibrate_finish2_kernel");
        if (rc) return rc;
    }
    return QAMW_OK;
}

extern "C" int qamw_encode_batch(const qamw_batch* b, int32_t* status_out, void* stream) {
    if (!b) return QAMW_ERR_ARG;
    for (int i = 0; i < b->n; ++i) {
        const qamw_matrix& it = b->items[i];
        if (!it.W || !it.sigma || !it.packed || !it.row_norm) return QAMW_ERR_ARG;
    }
    const uint32_t flags = b->items[0].p.flags;
    for (int c = 0; c < 3; ++c) {  // one launch per block size
        const RowSet& set = b->enc[c];
        if (set.descs.empty()) continue;
        int rc = QAMW_ERR_SHAPE;
        if (!(flags & QAMW_FLAG_GENERAL_KERNELS))
            rc = rows_encode(set.d_descs, set.descs.data(), int(set.descs.size()), set.d_spans, b->n_blocks, b->block, b->K,
                             b->w_dtype == QAMW_DTYPE_BF16, b->cb, flags, status_out, stream);
        if (rc == QAMW_ERR_SHAPE) {  // some matrix of the class needs the general kernel: one call per matrix
            rc = QAMW_OK;
            for (size_t k = 0; k < set.index.size() && rc == QAMW_OK; ++k) {
                const qamw_matrix& it = b->items[set.index[k]];
                rc = qamw_encode(it.W, &it.p, it.chan_scale, it.signs, it.sigma, b->cb, it.packed, it.row_norm, status_out,
                                 stream);
            }
        }
        if (rc) return rc;
    }
    return QAMW_OK;
}

extern "C" int qamw_decode_batch(const qamw_batch* b, void* stream) {
    if (!b) return QAMW_ERR_ARG;
    for (int i = 0; i < b->n; ++i) {
        const qamw_matrix& it = b->items[i];
        if (!it.sigma || !it.packed || !it.row_norm || !it.w_hat_bf16) return QAMW_ERR_ARG;
    }
    const uint32_t flags = b->items[0].p.flags;
    int rc = QAMW_ERR_SHAPE;
    if (!(flags & QAMW_FLAG_GENERAL_KERNELS))
        rc = rows_decode(b->dec.d_descs, b->dec.descs.data(), b->n, b->dec.d_spans, b->n_blocks, b->block, b->K,
                         static_cast<const float*>(b->cb->d_blob), flags, stream);
    if (rc != QAMW_ERR_SHAPE) return rc;
    for (int i = 0; i < b->n; ++i) {  // some matrix needs the general kernel: one call per matrix
        const qamw_matrix& it = b->items[i];
        rc = qamw_decode(it.packed, it.row_norm, it.chan_scale, it.signs, it.sigma, b->cb, &it.p, it.w_hat_bf16, stream);
        if (rc) return rc;
    }
    return QAMW_OK;
}

extern "C" int qamw_distortion_batch(const qamw_batch* b, void* stream) {
    if (!b) return QAMW_ERR_ARG;
    for (int i = 0; i < b->n; ++i) {
        const qamw_matrix& it = b->items[i];
        if (!it.W || !it.w_hat_bf16 || !it.dist4) return QAMW_ERR_ARG;
    }
    DistReduce red;
    red.partial = b->d_dist_partial;
    red.owner = b->d_dist_owner;
    red.counter = b->d_dist_counter;
    return distortion_batch_launch(b->dec.d_descs, b->n, b->d_spans_dist, b->n_blocks_dist, b->w_dtype == QAMW_DTYPE_BF16,
                                   red, stream);
}
