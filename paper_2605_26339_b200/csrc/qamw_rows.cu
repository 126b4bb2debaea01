// Row kernels of libqamw for the common layouts (16-byte aligned rows, d_in a multiple of 16,
// Hadamard blocks of 32 elements or more): one persistent launch walks any number of matrices.
//
// Geometry.
//   * A warp owns a "segment" of 256 * NS consecutive elements of a row: NS = 4 octets (32 elements)
//     per thread in the decoder, NS = 2 (16 elements) in the encoder, whose register budget then
//     allows 20 to 28 resident warps per SM instead of 15.  A row is owned by a group of
//     ceil(d_in / (256 NS)) warps; a block holds as many groups as fit and the grid is persistent.
//   * A launch takes an array of matrix descriptors.  Every block walks all matrices; the tables in
//     shared memory (codebook copies, cell records) are filled once per launch, and only the
//     per-column constants of a warp's segment are reloaded when the matrix changes.
//   * Walsh-Hadamard butterflies of a block of b elements: stages h = 1, 2, 4 inside an octet, then
//     one stage per octet slot bit inside the thread, then one "half exchange" per lane bit: a thread
//     keeps the slots whose top slot bit is 0, sends the others to its partner (lane ^ 2^j), and
//     computes both outputs (K + R, K - R) of the butterflies whose inputs it then holds.  Every
//     exchange uses the top slot bit, so after the last stage a thread holds runs of NS/2 adjacent
//     octets and the threads of a block cover consecutive runs: 32-byte stores that tile full
//     128-byte lines (decoder).  Which physical slot receives the sum and which the difference is
//     chosen so that the next stage can again keep slot 0 and send slot 1 without moving registers;
//     for threads that need the other placement the received value is multiplied by -1 first
//     (K - R, K + R).  An upper partner then holds R - K as K - R: some slots end up negated, by
//     a pattern that depends on the lane only and is folded into the per-column constants.
//     Stages run in ascending order of h with one f32 rounding per output, and a multiplication by
//     +-1 is exact, so the result is bit-identical to the plain butterfly.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <mutex>
#include <type_traits>
#include <unordered_map>

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
    // butterflies: NS consecutive octets per lane; odd lanes hold the two halves swapped
    __device__ static __forceinline__ int octet_before(int lane, int p) {
        return NS * lane + (S >= 1 ? (p ^ (TOP * (lane & 1))) : p);
    }
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
    // top slot bit (h = 8 for NS = 2, h = 16 for NS = 4).  An odd lane holds its halves swapped, so
    // its sum and difference change places: out_lo = s lo + hi, out_hi = lo - s hi with s = -1.
    if (Lay::S >= 1) {
        const float s0 = (lane & 1) ? -1.0f : 1.0f;
        const f32x2 sp = pack2(s0, s0), sn = pack2(-s0, -s0);
#pragma unroll
        for (int p = 0; p < TOP; ++p)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const f32x2 a = P[p][i], c = P[p + TOP][i];
                P[p][i] = fma2(a, sp, c);
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
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// ---------------------------------------------------------------------------------------------
// decoder
// ---------------------------------------------------------------------------------------------
struct Decode2Args {
    const MatDesc* descs;    // device array, or NULL: `one` is the only matrix
    MatDesc one;
    int n_mats;
    const float2* codebook;  // device, K entries
    int K, log2K, log2c;
    int seg_bytes;           // packed bytes of one warp segment: 16 * NS * B
    int stage_bytes;         // one staging buffer of a warp: seg_bytes + 16
    float inv_sqrt_b;
};

// A warp streams its segment of the packed row through its own two-deep shared-memory ring (16-byte
// asynchronous copies); nothing is shared between warps after the prologue, so there is no barrier.
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
    unsigned char* stage = smem + ((size_t(a.K) * 8) << a.log2c) + size_t(warp) * 2 * a.stage_bytes;
    const uint32_t stage_addr = smem_addr(stage);

    fill_codebook_copies(reinterpret_cast<float2*>(smem), a.codebook, a.K, a.log2c, true);
    // the 16 bytes after a staged segment are read (and masked away) by the last threads: keep them defined
    if (lane < 8) reinterpret_cast<uint32_t*>(stage + (lane >> 2) * a.stage_bytes + a.seg_bytes)[lane & 3] = 0u;
    __syncthreads();

    // where this thread's index bits sit inside a staged segment: two runs (physical slots with the
    // top slot bit 0 / 1), each 4 B TOP bits long
    uint32_t run_word[2], run_shift[2];
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        const unsigned bit0 = unsigned(4 * Lay::octet_before(lane, x * TOP)) * unsigned(B);
        run_word[x] = 4u * (bit0 >> 5);
        run_shift[x] = bit0 & 31u;
    }

    for (int m = 0; m < a.n_mats; ++m) {
        const MatDesc& d = a.descs ? a.descs[m] : a.one;
        const int d_in = d.d_in, d_out = d.d_out, n_pairs = d_in >> 1;
        const int n_seg = (d_in + WE - 1) / WE;
        const int groups = n_warps / n_seg;           // >= 1 (checked on the host)
        const int group = warp / n_seg, seg = warp - group * n_seg;
        if (group >= groups) continue;                // this warp has no segment in this matrix
        const uint8_t* packed = d.packed;
        const long long pstride = d.packed_row_stride;
        const int row_bytes = int((((long long)n_pairs * B + 7) / 8 + 15) & ~15LL);  // <= stride (a multiple of 16)
        const long long seg_off = (long long)seg * a.seg_bytes;
        const int seg_len = max(0, min(a.seg_bytes, row_bytes - int(seg_off)));
        const int n_chunks = seg_len >> 4;
        auto issue_row = [&](long long row, int buf) {
            const unsigned char* src = packed + row * pstride + seg_off;
            unsigned char* dst = stage + buf * a.stage_bytes;
            for (int c = lane; c < n_chunks; c += 32) cp_async(dst + (size_t(c) << 4), src + (size_t(c) << 4), 4);
            cp_async_commit();
        };
        const long long row_step = (long long)gridDim.x * groups;
        long long row = (long long)((blockIdx.x + 17u * unsigned(m)) % gridDim.x) * groups + group;
        __syncwarp();  // the previous matrix's last row has been read by every lane
        if (row < d_out) issue_row(row, 0);

        // per-column constants of this warp's segment
        const int oct0 = seg * (WE / 8);  // first octet of the segment
        float sg[NS][4];
        f32x2 mcol[NS][4];
        int e_out[NS];
#pragma unroll
        for (int p = 0; p < NS; ++p) {
            const int k0 = 4 * (oct0 + Lay::octet_before(lane, p));
            load4f(d.sigma, k0, n_pairs, 1, 0.f, sg[p]);
            const int e0 = 8 * (oct0 + Lay::octet_after(lane, p));
            e_out[p] = e0;
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
        __nv_bfloat16* out = static_cast<__nv_bfloat16*>(d.w_hat);
        const float* row_norm = d.row_norm;

        int buf = 0;
        for (; row < d_out; row += row_step, buf ^= 1) {
            const float rn = __ldg(row_norm + row);
            cp_async_wait_all();
            __syncwarp();  // every lane's part of this row has landed; the other buffer is no longer read
            if (row + row_step < d_out) issue_row(row + row_step, buf ^ 1);
            const uint32_t in = stage_addr + uint32_t(buf * a.stage_bytes);
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
            __nv_bfloat16* orow = out + row * d_in;
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
                const int e0 = e_out[p];
                if (e0 < d_in) {
                    if constexpr (NS == 4) {
                        st_global_256(orow + e0, w);
                    } else {
                        *reinterpret_cast<uint4*>(orow + e0) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
        cp_async_wait_all();
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
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemLimit));
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

}  // namespace

namespace qamw {

int rows_decode(const MatDesc* descs_dev, const MatDesc* descs_host, int n, int block, int K, const float* codebook_dev,
                uint32_t flags, void* stream) {
    constexpr int NS = 4, WE = 256 * NS, kWarps = 16;
    const int log2b = ilog2(block);
    if (log2b < 5 || n <= 0) return QAMW_ERR_SHAPE;
    long long max_rows = 0;
    int max_seg = 1;
    for (int i = 0; i < n; ++i) {
        const MatDesc& d = descs_host[i];
        if (d.d_in % 16 || d.d_in > WE * kWarps) return QAMW_ERR_SHAPE;
        if (!aligned(d.w_hat, 32) || !aligned(d.packed, 16) || d.packed_row_stride % 16) return QAMW_ERR_SHAPE;
        if (!aligned(d.chan_scale, 16) || !aligned(d.signs, 8) || !aligned(d.sigma, 16)) return QAMW_ERR_SHAPE;
        const int n_seg = (d.d_in + WE - 1) / WE;
        max_seg = std::max(max_seg, n_seg);
        max_rows = std::max(max_rows, (long long)(d.d_out + kWarps / n_seg - 1) / (kWarps / n_seg));
    }
    if (max_rows == 0) return QAMW_OK;
    Decode2Args a;
    a.descs = descs_dev;
    a.one = descs_host[0];
    a.n_mats = n;
    a.codebook = reinterpret_cast<const float2*>(codebook_dev);
    a.K = K;
    a.log2K = ilog2(K);
    a.seg_bytes = 16 * NS * a.log2K;
    a.stage_bytes = a.seg_bytes + 16;
    a.inv_sqrt_b = float(1.0 / std::sqrt(double(block)));
    const size_t stage_total = size_t(kWarps) * 2 * a.stage_bytes;
    a.log2c = pick_copies(K, std::min(size_t(128) * 1024, kSmemLimit - stage_total));
    const size_t smem = (size_t(K) * 8 << a.log2c) + stage_total;
    int grid = sm_count();
    if (flags & QAMW_FLAG_HALF_DEVICE) grid = std::max(1, grid / 2);
    const int blocks = int(std::max<long long>(1, std::min<long long>(grid, max_rows)));
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

}  // namespace qamw
