// Fused decode -> matrix-vector product: y = W_hat x straight from the packed stream, without ever
// writing W_hat (the paper's pipeline dequantises to BF16 before the matmul and names the fused kernel
// as its main engineering follow-up: Section 1, Limitations).
//
// Row i of the decoder's output is  w_hat_i = r_i D_s^-1 S F yhat_i  (Section 3.2, B.2), with
// yhat_i = (sigma_k c_idx_k)_k the scaled codewords and F the symmetric, orthonormal block Hadamard
// matrix (Lemma 1).  Hence
//     w_hat_i . x  =  r_i  yhat_i . (F S D_s^-1 x)  =  r_i  sum_k  c_idx_k . (sigma_k xt_k),
// where xt = R_fwd (x / s) is the *activation* rotated once per call.  The per-row inverse rotation
// disappears: a row costs one codeword gather and two fused multiply-adds per pair, and reads B/16
// bytes per weight instead of the 2 bytes of a BF16 matrix.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <mutex>
#include <unordered_map>

#include "qamw_device.cuh"
#include "qamw_internal.h"

using namespace qamw;

namespace {

// xt = F S (x / s), pair k scaled by sigma_k, for one activation vector per block; written chunk-
// transposed: pair 16 c + i of vector v at out[(v * 16 + i) * n_chunks + c], so that the lanes of the
// product kernel (one chunk of 16 pairs each) read consecutive addresses.
__global__ void gemv_rotate_kernel(const float* x, const float* chan_scale, const int8_t* signs, const float* sigma,
                                   int d_in, int log2b, float2* out) {
    extern __shared__ float v[];
    const int vec = blockIdx.x;
    const float* xv = x + size_t(vec) * d_in;
    for (int j = threadIdx.x; j < d_in; j += blockDim.x)
        v[j] = float(signs[j]) * xv[j] / (chan_scale ? chan_scale[j] : 1.0f);
    __syncthreads();
    for (int s = 0; s < log2b; ++s) {  // butterflies of every block, stage h = 2^s
        const int h = 1 << s;
        for (int t = threadIdx.x; t < d_in / 2; t += blockDim.x) {
            const int lo = ((t >> s) << (s + 1)) | (t & (h - 1));
            const float a = v[lo], c = v[lo + h];
            v[lo] = a + c;
            v[lo + h] = a - c;
        }
        __syncthreads();
    }
    const float scale = rsqrtf(float(1 << log2b));
    const int n_pairs = d_in >> 1, n_chunks = n_pairs >> 4;
    for (int k = threadIdx.x; k < n_pairs; k += blockDim.x) {
        const float sg = sigma[k] * scale;
        out[(size_t(vec) * 16 + (k & 15)) * n_chunks + (k >> 4)] = make_float2(v[2 * k] * sg, v[2 * k + 1] * sg);
    }
}

struct GemvArgs {
    const uint8_t* packed;
    long long stride;
    const float* row_norm;
    const float2* codebook;
    const float2* xt;  // rotated activations, chunk-transposed (see gemv_rotate_kernel)
    float* y;
    int d_out, n_pairs, K, B, log2c;
};

// One warp per row at a time, a lane per chunk of 16 pairs: 16 B index bits read as 32-bit words
// (rows are 4-byte aligned), cut with funnel shifts, codewords from bank-separated copies in shared
// memory, the rotated activations of all vectors from shared memory too.
template <int NVEC>
__global__ void __launch_bounds__(512, 1) gemv_kernel(const GemvArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int B = a.B;
    const uint32_t mask = (1u << B) - 1u;
    const uint32_t cb_stride = 8u << a.log2c;
    const uint32_t cb = smem_addr(smem) + 8u * (threadIdx.x & ((1 << a.log2c) - 1));
    const int n_chunks = a.n_pairs >> 4;
    float2* xs = reinterpret_cast<float2*>(smem + ((size_t(a.K) * 8) << a.log2c));
    fill_codebook_copies(reinterpret_cast<float2*>(smem), a.codebook, a.K, a.log2c);
    for (int i = threadIdx.x; i < NVEC * 16 * n_chunks; i += blockDim.x) xs[i] = a.xt[i];
    __syncthreads();
    const int words_per_chunk = B / 2;          // 16 B bits = B / 2 words when B is even ...
    const int row_words = int((((long long)a.n_pairs * B + 7) / 8 + 3) / 4);
    for (int row = blockIdx.x * n_warps + warp; row < a.d_out; row += gridDim.x * n_warps) {
        const uint32_t* w = reinterpret_cast<const uint32_t*>(a.packed + (long long)row * a.stride);
        float acc[NVEC];
#pragma unroll
        for (int v = 0; v < NVEC; ++v) acc[v] = 0.f;
        for (int c = lane; c < n_chunks; c += 32) {
            // ... and in general the chunk starts at bit 16 B c: word (B c) / 2, shift 16 (B c & 1)
            const unsigned bit0 = 16u * unsigned(B) * unsigned(c);
            const int w0 = int(bit0 >> 5);
            const uint32_t sh = bit0 & 31u;
            uint32_t word[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) word[i] = (i <= words_per_chunk + 1 && w0 + i < row_words) ? __ldg(w + w0 + i) : 0u;
            // shift the window down to bit 0, then cut two indices per step of 2 B bits
            uint32_t win[7];
#pragma unroll
            for (int i = 0; i < 7; ++i) win[i] = __funnelshift_r(word[i], word[i + 1], sh);
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint32_t i0 = win[0] & mask, i1 = (win[0] >> B) & mask;
                const float2 c0 = lds_f32x2(cb + i0 * cb_stride), c1 = lds_f32x2(cb + i1 * cb_stride);
#pragma unroll
                for (int v = 0; v < NVEC; ++v) {
                    const float2 x0 = xs[(v * 16 + 2 * t) * n_chunks + c], x1 = xs[(v * 16 + 2 * t + 1) * n_chunks + c];
                    acc[v] = fmaf(c0.x, x0.x, acc[v]);
                    acc[v] = fmaf(c0.y, x0.y, acc[v]);
                    acc[v] = fmaf(c1.x, x1.x, acc[v]);
                    acc[v] = fmaf(c1.y, x1.y, acc[v]);
                }
                if (t < 7) {
#pragma unroll
                    for (int i = 0; i < 6; ++i) win[i] = __funnelshift_r(win[i], win[i + 1], 2 * B);
                    win[6] >>= 2 * B;
                }
            }
        }
        const float rn = __ldg(a.row_norm + row);
#pragma unroll
        for (int v = 0; v < NVEC; ++v) {
            float s = acc[v];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFull, s, o);
            if (lane == 0) a.y[size_t(row) * NVEC + v] = rn * s;
        }
    }
}

__device__ __forceinline__ uint32_t lds_word(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// ---------------------------------------------------------------------------------------------
// Fast path (packed rows 16-byte aligned): column slices in registers.
//
// Block b owns rows b, b + gridDim, b + 2 gridDim, ...  Its warps form G row groups of S_par warps; a
// warp owns one *slice* of 512 pairs (1024 columns) and walks every G-th row of the block.  Lane l
// holds the rotated, scaled activations of chunk 32 slice + l (16 pairs, 32 floats per vector) in
// registers -- computed by the warp itself, since a slice is a whole number of Hadamard blocks -- so a
// pair costs one codeword gather and two fused multiply-adds per vector and nothing else on the
// shared-memory pipe.  The 64 B bytes of a row's slice arrive through a ring of 16-byte asynchronous
// copies, several rows ahead (one row in flight per warp leaves the memory system idle).  The slices'
// partial sums of a tile of rows meet in shared memory behind one block barrier per tile and are
// added in ascending slice order, so the result does not depend on timing.  Rows longer than the
// block has warps for are walked in several passes, each adding into y.
// ---------------------------------------------------------------------------------------------
struct Gemv2Args {
    const uint8_t* packed;
    long long stride;
    const float* x;           // [n_vec, d_in]
    const float* chan_scale;  // or NULL
    const int8_t* signs;
    const float* sigma;
    const float2* codebook;
    const float* row_norm;
    float* y;                 // [d_out][n_vec]
    int d_out, d_in, n_chunks, n_slices, K, B, log2c, log2b;
    int s_par;                // slices walked side by side: ceil(n_slices / passes)
    int seg_bytes, stage_bytes;
    float inv_sqrt_b;
};

template <int NVEC>
struct GemvGeom {
    static constexpr int kThreads = NVEC == 4 ? 320 : NVEC == 2 ? 384 : 512;  // 32 activation registers per thread and vector; warps per scheduler set the register cap
    static constexpr int kRowBatch = 4 / NVEC;              // rows whose sums are reduced together (four values)
    static constexpr int kDepth = NVEC == 4 ? 10 : NVEC == 2 ? 8 : 6;  // staged rows per warp: about 45 KB in flight per SM
    static constexpr int kTileRows = 32;                    // rows per warp between two block barriers
};

// Sums of four per-lane values over the warp with 6 shuffles instead of 20: the first two steps halve
// the number of values a lane carries.  Afterwards every lane holds the total of value
// 2 * bit4(lane) + bit3(lane).
__device__ __forceinline__ float warp_sum4(const float (&v)[4], int lane) {
    const bool hi = lane & 16;
    const float b0 = (hi ? v[2] : v[0]) + __shfl_xor_sync(kFull, hi ? v[0] : v[2], 16);
    const float b1 = (hi ? v[3] : v[1]) + __shfl_xor_sync(kFull, hi ? v[1] : v[3], 16);
    const bool h = lane & 8;
    float c = (h ? b1 : b0) + __shfl_xor_sync(kFull, h ? b0 : b1, 8);
    c += __shfl_xor_sync(kFull, c, 4);
    c += __shfl_xor_sync(kFull, c, 2);
    c += __shfl_xor_sync(kFull, c, 1);
    return c;
}

template <int N>
__device__ __forceinline__ void cp_async_wait_pending() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int NVEC>
__global__ void __launch_bounds__(GemvGeom<NVEC>::kThreads, 1) gemv2_kernel(const Gemv2Args a) {
    constexpr int RB = GemvGeom<NVEC>::kRowBatch, D = GemvGeom<NVEC>::kDepth;
    extern __shared__ __align__(16) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int B = a.B;
    const uint32_t mask = (1u << B) - 1u;
    const uint32_t cb_stride = 8u << a.log2c;
    const uint32_t cb = smem_addr(smem) + 8u * (threadIdx.x & ((1 << a.log2c) - 1));
    unsigned char* stage = smem + ((size_t(a.K) * 8) << a.log2c) + size_t(warp) * D * a.stage_bytes;
    const uint32_t stage_addr = smem_addr(stage);

    const int S = a.n_slices;
    const int S_par = a.s_par;                // slices walked side by side
    const int G = n_warps / S_par;            // row groups
    const bool in_group = warp < S_par * G;
    const int s0 = warp % S_par, g = warp / S_par;
    constexpr int JT = GemvGeom<NVEC>::kTileRows;
    const int TI = JT * G;                    // rows of the block per tile
    // rows of this block: blockIdx.x + gridDim.x * i, i < n_b
    const int n_b = int(blockIdx.x) < a.d_out ? (a.d_out - int(blockIdx.x) + int(gridDim.x) - 1) / int(gridDim.x) : 0;
    const int n_tiles = (n_b + TI - 1) / TI;
    float* ps_base = reinterpret_cast<float*>(smem + ((size_t(a.K) * 8) << a.log2c) + size_t(n_warps) * D * a.stage_bytes);
    // where the lane's 16 B index bits start inside a staged segment
    const uint32_t w_off = 4u * ((uint32_t(B) * uint32_t(lane)) >> 1), sh = ((uint32_t(B) * uint32_t(lane)) & 1u) * 16u;
    const int row_bytes = int(((((long long)(a.d_in >> 1)) * B + 7) / 8 + 15) & ~15LL);  // <= stride (a multiple of 16)
    const long long src_step = (long long)G * int(gridDim.x) * a.stride;
    int n_rows = 0;  // rows of the current pass for this warp

    // the ring of a warp: D staged rows of its slice, one commit group per row (empty past the end)
    const unsigned char* src = nullptr;
    bool copy0 = false, copy1 = false;
    int issued = 0;
    auto issue_row = [&]() {
        if (issued < n_rows) {
            unsigned char* dst = stage + (issued % D) * a.stage_bytes;
            if (copy0) cp_async(dst + (lane << 4), src + (lane << 4), 4);
            if (copy1) cp_async(dst + ((lane + 32) << 4), src + ((lane + 32) << 4), 4);
            src += src_step;
        }
        ++issued;
        cp_async_commit();
    };
    auto open_slice = [&](int slice) {
        const long long seg_off = (long long)slice * a.seg_bytes;
        const int n16 = max(0, min(a.seg_bytes, row_bytes - int(seg_off))) >> 4;  // at most 48 pieces of 16 bytes
        copy0 = lane < n16;
        copy1 = lane + 32 < n16;
        src = a.packed + ((long long)blockIdx.x + (long long)gridDim.x * g) * a.stride + seg_off;
        issued = 0;
        for (int i = 0; i < D - 1; ++i) issue_row();
    };
    auto rows_of = [&](int slice) { return in_group && slice < S && g < n_b ? (n_b - g + G - 1) / G : 0; };
    n_rows = rows_of(s0);
    if (n_rows > 0) open_slice(s0);  // the first rows travel while the tables are built
    fill_codebook_copies(reinterpret_cast<float2*>(smem), a.codebook, a.K, a.log2c);
    __syncthreads();

    for (int pass = 0; pass * S_par < S; ++pass) {
        const int slice = pass * S_par + s0;
        const int n_live = min(S_par, S - pass * S_par);
        if (pass > 0) {
            __syncthreads();  // the previous pass's sums have been read; its last rows too
            n_rows = rows_of(slice);
            if (n_rows > 0) open_slice(slice);
        }
        const int chunk = slice * 32 + lane;
        const bool valid = n_rows > 0 && chunk < a.n_chunks;
        // rotated activations of this lane's chunk: xr[v][2 i], xr[v][2 i + 1] = sigma_k (F S D_s^-1 x_v) at pair k = 16 chunk + i
        float xr[NVEC][32];
        if (valid) {
            const int col0 = 32 * chunk;
            const uint4* sp = reinterpret_cast<const uint4*>(a.signs + col0);
            const uint4 s0 = __ldg(sp), s1 = __ldg(sp + 1);
            const uint32_t sw[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};  // one sign byte per column
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                float tj[4];  // sign_j / s_j
#pragma unroll
                for (int i = 0; i < 4; ++i) tj[i] = float(int(int8_t((sw[e] >> (8 * i)) & 0xffu)));
                if (a.chan_scale) {
                    const float4 q = __ldg(reinterpret_cast<const float4*>(a.chan_scale + col0) + e);
                    tj[0] = __fdividef(tj[0], q.x);
                    tj[1] = __fdividef(tj[1], q.y);
                    tj[2] = __fdividef(tj[2], q.z);
                    tj[3] = __fdividef(tj[3], q.w);
                }
#pragma unroll
                for (int v = 0; v < NVEC; ++v) {
                    const float4 q = __ldg(reinterpret_cast<const float4*>(a.x + size_t(v) * a.d_in + col0) + e);
                    xr[v][4 * e] = q.x * tj[0];
                    xr[v][4 * e + 1] = q.y * tj[1];
                    xr[v][4 * e + 2] = q.z * tj[2];
                    xr[v][4 * e + 3] = q.w * tj[3];
                }
            }
        } else {
#pragma unroll
            for (int v = 0; v < NVEC; ++v)
#pragma unroll
                for (int e = 0; e < 32; ++e) xr[v][e] = 0.f;
        }
#pragma unroll
        for (int v = 0; v < NVEC; ++v) {
            float* t = xr[v];
#pragma unroll
            for (int st = 0; st < 5; ++st) {  // butterflies inside the lane's 32 columns
                if (st < a.log2b) {
                    const int h = 1 << st;
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (!(e & h)) {
                            const float lo = t[e], up = t[e + h];
                            t[e] = lo + up;
                            t[e + h] = lo - up;
                        }
                }
            }
            for (int st = 5; st < a.log2b; ++st) {  // blocks wider than a chunk: lanes 2^(st-5) apart
                const int m = 1 << (st - 5);
                const bool upper = lane & m;
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float o = __shfl_xor_sync(kFull, t[e], m);
                    t[e] = upper ? o - t[e] : t[e] + o;
                }
            }
        }
        if (valid) {
            const float4* gp = reinterpret_cast<const float4*>(a.sigma + 16 * chunk);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float4 q = __ldg(gp + e);
                const float sg[4] = {q.x * a.inv_sqrt_b, q.y * a.inv_sqrt_b, q.z * a.inv_sqrt_b, q.w * a.inv_sqrt_b};
#pragma unroll
                for (int v = 0; v < NVEC; ++v)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        xr[v][8 * e + 2 * i] *= sg[i];
                        xr[v][8 * e + 2 * i + 1] *= sg[i];
                    }
            }
        }

        for (int tile = 0; tile < n_tiles; ++tile) {
            float* ps = ps_base + (tile & 1) * (S_par * TI * NVEC);  // [slice][row of the tile][vector]
            for (int jj = 0; jj < JT; jj += RB) {
                const int it = tile * JT + jj;  // this warp's row counter
                if (it >= n_rows) break;
                float acc[4] = {0.f, 0.f, 0.f, 0.f};  // RB rows x NVEC vectors
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    if (it + r >= n_rows) break;
                    cp_async_wait_pending<D - 2>();
                    __syncwarp();  // every lane's part of this row has landed; the buffer refilled next is no longer read
                    issue_row();
                    const uint32_t in = stage_addr + uint32_t(((it + r) % D) * a.stage_bytes) + w_off;
                    uint32_t word[6], win[6];
#pragma unroll
                    for (int i = 0; i < 6; ++i) word[i] = lds_word(in + 4u * i);
#pragma unroll
                    for (int i = 0; i < 5; ++i) win[i] = __funnelshift_r(word[i], word[i + 1], sh);
                    win[5] = word[5] >> sh;
#pragma unroll
                    for (int t = 0; t < 8; ++t) {  // two indices per step of 2 B bits
                        const uint32_t i0 = win[0] & mask, i1 = (win[0] >> B) & mask;
                        const float2 c0 = lds_f32x2(cb + i0 * cb_stride), c1 = lds_f32x2(cb + i1 * cb_stride);
#pragma unroll
                        for (int v = 0; v < NVEC; ++v) {
                            float sum = acc[r * NVEC + v];
                            sum = fmaf(c0.x, xr[v][4 * t], sum);
                            sum = fmaf(c0.y, xr[v][4 * t + 1], sum);
                            sum = fmaf(c1.x, xr[v][4 * t + 2], sum);
                            sum = fmaf(c1.y, xr[v][4 * t + 3], sum);
                            acc[r * NVEC + v] = sum;
                        }
                        if (t < 7) {
#pragma unroll
                            for (int i = 0; i < 5; ++i) win[i] = __funnelshift_r(win[i], win[i + 1], 2 * B);
                            win[5] >>= 2 * B;
                        }
                    }
                }
                const float total = warp_sum4(acc, lane);
                if ((lane & 7) == 0) {  // lanes 0, 8, 16, 24 hold values 0, 1, 2, 3
                    const int id = lane >> 3, r = id / NVEC, v = id - r * NVEC;
                    if (it + r < n_rows) ps[(s0 * TI + (jj + r) * G + g) * NVEC + v] = total;
                }
            }
            __syncthreads();  // the tile's partial sums are complete
            for (int idx = threadIdx.x; idx < TI * NVEC; idx += blockDim.x) {
                const int il = idx / NVEC, v = idx - il * NVEC;
                const int i = tile * TI + il;
                if (i >= n_b) continue;
                const long long row = (long long)blockIdx.x + (long long)gridDim.x * i;
                float sum = 0.f;
                for (int sl = 0; sl < n_live; ++sl) sum += ps[(sl * TI + il) * NVEC + v];
                sum *= __ldg(a.row_norm + row);
                if (pass == 0) a.y[row * NVEC + v] = sum;
                else a.y[row * NVEC + v] += sum;
            }
        }
        cp_async_wait_all();
    }
}

int gemv_check(const char* what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_cuda_error(what, int(e));
        return QAMW_ERR_CUDA;
    }
    return QAMW_OK;
}

template <int NVEC>
int launch_gemv(const GemvArgs& a, int blocks, size_t smem, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(gemv_kernel<NVEC>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemLimit));
    if (e != cudaSuccess) {
        set_cuda_error("cudaFuncSetAttribute", int(e));
        return QAMW_ERR_NOMEM;
    }
    gemv_kernel<NVEC><<<blocks, 512, smem, st>>>(a);
    return gemv_check("gemv_kernel");
}

// cudaFuncSetAttribute once per kernel and device
int gemv_raise_smem(const void* kernel) {
    static std::mutex mu;
    static std::unordered_map<const void*, unsigned long long> done;
    int dev = 0;
    cudaGetDevice(&dev);
    const unsigned long long bit = 1ull << (dev & 63);
    std::lock_guard<std::mutex> lock(mu);
    unsigned long long& m = done[kernel];
    if (m & bit) return QAMW_OK;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemLimit));
    if (e != cudaSuccess) {
        set_cuda_error("cudaFuncSetAttribute", int(e));
        return QAMW_ERR_NOMEM;
    }
    m |= bit;
    return QAMW_OK;
}

template <int NVEC>
int launch_gemv2(const Gemv2Args& a, int sms, cudaStream_t st) {
    constexpr int kThreads = GemvGeom<NVEC>::kThreads, kWarps = kThreads / 32;
    // as many passes as the warps of a block require, the slices spread evenly over them
    const int passes = (a.n_slices + kWarps - 1) / kWarps;
    const int S_par = (a.n_slices + passes - 1) / passes, G = kWarps / S_par;
    Gemv2Args b = a;
    b.s_par = S_par;
    const int threads = 32 * S_par * G;
    const size_t sums = size_t(2) * S_par * GemvGeom<NVEC>::kTileRows * G * NVEC * sizeof(float);
    const size_t smem = (size_t(a.K) * 8 << a.log2c) + size_t(S_par * G) * GemvGeom<NVEC>::kDepth * a.stage_bytes + sums;
    if (smem > kSmemLimit) return QAMW_ERR_NOMEM;
    int rc = gemv_raise_smem(reinterpret_cast<const void*>(&gemv2_kernel<NVEC>));
    if (rc) return rc;
    const int blocks = std::max(1, std::min(sms, a.d_out));
    gemv2_kernel<NVEC><<<blocks, threads, smem, st>>>(b);
    return gemv_check("gemv2_kernel");
}

int gemv_slices(int d_in) { return (d_in / 32 + 31) / 32; }

}  // namespace

extern "C" size_t qamw_gemv_workspace_bytes(const qamw_params* p, int n_vec) {
    if (check_matrix_params(p) || n_vec < 1) return 0;
    return size_t(n_vec) * size_t(p->d_in) * sizeof(float);  // the layout-agnostic kernel's rotated activations
}

extern "C" int qamw_decode_gemv(const uint8_t* packed, const float* row_norm, const float* chan_scale,
                                const int8_t* signs, const float* sigma, const qamw_codebook* cb, const qamw_params* p,
                                const float* x, int n_vec, float* y_out, void* workspace, size_t workspace_bytes,
                                void* stream) {
    int rc = check_matrix_params(p);
    if (rc) return rc;
    if (!packed || !row_norm || !signs || !sigma || !cb || !x || !y_out || !workspace) return QAMW_ERR_ARG;
    if (cb->K != p->K) return QAMW_ERR_ARG;
    if (n_vec != 1 && n_vec != 2 && n_vec != 4) return QAMW_ERR_ARG;
    if (p->d_in % 32) return QAMW_ERR_SHAPE;  // whole chunks of 16 pairs
    const size_t row_bytes = qamw_packed_row_bytes(p->d_in, p->K);
    if (p->packed_row_stride < (long long)row_bytes || p->packed_row_stride % 4) return QAMW_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(packed) % 4 || reinterpret_cast<uintptr_t>(workspace) % 8) return QAMW_ERR_ALIGN;
    if (workspace_bytes < qamw_gemv_workspace_bytes(p, n_vec)) return QAMW_ERR_NOMEM;
    if (p->d_out == 0) return QAMW_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool general = (p->flags & QAMW_FLAG_GENERAL_KERNELS) != 0;
    if (!general && reinterpret_cast<uintptr_t>(packed) % 16 == 0 && p->packed_row_stride % 16 == 0 &&
        reinterpret_cast<uintptr_t>(x) % 16 == 0) {
        Gemv2Args g;
        g.packed = packed;
        g.stride = p->packed_row_stride;
        g.x = x;
        g.chan_scale = chan_scale;
        g.signs = signs;
        g.sigma = sigma;
        g.codebook = static_cast<const float2*>(cb->d_blob);
        g.row_norm = row_norm;
        g.y = y_out;
        g.d_out = p->d_out;
        g.d_in = p->d_in;
        g.n_chunks = p->d_in / 32;
        g.n_slices = gemv_slices(p->d_in);
        g.K = p->K;
        g.B = ilog2(p->K);
        g.log2b = ilog2(p->block);
        g.log2c = 4;
        while (g.log2c > 0 && (size_t(p->K) * 8 << g.log2c) > size_t(128) * 1024) --g.log2c;
        g.seg_bytes = 64 * g.B;
        g.stage_bytes = (g.seg_bytes + 32 + 127) & ~127;  // a lane reads six words from its first one
        g.inv_sqrt_b = 1.0f / std::sqrt(float(p->block));
        const int sms = sm_count();
        return n_vec == 1 ? launch_gemv2<1>(g, sms, st) : n_vec == 2 ? launch_gemv2<2>(g, sms, st) : launch_gemv2<4>(g, sms, st);
    }
    const size_t x_bytes = size_t(n_vec) * p->d_in * sizeof(float);
    if (x_bytes + size_t(p->K) * 8 > kSmemLimit || size_t(p->d_in) * sizeof(float) > kSmemLimit) return QAMW_ERR_NOMEM;
    float2* xt = static_cast<float2*>(workspace);
    if (size_t(p->d_in) * sizeof(float) > 48 * 1024) {  // beyond the default dynamic limit
        cudaError_t e = cudaFuncSetAttribute(gemv_rotate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemLimit));
        if (e != cudaSuccess) {
            set_cuda_error("cudaFuncSetAttribute", int(e));
            return QAMW_ERR_NOMEM;
        }
    }
    gemv_rotate_kernel<<<n_vec, 1024, size_t(p->d_in) * sizeof(float), st>>>(x, chan_scale, signs, sigma, p->d_in,
                                                                           ilog2(p->block), xt);
    rc = gemv_check("gemv_rotate_kernel");
    if (rc) return rc;
    GemvArgs a;
    a.packed = packed;
    a.stride = p->packed_row_stride;
    a.row_norm = row_norm;
    a.codebook = static_cast<const float2*>(cb->d_blob);
    a.xt = xt;
    a.y = y_out;
    a.d_out = p->d_out;
    a.n_pairs = p->d_in / 2;
    a.K = p->K;
    a.B = ilog2(p->K);
    a.log2c = 4;
    while (a.log2c > 0 && (size_t(p->K) * 8 << a.log2c) + x_bytes > std::min(kSmemLimit, size_t(128) * 1024 + x_bytes)) --a.log2c;
    const size_t smem = (size_t(p->K) * 8 << a.log2c) + x_bytes;
    const int blocks = std::max(1, std::min(sm_count(), (p->d_out + 15) / 16));
    if (n_vec == 1) return launch_gemv<1>(a, blocks, smem, st);
    if (n_vec == 2) return launch_gemv<2>(a, blocks, smem, st);
    return launch_gemv<4>(a, blocks, smem, st);
}
