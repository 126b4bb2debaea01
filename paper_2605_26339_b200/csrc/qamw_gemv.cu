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

}  // namespace

extern "C" size_t qamw_gemv_workspace_bytes(const qamw_params* p, int n_vec) {
    if (check_matrix_params(p) || n_vec < 1) return 0;
    return size_t(n_vec) * size_t(p->d_in) * sizeof(float);
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
