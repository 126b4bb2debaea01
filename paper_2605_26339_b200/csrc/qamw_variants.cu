// Small device-side switches around the codec's path: metadata rounded to 16 bits (Section 3.2) and
// the optional direction renormalisation of the decoder (Section A.3).
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "qamw_internal.h"

using namespace qamw;

namespace {

__global__ void round_f16_kernel(float* v, size_t n) {
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < n; i += size_t(gridDim.x) * blockDim.x)
        v[i] = __half2float(__float2half_rn(v[i]));
}

// One warp per row: |yhat|^2 = sum_k sigma_k^2 |c_idx_k|^2 in double (lane-serial, then a shuffle
// tree), out = f32(r / |yhat|), 0 for an all-zero reconstruction.
__global__ void renorm_kernel(const uint8_t* packed, long long stride, const float* row_norm, const float* sigma,
                              const float2* codebook, int B, int d_out, int n_pairs, float* out) {
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= d_out) return;
    const uint32_t* w = reinterpret_cast<const uint32_t*>(packed + (long long)row * stride);
    const int n_words = int((((long long)n_pairs * B + 7) / 8 + 3) / 4);
    const uint32_t mask = (1u << B) - 1u;
    double ss = 0.0;
    for (int k = lane; k < n_pairs; k += 32) {
        const unsigned bit = unsigned(k) * unsigned(B);
        const int wi = int(bit >> 5);
        const uint32_t lo = w[wi], hi = wi + 1 < n_words ? w[wi + 1] : 0u;
        const uint32_t idx = __funnelshift_r(lo, hi, bit & 31u) & mask;
        const float2 c = __ldg(codebook + idx);
        const double sg = double(sigma[k]);
        const double cx = double(c.x) * sg, cy = double(c.y) * sg;
        ss += cx * cx + cy * cy;
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, s);
    if (lane == 0) out[row] = ss > 0.0 ? float(double(row_norm[row]) / sqrt(ss)) : 0.f;
}

int launched(const char* what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_cuda_error(what, int(e));
        return QAMW_ERR_CUDA;
    }
    return QAMW_OK;
}

}  // namespace

extern "C" int qamw_round_f16(float* values, size_t n, void* stream) {
    if (!values && n) return QAMW_ERR_ARG;
    if (n == 0) return QAMW_OK;
    const int blocks = int(std::min<size_t>((n + 255) / 256, size_t(8) * size_t(sm_count())));
    round_f16_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(values, n);
    return launched("round_f16_kernel");
}

extern "C" int qamw_renorm_row_norms(const uint8_t* packed, const float* row_norm, const float* sigma,
                                     const qamw_codebook* cb, const qamw_params* p, float* row_norm_out, void* stream) {
    int rc = check_matrix_params(p);
    if (rc) return rc;
    if (!packed || !row_norm || !sigma || !cb || !row_norm_out) return QAMW_ERR_ARG;
    if (cb->K != p->K) return QAMW_ERR_ARG;
    const size_t row_bytes = qamw_packed_row_bytes(p->d_in, p->K);
    if (p->packed_row_stride < (long long)row_bytes || p->packed_row_stride % 4) return QAMW_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(packed) % 4) return QAMW_ERR_ALIGN;
    if (p->d_out == 0) return QAMW_OK;
    const int warps = 8;
    renorm_kernel<<<(p->d_out + warps - 1) / warps, warps * 32, 0, static_cast<cudaStream_t>(stream)>>>(
        packed, p->packed_row_stride, row_norm, sigma, static_cast<const float2*>(cb->d_blob), ilog2(p->K), p->d_out,
        p->d_in / 2, row_norm_out);
    return launched("renorm_kernel");
}

// ---------------------------------------------------------------------------------------------
// FP32 issue-rate probe: the plain-ALU roofline that an exhaustive search would be measured against
// ---------------------------------------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(256) fma_probe_kernel(float* out, int iters, float a, float b) {
    float x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = float(threadIdx.x + i);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 16; ++u)
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = fmaf(x[i], a, b);  // eight independent chains
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += x[i];
    if (s == 12345.678f) out[0] = s;  // never true: keeps the chains alive
}
}  // namespace

extern "C" int qamw_measure_fp32_peak(float* scratch_dev, double* lane_inst_per_s_out) {
    if (!scratch_dev || !lane_inst_per_s_out) return QAMW_ERR_ARG;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return QAMW_ERR_CUDA;
    const int blocks = 8 * sm_count(), iters = 4096;
    fma_probe_kernel<<<blocks, 256>>>(scratch_dev, 64, 1.0000001f, 1e-9f);  // warm-up
    cudaEventRecord(e0);
    fma_probe_kernel<<<blocks, 256>>>(scratch_dev, iters, 1.0000001f, 1e-9f);
    cudaEventRecord(e1);
    cudaError_t e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess || !(ms > 0.f)) {
        set_cuda_error("qamw_measure_fp32_peak", int(e));
        return QAMW_ERR_CUDA;
    }
    *lane_inst_per_s_out = double(blocks) * 256.0 * double(iters) * 128.0 / (double(ms) * 1e-3);
    return QAMW_OK;
}
