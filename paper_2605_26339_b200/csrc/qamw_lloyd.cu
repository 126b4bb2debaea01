// Codebook training on the device (Section 3.6: Lloyd iterations on the unit circular Gaussian).
//
// One iteration = an exact assignment pass (every sample against every codeword, in double, lowest
// index on ties) and a centroid pass.  The centroid pass is arranged so that every cell's samples
// are added in sample order by one thread: the samples are first sorted by cell with a stable
// counting sort (per-chunk histograms, one exclusive scan, a scatter that ranks equal keys inside a
// warp by lane), which is deterministic, and the sums then are bit for bit those of a sequential
// loop over the samples.  Training therefore gives the same codebook run after run.
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdint>
#include <vector>

#include "qamw_internal.h"

using namespace qamw;

namespace {

constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kAssignThreads = 256;
constexpr int kChunk = 4096;  // samples per sorting chunk (one warp sorts a chunk)

__device__ __forceinline__ unsigned long long mix64(unsigned long long x) {  // SplitMix64 finaliser
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ULL;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBULL;
    x ^= x >> 31;
    return x;
}

// Unit circular Gaussian samples by Box-Muller from the counter stream of the header: sample i uses
// the uniforms of counters 2i and 2i+1.
__global__ void sample_kernel(unsigned long long key, unsigned long long n, double2* out) {
    const unsigned long long golden = 0x9E3779B97F4A7C15ULL;
    for (unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; i < n;
         i += (unsigned long long)gridDim.x * blockDim.x) {
        const double u1 = (double(mix64(key + golden * (2 * i + 1)) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
        const double u2 = (double(mix64(key + golden * (2 * i + 2)) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
        const double rad = sqrt(-2.0 * log(u1));
        double s, c;
        sincos(6.283185307179586476925286766559 * u2, &s, &c);
        out[i] = make_double2(rad * c, rad * s);
    }
}

// Exact nearest codeword of every sample: d = dx*dx + dy*dy with one rounding per operation (no
// fused multiply-add: the result must not depend on how a compiler contracts the expression), a
// later codeword wins only when strictly closer.  The codebook sits in shared memory and every
// lane reads the same entry (a broadcast).  Also adds up the distances of the block's samples in a
// fixed order (thread-serial, then a shuffle tree, then by warp).
__global__ void __launch_bounds__(kAssignThreads) assign_kernel(const double2* samples, unsigned long long n,
                                                                const double2* codebook, int K, int* assign,
                                                                double* block_err) {
    extern __shared__ double2 cb[];
    __shared__ double warp_err[kAssignThreads / 32];
    for (int c = threadIdx.x; c < K; c += blockDim.x) cb[c] = codebook[c];
    __syncthreads();
    double err = 0.0;
    for (unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; i < n;
         i += (unsigned long long)gridDim.x * blockDim.x) {
        const double2 z = samples[i];
        double best = INFINITY;
        int arg = 0;
#pragma unroll 4
        for (int c = 0; c < K; ++c) {
            const double dx = __dsub_rn(z.x, cb[c].x), dy = __dsub_rn(z.y, cb[c].y);
            const double d = __dadd_rn(__dmul_rn(dx, dx), __dmul_rn(dy, dy));
            if (d < best) {
                best = d;
                arg = c;
            }
        }
        if (assign) assign[i] = arg;
        err += best;
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) err += __shfl_xor_sync(kFullMask, err, s);
    if ((threadIdx.x & 31) == 0) warp_err[threadIdx.x >> 5] = err;
    __syncthreads();
    if (threadIdx.x == 0) {
        double e = 0.0;
        for (int w = 0; w < kAssignThreads / 32; ++w) e += warp_err[w];
        block_err[blockIdx.x] = e;
    }
}

// Histogram of the cells of one chunk of samples: hist[cell * n_chunks + chunk].
__global__ void hist_kernel(const int* assign, unsigned long long n, int K, int n_chunks, int* hist) {
    extern __shared__ int h[];
    for (int c = threadIdx.x; c < K; c += blockDim.x) h[c] = 0;
    __syncthreads();
    const unsigned long long lo = (unsigned long long)blockIdx.x * kChunk, hi = min(n, lo + kChunk);
    for (unsigned long long i = lo + threadIdx.x; i < hi; i += blockDim.x) atomicAdd(&h[assign[i]], 1);
    __syncthreads();
    for (int c = threadIdx.x; c < K; c += blockDim.x) hist[(size_t)c * n_chunks + blockIdx.x] = h[c];
}

// Exclusive scan of hist in (cell, chunk) order, in place, by one block (K * n_chunks entries, some
// hundred thousand); cell_start[c] = first position of cell c, cell_start[K] = n.
__global__ void scan_kernel(int* hist, int total, int K, int n_chunks, int* cell_start) {
    __shared__ int carry, part[1024];
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < total; base += blockDim.x) {
        const int i = base + threadIdx.x;
        const int v = i < total ? hist[i] : 0;
        part[threadIdx.x] = v;
        __syncthreads();
        for (int s = 1; s < blockDim.x; s <<= 1) {  // Hillis-Steele inclusive scan
            const int add = threadIdx.x >= s ? part[threadIdx.x - s] : 0;
            __syncthreads();
            part[threadIdx.x] += add;
            __syncthreads();
        }
        const int excl = carry + part[threadIdx.x] - v;
        if (i < total) {
            hist[i] = excl;
            if (i % n_chunks == 0) cell_start[i / n_chunks] = excl;
        }
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry += part[threadIdx.x];
        __syncthreads();
    }
    if (threadIdx.x == 0) cell_start[K] = carry;
}

// Stable scatter: one warp walks its chunk 32 samples at a time; lanes with the same cell are ranked
// by lane, the cell's cursor (from the scan) advances by their number.  order[pos] = sample index.
__global__ void scatter_kernel(const int* assign, unsigned long long n, int K, int n_chunks, const int* offsets,
                               int* order) {
    extern __shared__ int cursor[];
    const int chunk = blockIdx.x, lane = threadIdx.x;
    for (int c = lane; c < K; c += 32) cursor[c] = offsets[(size_t)c * n_chunks + chunk];
    __syncwarp();
    const unsigned long long lo = (unsigned long long)chunk * kChunk, hi = min(n, lo + kChunk);
    for (unsigned long long base = lo; base < hi; base += 32) {
        const unsigned long long i = base + lane;
        const bool live = i < hi;
        const int cell = live ? assign[i] : -1 - lane;  // dead lanes get keys of their own
        const unsigned peers = __match_any_sync(kFullMask, cell);
        const int rank = __popc(peers & ((1u << lane) - 1u));
        int pos = 0;
        if (live) pos = cursor[cell] + rank;
        __syncwarp();
        if (live && rank == 0) cursor[cell] += __popc(peers);
        __syncwarp();
        if (live) order[pos] = int(i);
    }
}

// New codewords: thread c adds the samples of cell c in sample order and divides by their number;
// an empty cell keeps its codeword.
__global__ void centroid_kernel(const double2* samples, const int* order, const int* cell_start, int K,
                                double2* codebook) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= K) return;
    const int lo = cell_start[c], hi = cell_start[c + 1];
    if (hi <= lo) return;
    double sx = 0.0, sy = 0.0;
    for (int k = lo; k < hi; ++k) {
        const double2 z = samples[order[k]];
        sx += z.x;
        sy += z.y;
    }
    const double cnt = double(hi - lo);
    codebook[c] = make_double2(sx / cnt, sy / cnt);
}

}  // namespace

namespace {
struct DeviceBuffers {  // frees whatever was allocated when it goes out of scope
    std::vector<void*> ptrs;
    ~DeviceBuffers() {
        for (void* p : ptrs) cudaFree(p);
    }
    template <class T>
    cudaError_t alloc(T** out, size_t count) {
        void* p = nullptr;
        cudaError_t e = cudaMalloc(&p, sizeof(T) * std::max<size_t>(count, 1));
        if (e == cudaSuccess) ptrs.push_back(p);
        *out = static_cast<T*>(p);
        return e;
    }
};
}  // namespace

extern "C" int qamw_train_codebook_gpu(int K, uint64_t n_samples, uint64_t seed, const double* samples_dev,
                                       int max_iters, double rel_tol, float* codebook_out, double* train_mse_out,
                                       int* iters_out, double* mse_trace_out, double* seconds_out) {
    if (!codebook_out) return QAMW_ERR_ARG;
    if (K < 1 || K > QAMW_MAX_K || !is_pow2(K)) return QAMW_ERR_SHAPE;
    if (n_samples < uint64_t(K) || n_samples >= (uint64_t(1) << 31) || max_iters < 0 || !(rel_tol >= 0.0)) return QAMW_ERR_ARG;
    const auto t_begin = std::chrono::steady_clock::now();
    const unsigned long long n = n_samples;
    const int n_chunks = int((n + kChunk - 1) / kChunk);
    const int assign_blocks = std::max(1, std::min(int((n + kAssignThreads - 1) / kAssignThreads), 8 * sm_count()));
    DeviceBuffers buf;
    double2 *d_samples = nullptr, *d_cb = nullptr;
    int *d_assign = nullptr, *d_hist = nullptr, *d_start = nullptr, *d_order = nullptr;
    double* d_err = nullptr;
    cudaError_t e = cudaSuccess;
    auto ok = [&](cudaError_t r) {
        if (e == cudaSuccess) e = r;
        return e == cudaSuccess;
    };
    if (!samples_dev) ok(buf.alloc(&d_samples, n));
    ok(buf.alloc(&d_cb, size_t(K)));
    ok(buf.alloc(&d_assign, n));
    ok(buf.alloc(&d_hist, size_t(K) * n_chunks));
    ok(buf.alloc(&d_start, size_t(K) + 1));
    ok(buf.alloc(&d_order, n));
    ok(buf.alloc(&d_err, size_t(assign_blocks)));
    if (e != cudaSuccess) {
        set_cuda_error("qamw_train_codebook_gpu: cudaMalloc", int(e));
        return QAMW_ERR_CUDA;
    }
    const double2* samples = samples_dev ? reinterpret_cast<const double2*>(samples_dev) : d_samples;
    if (!samples_dev) {
        // stream key as in the header of qamw_train_codebook: mix64(seed ^ 0xD1B54A32D192ED03)
        unsigned long long key = seed ^ 0xD1B54A32D192ED03ULL;
        key ^= key >> 30;
        key *= 0xBF58476D1CE4E5B9ULL;
        key ^= key >> 27;
        key *= 0x94D049BB133111EBULL;
        key ^= key >> 31;
        sample_kernel<<<8 * sm_count(), 256>>>(key, n, d_samples);
    }
    // initial codewords: sqrt(2) * sample_i
    std::vector<double> cb(size_t(2) * K), first(size_t(2) * K);
    ok(cudaMemcpy(first.data(), samples, sizeof(double) * 2 * K, cudaMemcpyDeviceToHost));
    const double root2 = 1.4142135623730950488016887242097;
    for (int c = 0; c < 2 * K; ++c) cb[size_t(c)] = root2 * first[size_t(c)];
    ok(cudaMemcpy(d_cb, cb.data(), sizeof(double) * 2 * K, cudaMemcpyHostToDevice));
    std::vector<double> err(size_t(assign_blocks), 0.0);
    if (sizeof(double2) * size_t(K) > 48 * 1024)  // K = 4096: the codebook needs more than the default dynamic limit
        ok(cudaFuncSetAttribute(assign_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(double2) * size_t(K))));
    auto assign_pass = [&](bool keep) -> double {
        assign_kernel<<<assign_blocks, kAssignThreads, sizeof(double2) * K>>>(samples, n, d_cb, K, keep ? d_assign : nullptr,
                                                                             d_err);
        ok(cudaMemcpy(err.data(), d_err, sizeof(double) * assign_blocks, cudaMemcpyDeviceToHost));
        double total = 0.0;
        for (double v : err) total += v;
        return total / double(n);
    };
    double prev = INFINITY;
    int updates = 0, t = 0;
    while (e == cudaSuccess) {
        const double D = assign_pass(true);
        if (mse_trace_out) mse_trace_out[t] = D;
        ++t;
        if (t > 1 && prev - D <= rel_tol * prev) break;
        if (updates >= max_iters) break;
        hist_kernel<<<n_chunks, 256, sizeof(int) * K>>>(d_assign, n, K, n_chunks, d_hist);
        scan_kernel<<<1, 1024>>>(d_hist, K * n_chunks, K, n_chunks, d_start);
        scatter_kernel<<<n_chunks, 32, sizeof(int) * K>>>(d_assign, n, K, n_chunks, d_hist, d_order);
        centroid_kernel<<<(K + 63) / 64, 64>>>(samples, d_order, d_start, K, d_cb);
        ok(cudaGetLastError());
        ++updates;
        prev = D;
    }
    ok(cudaMemcpy(cb.data(), d_cb, sizeof(double) * 2 * K, cudaMemcpyDeviceToHost));
    if (e != cudaSuccess) {
        set_cuda_error("qamw_train_codebook_gpu", int(e));
        return QAMW_ERR_CUDA;
    }
    // order by (squared radius, angle) so that indices are reproducible, round to f32
    std::vector<int> order(size_t(K), 0);
    for (int k = 0; k < K; ++k) order[size_t(k)] = k;
    auto r2 = [&](int k) { return cb[2 * size_t(k)] * cb[2 * size_t(k)] + cb[2 * size_t(k) + 1] * cb[2 * size_t(k) + 1]; };
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        const double ra = r2(a), rb = r2(b);
        if (ra != rb) return ra < rb;
        return std::atan2(cb[2 * size_t(a) + 1], cb[2 * size_t(a)]) < std::atan2(cb[2 * size_t(b) + 1], cb[2 * size_t(b)]);
    });
    for (int k = 0; k < K; ++k) {
        codebook_out[2 * k] = float(cb[2 * size_t(order[size_t(k)])]);
        codebook_out[2 * k + 1] = float(cb[2 * size_t(order[size_t(k)]) + 1]);
    }
    if (train_mse_out) {
        for (int c = 0; c < 2 * K; ++c) cb[size_t(c)] = double(codebook_out[c]);
        ok(cudaMemcpy(d_cb, cb.data(), sizeof(double) * 2 * K, cudaMemcpyHostToDevice));
        *train_mse_out = assign_pass(false);
    }
    if (iters_out) *iters_out = updates;
    if (e != cudaSuccess) {
        set_cuda_error("qamw_train_codebook_gpu", int(e));
        return QAMW_ERR_CUDA;
    }
    if (seconds_out) *seconds_out = std::chrono::duration<double>(std::chrono::steady_clock::now() - t_begin).count();
    return QAMW_OK;
}
