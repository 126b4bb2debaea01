// Device-side building blocks shared by the translation units of libqamw: packed f32x2 arithmetic,
// shared-memory loads, the bank-separated codebook copies and the nearest-codeword search.
// Everything here has internal linkage (anonymous namespace) and is compiled into each .cu file.
#ifndef QAMW_DEVICE_CUH_
#define QAMW_DEVICE_CUH_

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr size_t kSmemLimit = 227 * 1024;

// ---------------------------------------------------------------------------------------------
// packed f32x2 arithmetic: two IEEE f32 operations (round to nearest even, each half rounded on
// its own) in one instruction; it halves the issue slots of the butterflies.
// ---------------------------------------------------------------------------------------------
typedef unsigned long long f32x2;

__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// (a, c) -> (a + c, a - c) on two packed registers.
__device__ __forceinline__ void bfly2(f32x2& a, f32x2& c) {
    const f32x2 s = add2(a, c), d = sub2(a, c);
    a = s;
    c = d;
}
__device__ __forceinline__ f32x2 shfl_xor2(f32x2 v, int lane_mask) {
    float lo, hi;
    unpack2(v, lo, hi);
    lo = __shfl_xor_sync(kFull, lo, lane_mask);
    hi = __shfl_xor_sync(kFull, hi, lane_mask);
    return pack2(lo, hi);
}

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

// Eight consecutive per-column constants starting at column e0 (a multiple of 8): 16-byte loads
// when the arrays allow it (checked on the host: `cvec`), element-wise otherwise.  Columns beyond
// n read as `fill`.
__device__ __forceinline__ void load8f(const float* p, int e0, int n, int cvec, float fill, float (&v)[8]) {
    if (cvec && e0 + 8 <= n) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p + e0));
        const float4 c = __ldg(reinterpret_cast<const float4*>(p + e0) + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = (e0 + e < n) ? __ldg(p + e0 + e) : fill;
    }
}
__device__ __forceinline__ void load4f(const float* p, int k0, int n, int cvec, float fill, float (&v)[4]) {
    if (cvec && k0 + 4 <= n) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p + k0));
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = (k0 + e < n) ? __ldg(p + k0 + e) : fill;
    }
}
// signs (+1 / -1 bytes) of 8 consecutive columns as floats; 0 beyond n
__device__ __forceinline__ void load8s(const int8_t* p, int e0, int n, int cvec, float (&v)[8]) {
    if (cvec && e0 + 8 <= n) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(p + e0));
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint32_t w = e < 4 ? raw.x : raw.y;
            const uint32_t byte = (w >> (8 * (e & 3))) & 0xffu;
            v[e] = __uint_as_float(0x3f800000u | ((byte & 0x80u) << 24));  // +-1.0f from the byte's sign bit
        }
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = (e0 + e < n) ? float(__ldg(p + e0 + e)) : 0.f;
    }
}

// ---------------------------------------------------------------------------------------------
// codebook in shared memory: C = 2^log2c copies; entry i of copy c sits at byte (i*C + c) * 8, so
// the copies of one entry fill consecutive 8-byte bank pairs and a lane that always reads copy
// (lane mod C) only ever touches its own 16/C bank pairs.
// ---------------------------------------------------------------------------------------------
// `butterfly`: store (x + y, x - y) instead of (x, y) -- the decoder's first butterfly stage works
// on exactly these two numbers of every pair (scaled by the pair's sigma), so it can be done once
// per codeword here instead of once per decoded pair.
__device__ __forceinline__ void fill_codebook_copies(float2* dst, const float2* src, int K, int log2c,
                                                     bool butterfly = false) {
    // all loads of a thread first (up to 8 in flight), then the copies as 16-byte stores
    constexpr int kMaxPerThread = 8;
    float2 c[kMaxPerThread];
    const int T = blockDim.x;
    for (int base = 0; base < K; base += kMaxPerThread * T) {
#pragma unroll
        for (int u = 0; u < kMaxPerThread; ++u) {
            const int i = base + u * T + threadIdx.x;
            c[u] = i < K ? __ldg(src + i) : make_float2(0.f, 0.f);
            if (butterfly) c[u] = make_float2(c[u].x + c[u].y, c[u].x - c[u].y);
        }
#pragma unroll
        for (int u = 0; u < kMaxPerThread; ++u) {
            const int i = base + u * T + threadIdx.x;
            if (i >= K) continue;
            if (log2c == 0) {
                dst[i] = c[u];
            } else {
                // 2^m 16-byte pieces per entry; consecutive lanes own consecutive entries, so a lane
                // starts at the piece that puts the warp's stores on all banks at once
                float4* d4 = reinterpret_cast<float4*>(dst + (size_t(i) << log2c));
                const float4 v = make_float4(c[u].x, c[u].y, c[u].x, c[u].y);
                const int m = log2c - 1, first = (threadIdx.x & 31) >> (3 - m);
                for (int k = 0; k < (1 << m); ++k) d4[(first + k) & ((1 << m) - 1)] = v;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// nearest-codeword search
// ---------------------------------------------------------------------------------------------

// Shared-memory reads of the read-only tables, by 32-bit shared address.  Written as plain
// (non-volatile) asm: the tables never change after the prologue's barrier, so these loads may be
// scheduled freely around the stores to the staging buffers.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ float2 lds_f32x2(uint32_t addr) {
    float2 v;
    asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds_u32x2(uint32_t addr) {
    uint2 v;
    asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

struct SearchSmem {       // all fields are shared-memory byte addresses
    uint32_t cb;          // codebook copies, already offset to this lane's copy
    uint32_t cb_stride;   // byte distance between consecutive entries (8 << log2c)
    uint32_t cells;       // grid*grid records of 8 bytes; minus 8 * (grid + 1) * kMagicBits, see search_cell
    uint32_t overflow;    // u16 lists
    uint32_t grid;
    int K;
    f32x2 zlo;            // the cell map, each value twice: -zmax,
    f32x2 c0, c1, c2;     // the polynomial's coefficients,
    f32x2 bias;           // 1.5 * 2^23 + half
};

constexpr uint32_t kMagicBits = 0x4B400000u;  // bit pattern of 1.5 * 2^23 = 12582912.0f

__device__ __forceinline__ float2 codeword(const SearchSmem& s, int k) {
    return lds_f32x2(s.cb + uint32_t(k) * s.cb_stride);
}

// Squared distance in direct form, one rounding per operation: f32(f32(dx^2) + f32(dy^2)); the two
// subtractions and the two squares are one packed instruction each.
__device__ __forceinline__ float dist2(float2 c, float zx, float zy) {
    const f32x2 d = sub2(pack2(zx, zy), pack2(c.x, c.y));
    float sx, sy;
    unpack2(mul2(d, d), sx, sy);
    return __fadd_rn(sx, sy);
}

__device__ __forceinline__ void consider(const SearchSmem& s, int k, float zx, float zy, float& best, int& arg) {
    const float d = dist2(codeword(s, k), zx, zy);
    if (d < best) {
        best = d;
        arg = k;
    }
}

__device__ __noinline__ int search_exhaustive(const SearchSmem& s, float zx, float zy) {
    float best = INFINITY;
    int arg = 0;
    for (int k = 0; k < s.K; ++k) consider(s, k, zx, zy, best, arg);
    return arg;
}

__device__ __forceinline__ int search_overflow(const SearchSmem& s, uint2 rec, float zx, float zy) {
    const int off = int(rec.x >> 16), cnt = int(rec.y & 0xffffu);
    float best = INFINITY;
    int arg = 0;
#pragma unroll 1
    for (int i = 0; i < cnt; ++i) consider(s, int(lds_u16(s.overflow + 2u * uint32_t(off + i))), zx, zy, best, arg);
    return arg;
}

// A cell record whose first field is 0xFFFF points to an overflow list: {0xFFFF, offset, count, 0}.
__device__ __forceinline__ bool cell_overflows(uint2 rec) { return (rec.x & 0xffffu) == 0xffffu; }

// Nearest of the four candidates in the record of the point's cell, for a point inside the table's
// reach (|z| < 16000; a NaN coordinate is clamped like a large one and gets some index).  There is
// no branch in here, so that the searches of the four points of an octet interleave: the fields are
// masked to valid indices, and the caller tests the record it gets back with cell_overflows() and
// runs search_overflow() for such a cell (whose masked fields gave a meaningless result).
__device__ __forceinline__ int search_cell(const SearchSmem& s, float zx, float zy, uint2& rec_out) {
    // Column and row: c = clamp(z, +-zmax), half + rn(c (c0 + t (c1 + t c2))), t = c^2, both axes in
    // packed arithmetic.  The last fused multiply-add lands on 1.5 * 2^23 + half, where the spacing
    // of f32 is 1: its rounding is the rounding to an integer, and the integer sits in the low
    // mantissa bits, kMagicBits above zero.  That offset is folded into s.cells.
    float lo, hi;
    unpack2(s.zlo, lo, hi);
    const float cx = fminf(fmaxf(zx, lo), -lo), cy = fminf(fmaxf(zy, lo), -lo);
    const f32x2 c = pack2(cx, cy);
    const f32x2 t = mul2(c, c);
    const f32x2 v = fma2(c, fma2(t, fma2(t, s.c2, s.c1), s.c0), s.bias);
    float vx, vy;
    unpack2(v, vx, vy);
    const uint32_t bx = __float_as_uint(vx), by = __float_as_uint(vy);
    const uint2 rec = lds_u32x2(s.cells + ((by * s.grid + bx) << 3));
    rec_out = rec;
    const uint32_t km = uint32_t(s.K - 1);  // K is a power of two
    const int k0 = int(rec.x & km), k1 = int((rec.x >> 16) & km), k2 = int(rec.y & km), k3 = int((rec.y >> 16) & km);
    // The list is ascending and padded by repeating its last entry (a repeated slot cannot win).
    const float2 c0 = codeword(s, k0), c1 = codeword(s, k1), c2 = codeword(s, k2), c3 = codeword(s, k3);
    const float d0 = dist2(c0, zx, zy), d1 = dist2(c1, zx, zy), d2 = dist2(c2, zx, zy), d3 = dist2(c3, zx, zy);
    // lowest slot (= lowest index) among equal distances: a later slot wins only when strictly closer
    const bool s1 = d1 < d0, s3 = d3 < d2;
    const float da = s1 ? d1 : d0, db = s3 ? d3 : d2;
    const int ka = s1 ? k1 : k0, kb = s3 ? k3 : k2;
    return db < da ? kb : ka;
}

__device__ __noinline__ int search_table(const SearchSmem& s, float zx, float zy) {
    // beyond the table's reach (or NaN): exhaustive scan
    if (!(fmaxf(fabsf(zx), fabsf(zy)) < 16000.0f)) return search_exhaustive(s, zx, zy);
    uint2 rec;
    const int v = search_cell(s, zx, zy, rec);
    return cell_overflows(rec) ? search_overflow(s, rec, zx, zy) : v;
}

// Asynchronous global -> shared copies (no register staging, completion tracked per thread).
__device__ __forceinline__ void cp_async(void* smem_dst, const void* gmem_src, int log2_bytes) {
    const unsigned dst = unsigned(__cvta_generic_to_shared(smem_dst));
    if (log2_bytes == 4)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

}  // namespace

#endif  // QAMW_DEVICE_CUH_
