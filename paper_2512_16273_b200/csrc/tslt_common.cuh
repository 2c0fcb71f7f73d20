// Shared device helpers of libtslt: layout constants, mbarrier / bulk-copy (TMA) wrappers
// with bounded waits, block-level scans and reductions, and the order-preserving key map.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tslt.h"

namespace tslt {

// ---- CTA shape ---------------------------------------------------------------------------
// 8 consumer warps do the arithmetic; one extra producer warp drives the bulk-copy ring.
constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kBlockThreads = kConsumerThreads + 32;
// A tile is what one bulk copy brings in; each consumer warp owns one contiguous chunk of it.
constexpr int kTileBytes = 16384;
constexpr int kChunkBytes = kTileBytes / kConsumerWarps;  // 2048 B: the unit of per-chunk partial sums
constexpr int kVecBytes = 16;
constexpr int kVecsPerLane = kChunkBytes / (32 * kVecBytes);  // 4
constexpr int kStages = 3;
constexpr int kRingBytes = kStages * kTileBytes;

// Named barrier for the consumer warps (barrier 0 is left to __syncthreads before the roles split).
constexpr int kConsumerBarrier = 1;

// Workspace header: word 0 is the device status (0 = fine).
constexpr int kWsHeaderBytes = 256;
constexpr int kStatusWaitTimeout = 1;

// Spin limits for device-side waits (each probe suspends for a while in hardware first).
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ void consumer_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(kConsumerBarrier), "n"(kConsumerThreads) : "memory");
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier ----------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false when the limit ran out or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    return false;
}

// ---- bulk asynchronous copy (TMA, untiled): global -> this CTA's shared memory ------------
// dst, src 16-byte aligned, bytes a non-zero multiple of 16; completion is signalled on `bar`.
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// ---- small math --------------------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Order-preserving map float -> uint32 (ascending), with -0 folded onto +0 so that equal
// floats get equal keys.  Non-finite values are never turned into keys by the callers.
__device__ __forceinline__ uint32_t float_to_key(float f) {
    uint32_t b = __float_as_uint(f + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k) {
    uint32_t b = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(b);
}

__device__ __forceinline__ float clamp_uniform(float u) {
    if (!(u >= 0.0f)) return 0.0f;
    if (u >= 1.0f) return 0.99999994f;  // largest float below 1
    return u;
}

// ---- block-level helpers for the 256 consumer threads ------------------------------------
// All take `tid` in [0, 256) and a scratch array of >= 8 elements in shared memory, and end
// with a consumer_sync() so the scratch can be reused right away.
__device__ __forceinline__ double block_sum(double v, int tid, double* scratch) {
    v = warp_sum(v);
    if ((tid & 31) == 0) scratch[tid >> 5] = v;
    consumer_sync();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) t += scratch[w];
    consumer_sync();
    return t;
}
__device__ __forceinline__ double block_max(double v, int tid, double* scratch) {
    v = warp_max(v);
    if ((tid & 31) == 0) scratch[tid >> 5] = v;
    consumer_sync();
    double t = scratch[0];
#pragma unroll
    for (int w = 1; w < kConsumerWarps; ++w) t = fmax(t, scratch[w]);
    consumer_sync();
    return t;
}
__device__ __forceinline__ int block_sum_int(int v, int tid, int* scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((tid & 31) == 0) scratch[tid >> 5] = v;
    consumer_sync();
    int t = 0;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) t += scratch[w];
    consumer_sync();
    return t;
}

// In-place inclusive scan of a[0..n) (shared memory, fp64) by the 256 consumer threads.
// Each thread owns a contiguous run, so the result is the same left-to-right sum order
// inside a run and a fixed tree across runs: deterministic.
__device__ __forceinline__ void block_inclusive_scan(double* a, int n, int tid, double* scratch /* >= 9 */) {
    const int per = (n + kConsumerThreads - 1) / kConsumerThreads;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    double run = 0.0;
    for (int i = lo; i < hi; ++i) run += a[i];
    // exclusive scan of the per-thread totals
    double incl = run;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) scratch[warp] = incl;
    consumer_sync();
    double base = 0.0;
    for (int w = 0; w < warp; ++w) base += scratch[w];
    double acc = base + (incl - run);
    for (int i = lo; i < hi; ++i) {
        acc += a[i];
        a[i] = acc;
    }
    consumer_sync();
}

// First index i in [0, n) with cum[i] > target, for a non-decreasing array; n if none.
__device__ __forceinline__ int first_greater(const double* cum, int n, double target) {
    int lo = 0, hi = n;
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (cum[mid] > target) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// ---- element access ----------------------------------------------------------------------
template <typename T> struct Elt;
template <> struct Elt<float> {
    static constexpr int kBytes = 4;
    static constexpr int kPerVec = 4;
    static __device__ __forceinline__ float load(const void* row, long long i) {
        return __ldg(reinterpret_cast<const float*>(row) + i);
    }
};
struct bf16_t { uint16_t bits; };
template <> struct Elt<bf16_t> {
    static constexpr int kBytes = 2;
    static constexpr int kPerVec = 8;
    static __device__ __forceinline__ float load(const void* row, long long i) {
        uint32_t b = __ldg(reinterpret_cast<const unsigned short*>(row) + i);
        return __uint_as_float(b << 16);
    }
};

__device__ __forceinline__ uint4 lds_vec(const unsigned char* p) {
    return *reinterpret_cast<const uint4*>(p);
}

// Unpack one 16-byte vector into fp32 values.
template <typename T> __device__ __forceinline__ void unpack_vec(const uint4& v, float* z);
template <> __device__ __forceinline__ void unpack_vec<float>(const uint4& v, float* z) {
    z[0] = __uint_as_float(v.x); z[1] = __uint_as_float(v.y);
    z[2] = __uint_as_float(v.z); z[3] = __uint_as_float(v.w);
}
template <> __device__ __forceinline__ void unpack_vec<bf16_t>(const uint4& v, float* z) {
    z[0] = __uint_as_float(v.x << 16); z[1] = __uint_as_float(v.x & 0xffff0000u);
    z[2] = __uint_as_float(v.y << 16); z[3] = __uint_as_float(v.y & 0xffff0000u);
    z[4] = __uint_as_float(v.z << 16); z[5] = __uint_as_float(v.z & 0xffff0000u);
    z[6] = __uint_as_float(v.w << 16); z[7] = __uint_as_float(v.w & 0xffff0000u);
}

// The scale that turns a stored logit into the base-2 exponent z * log2(e) / T, split in
// two floats so that the product is accurate to ~1e-15 relative: hi <= c, lo > 0.
struct ScaleC {
    float hi, lo;
    double d;  // hi + lo as a double: the value all fp64 code uses
};

}  // namespace tslt
