// Shared device helpers of libtslt: layout constants, block-level scans and reductions, the
// order-preserving key map and the element accessors.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tslt.h"

namespace tslt {

// ---- CTA shape ---------------------------------------------------------------------------
// 8 warps per CTA.  A chunk is the 2 KB a warp reads in one step (four 16-byte vectors per lane,
// vector j of lane l at byte offset (j * 32 + l) * 16, so that every load instruction of the warp
// covers 512 contiguous bytes); it is also the unit of the verifier's per-chunk partial sums.
constexpr int kWarps = 8;
constexpr int kBlockThreads = kWarps * 32;
constexpr int kConsumerWarps = kWarps;
constexpr int kConsumerThreads = kBlockThreads;
constexpr int kChunkBytes = 2048;
constexpr int kVecBytes = 16;
constexpr int kVecsPerLane = kChunkBytes / (32 * kVecBytes);  // 4
constexpr int kVecsPerChunk = kChunkBytes / kVecBytes;        // 128

// Named barrier used by the block-level helpers (all 256 threads take part).
constexpr int kConsumerBarrier = 1;

// How the rows of a call map to CTAs: every row is cut into nseg segments of cps chunks (the last
// may be shorter), one CTA per segment, block = row * nseg + seg.
struct RowSplit {
    int rows, nseg, cps, grid;
};
struct RowWork {
    int row, seg, nseg, chunk_begin, chunk_end;
};
__host__ __device__ inline RowWork locate_work(const RowSplit& sp, int block, int nchunks) {
    RowWork w;
    w.row = block / sp.nseg;
    w.seg = block - w.row * sp.nseg;
    w.nseg = sp.nseg;
    w.chunk_begin = w.seg * sp.cps;
    w.chunk_end = w.chunk_begin + sp.cps < nchunks ? w.chunk_begin + sp.cps : nchunks;
    return w;
}
// slots = CTAs the machine holds at once; max_seg = most segments a row may be cut into;
// big_cps = segment length (chunks) to use when there are at least `slots` rows (0: whole rows).
// With fewer rows than slots, rows are cut so that about two CTAs per slot exist, a segment
// keeping at least two chunks per warp.
inline RowSplit make_row_split(long long rows, int nchunks, int slots, int max_seg, int big_cps) {
    RowSplit sp;
    sp.rows = (int)rows;
    if (nchunks < 1) nchunks = 1;
    int by_len = nchunks / 16;
    if (by_len < 1) by_len = 1;
    if (max_seg > by_len) max_seg = by_len;
    if (max_seg < 1) max_seg = 1;
    int nseg = 1;
    if (rows >= slots) {
        if (big_cps > 0) nseg = (nchunks + big_cps - 1) / big_cps;
    } else if (rows > 0) {
        nseg = (int)((2LL * slots + rows - 1) / rows);
    }
    if (nseg > max_seg) nseg = max_seg;
    if (nseg < 1) nseg = 1;
    int cps = (nchunks + nseg - 1) / nseg;
    cps = (cps + 7) / 8 * 8;
    sp.nseg = (nchunks + cps - 1) / cps;
    sp.cps = cps;
    sp.grid = sp.rows * sp.nseg;
    return sp;
}

// Workspace header: word 0 is the device status (0 = fine).
constexpr int kWsHeaderBytes = 256;
inline size_t align_up256(size_t x) { return (x + 255) / 256 * 256; }

__device__ __forceinline__ void consumer_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(kConsumerBarrier), "n"(kConsumerThreads) : "memory");
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- programmatic dependent launch ---------------------------------------------------------------
// An entry point is a streaming kernel followed by a finish / resolve kernel on the same stream.
// The second kernel is launched with programmatic stream serialization: its CTAs may be placed on
// SMs that the first kernel's last wave leaves free, and wait at their very first instruction
// until the first kernel has completed and its writes are visible.  The first kernel allows that
// as soon as it starts.  (Launched without the attribute, both instructions do nothing.)
__device__ __forceinline__ void allow_dependent_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void wait_for_primary_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Ready flags between the two kernels of tslt_sparsify (one per row segment).  The finish kernel is
// the streaming kernel's programmatic dependent, so by the time one of its CTAs runs, every CTA of
// the streaming kernel has started (dependents are scheduled once all CTAs of the primary have
// issued launch_dependents or exited): each streaming CTA still running is resident and finishes
// on its own, whatever the finish CTAs do.  A finish CTA can therefore begin as soon as its own
// row has been handed over instead of when the whole streaming kernel has ended.  The wait is
// bounded all the same: after `limit` polls (kReadyPollLimit by default, about a second) the CTA
// records that in the workspace's status word and falls back to griddepcontrol.wait, which returns
// when the streaming kernel has completed; the results are the same.  Without the launch
// attribute the finish kernel starts after the streaming kernel and finds every flag set.  Each
// streaming CTA clears its own flag (and fences) before it issues launch_dependents, so a flag
// left set by an earlier call on the same workspace is gone before any finish CTA can look at it.
constexpr int kReadyPollLimit = 1 << 22;
__device__ __forceinline__ void publish_row_ready(int* flag) {  // one thread, after a barrier that follows the segment's writes
    __threadfence();
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(flag), "r"(1) : "memory");
}
__device__ __forceinline__ bool poll_row_ready(const int* flag, int limit) {  // one thread
    for (int it = 0; it < limit; ++it) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v != 0) return true;
        __nanosleep(200);
    }
    return false;
}

// A streaming kernel that uses no shared memory leaves its SMs configured with (next to) none, and
// the CTAs of the dependent kernel, which need some, then cannot be placed beside its last wave:
// they wait until an SM has drained completely (measured: the first finish CTA entered 36 us after
// the last streaming CTA had started, and the overlap was lost).  Both kernels of an entry point
// therefore ask for the same carve-out, once per device and kernel: 58 % of the SM's 228 KB for
// shared memory (132 KB).  The streaming kernels need the rest as L1 for their loads in flight:
// with the largest carve-out they ran a third slower, with 14 % the finish CTAs did not fit
// (2048 rows of 256 000 bf16 logits, k = 64 / 1024: 242 / 574 us at 14 %, 217 / 548 at 28 %,
// 215 / 396 at 44 %, 217 / 376 at 58 %, 221 / 411 at 72 %, 295 / 589 at 100 %).
// slot: a small number unique to the kernel instantiation.
constexpr int kPreferredCarveoutPercent = 58;
template <typename K> inline bool prefer_shared_carveout_once(K kern, int slot) {
    constexpr int kMaxDevices = 64, kSlots = 16;
    static bool done[kSlots][kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const bool cached = dev >= 0 && dev < kMaxDevices && slot >= 0 && slot < kSlots;
    if (cached && done[slot][dev]) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, kPreferredCarveoutPercent) != cudaSuccess)
        return false;
    if (cached) done[slot][dev] = true;
    return true;
}

template <typename Params>
inline cudaError_t launch_dependent(void (*kernel)(const Params), unsigned grid, unsigned block, size_t smem,
                                    cudaStream_t st, const Params& p) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// ---- optional time stamps (build with -DTSLT_STAMPS; see paper_2512_16273_b200/timeline.py) -----------------
// Thread 0 of a CTA writes %globaltimer into stamps[cta * kStampSlots + slot]: where the microseconds of a
// call go, phase by phase.  The array is per translation unit; each .cu file that stamps exports a reader.
// In the ordinary build the macro is empty and nothing of this exists.
#ifdef TSLT_STAMPS
constexpr int kStampCtas = 16384, kStampSlots = 8;
static __device__ unsigned long long g_stamps[kStampCtas * kStampSlots];
__device__ __forceinline__ void stamp_now(int cta, int slot) {
    if (threadIdx.x == 0 && cta < kStampCtas) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        g_stamps[cta * kStampSlots + slot] = t;
    }
}
#define TSLT_STAMP(cta, slot) stamp_now((cta), (slot))
#else
#define TSLT_STAMP(cta, slot) do { } while (0)
#endif

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

// ---- block-level helpers for the 256 threads of a CTA ------------------------------------
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

// Ask the copy engine to bring `bytes` (a non-zero multiple of 16) at the 16-byte aligned global
// address p into L2; nothing is written anywhere else and nothing has to be waited for.
__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// 16-byte streaming load of logits: read once, so marked evict-first.
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) { return __ldcs(p); }

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

// The reverse, for values that came from the storage type (exact).
template <typename T> __device__ __forceinline__ uint4 pack_vec(const float* z);
template <> __device__ __forceinline__ uint4 pack_vec<float>(const float* z) {
    return make_uint4(__float_as_uint(z[0]), __float_as_uint(z[1]), __float_as_uint(z[2]), __float_as_uint(z[3]));
}
template <> __device__ __forceinline__ uint4 pack_vec<bf16_t>(const float* z) {
    return make_uint4((__float_as_uint(z[0]) >> 16) | (__float_as_uint(z[1]) & 0xffff0000u),
                      (__float_as_uint(z[2]) >> 16) | (__float_as_uint(z[3]) & 0xffff0000u),
                      (__float_as_uint(z[4]) >> 16) | (__float_as_uint(z[5]) & 0xffff0000u),
                      (__float_as_uint(z[6]) >> 16) | (__float_as_uint(z[7]) & 0xffff0000u));
}

// The scale c = log2(e) / T that turns a stored logit into a base-2 exponent.  The streaming
// pass uses its fp32 rounding `f` in one fused multiply-add per logit, y = z * f - M, where M is
// the fp32 exponent of a running maximum; `d` is the value all fp64 code uses.  |f/d - 1| <=
// 2^-25 moves a row's log-normaliser by less than 1e-7 relative.
struct ScaleC {
    float f;
    double d;
};

}  // namespace tslt
