// Per-lane arithmetic of the streaming pass.  A "lane tile" is the four 16-byte vectors a lane
// owns in one 2 KB chunk (32 bf16 or 16 fp32 logits), loaded straight from global memory into
// registers: all four loads are issued before any math so their latency overlaps, the running
// maximum is taken once per lane tile (on packed bf16x2 for bf16 input), and the exponent
// arithmetic uses the packed f32x2 instructions of sm_100 so that one FMA-pipe instruction
// serves two logits.
#pragma once

#include "tslt_common.cuh"

namespace tslt {

__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Where a row's data ends: whole 16-byte vectors, then `rem` elements of one ragged vector.
struct RowExtent {
    int nvec_full;  // number of whole vectors
    int rem;        // elements of the ragged last vector (0 if none)
};
template <typename T> __host__ __device__ inline RowExtent row_extent(int V) {
    constexpr int per = 16 / Elt<T>::kBytes;
    RowExtent e;
    e.nvec_full = V / per;
    e.rem = V % per;
    return e;
}

// One lane of the warp asks for chunk `ch` of the row (clipped to the row's whole vectors) to be
// brought into L2, so that the warp's loads of it, one step later, are L2 hits.
__device__ __forceinline__ void prefetch_chunk(const unsigned char* row, int ch, int chunk_end, int lane,
                                               const RowExtent& ext) {
    if (lane == 0 && ch < chunk_end) {
        const int v0 = ch * kVecsPerChunk;
        int nv = ext.nvec_full - v0;
        if (nv > kVecsPerChunk) nv = kVecsPerChunk;
        if (nv > 0) prefetch_l2(row + (size_t)v0 * kVecBytes, (uint32_t)nv * kVecBytes);
    }
}

// Online softmax state of one lane: sum of 2^(z * c - M) in four packed accumulators.  The
// reference M is raised only when a logit's exponent would exceed it by more than kRaiseSlack:
// terms up to 2^32 are as exact in fp32 as terms below 1, and a reference that follows every new
// maximum would be rescaled by some lane of the warp on most steps.
constexpr float kRaiseSlack = 32.0f;
struct LaneSum {
    float2 acc[4];
    float M;     // reference exponent (base 2), -3e38 while the lane has seen nothing finite
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = make_float2(0.f, 0.f);
        M = -3.0e38f;
    }
    // Before a lane tile whose largest logit is lm is added: move the reference to lm's exponent if
    // that exceeds it by more than the slack.  Called by all lanes of a warp; the rescaling is
    // skipped by the whole warp unless some lane needs it (a handful of times per row), which a
    // per-lane branch would not achieve: the compiler turns it into selects executed on every step.
    __device__ __forceinline__ void raise_to(float lm, float c) {
        const float Mn = lm * c;
        const bool up = Mn - M > kRaiseSlack;
        if (!__any_sync(0xffffffffu, up)) return;
        const float sc = up ? ex2_approx(M - Mn) : 1.0f;
        const float2 sc2 = make_float2(sc, sc);
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = __fmul2_rn(acc[i], sc2);
        M = up ? Mn : M;
    }
    __device__ __forceinline__ float total() const {
        return ((acc[0].x + acc[0].y) + (acc[1].x + acc[1].y)) + ((acc[2].x + acc[2].y) + (acc[3].x + acc[3].y));
    }
    __device__ __forceinline__ double total_f64() const {
        double s = 0.0;
#pragma unroll
        for (int i = 0; i < 4; ++i) s += (double)acc[i].x + (double)acc[i].y;
        return s;
    }
};

template <typename T> struct LaneTile;

template <> struct LaneTile<bf16_t> {
    static constexpr int kElems = 32;
    uint32_t w[16];  // vector j holds words 4j..4j+3, each two bf16 (low half = lower index)
    uint32_t vm[4];  // packed maximum of vector j (set by reduce_max)
    uint32_t m2;     // packed maximum of the lane tile (set by reduce_max)

    // A whole chunk from lane_row = row + 16 * lane, so that the common case needs no lane number.
    __device__ __forceinline__ void load_lane(const unsigned char* lane_row, int vec0, const RowExtent& ext) {
        if (vec0 + kVecsPerChunk <= ext.nvec_full) {
            const uint4* base = reinterpret_cast<const uint4*>(lane_row) + vec0;
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                const uint4 v = ldg_stream(base + j * 32);
                w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
            }
        } else {
            const int lane = threadIdx.x & 31;
            load(lane_row - lane * kVecBytes, vec0, lane, ext);
        }
    }
    // Chunk whose first vector is number vec0 of the row at `row`; vectors past the row's end read
    // as -inf, the ragged last vector is fetched element by element.
    __device__ __forceinline__ void load(const unsigned char* row, int vec0, int lane, const RowExtent& ext) {
        const uint4* base = reinterpret_cast<const uint4*>(row) + vec0 + lane;
        if (vec0 + kVecsPerChunk <= ext.nvec_full) {
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                const uint4 v = ldg_stream(base + j * 32);
                w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                const int vi = vec0 + j * 32 + lane;
                uint4 v = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);  // -inf
                if (vi < ext.nvec_full) {
                    v = ldg_stream(base + j * 32);
                } else if (vi == ext.nvec_full && ext.rem) {
                    const unsigned short* e = reinterpret_cast<const unsigned short*>(base + j * 32);
                    uint32_t h[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) h[i] = i < ext.rem ? (uint32_t)__ldg(e + i) : 0xff80u;
                    v = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
                }
                w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
            }
        }
    }
    static __device__ __forceinline__ float lo(uint32_t x) { return __uint_as_float(x << 16); }
    static __device__ __forceinline__ float hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }
    // Fills vm[] and m2 and returns the largest logit of the lane tile.
    __device__ __forceinline__ float reduce_max() {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            vm[j] = bf16x2_max(bf16x2_max(w[4 * j], w[4 * j + 1]), bf16x2_max(w[4 * j + 2], w[4 * j + 3]));
        m2 = bf16x2_max(bf16x2_max(vm[0], vm[1]), bf16x2_max(vm[2], vm[3]));
        return fmaxf(lo(m2), hi(m2));
    }
    __device__ __forceinline__ float vec_max(int j) const { return fmaxf(lo(vm[j]), hi(vm[j])); }
    // s += sum 2^(z * c - M) over the 32 logits
    __device__ __forceinline__ void accumulate(LaneSum& s, float c) const {
        const float2 c2 = make_float2(c, c), negM2 = make_float2(-s.M, -s.M);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float2 t = __ffma2_rn(make_float2(lo(w[i]), hi(w[i])), c2, negM2);
            s.acc[i & 3] = __fadd2_rn(s.acc[i & 3], make_float2(ex2_approx(t.x), ex2_approx(t.y)));
        }
    }
    // logit e (0..7) of vector j
    __device__ __forceinline__ float elem(int j, int e) const {
        const uint32_t x = w[4 * j + (e >> 1)];
        return (e & 1) ? hi(x) : lo(x);
    }
};

template <> struct LaneTile<float> {
    static constexpr int kElems = 16;
    float z[16];
    float vm[4];  // maximum of vector j (set by reduce_max)

    __device__ __forceinline__ void load_lane(const unsigned char* lane_row, int vec0, const RowExtent& ext) {
        if (vec0 + kVecsPerChunk <= ext.nvec_full) {
            const uint4* base = reinterpret_cast<const uint4*>(lane_row) + vec0;
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                const uint4 v = ldg_stream(base + j * 32);
                z[4 * j] = __uint_as_float(v.x); z[4 * j + 1] = __uint_as_float(v.y);
                z[4 * j + 2] = __uint_as_float(v.z); z[4 * j + 3] = __uint_as_float(v.w);
            }
        } else {
            const int lane = threadIdx.x & 31;
            load(lane_row - lane * kVecBytes, vec0, lane, ext);
        }
    }
    __device__ __forceinline__ void load(const unsigned char* row, int vec0, int lane, const RowExtent& ext) {
        const uint4* base = reinterpret_cast<const uint4*>(row) + vec0 + lane;
        if (vec0 + kVecsPerChunk <= ext.nvec_full) {
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                const uint4 v = ldg_stream(base + j * 32);
                z[4 * j] = __uint_as_float(v.x); z[4 * j + 1] = __uint_as_float(v.y);
                z[4 * j + 2] = __uint_as_float(v.z); z[4 * j + 3] = __uint_as_float(v.w);
            }
        } else {
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                const int vi = vec0 + j * 32 + lane;
                uint4 v = make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);  // -inf
                if (vi < ext.nvec_full) {
                    v = ldg_stream(base + j * 32);
                } else if (vi == ext.nvec_full && ext.rem) {
                    const uint32_t* e = reinterpret_cast<const uint32_t*>(base + j * 32);
                    uint32_t h[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) h[i] = i < ext.rem ? __ldg(e + i) : 0xff800000u;
                    v = make_uint4(h[0], h[1], h[2], h[3]);
                }
                z[4 * j] = __uint_as_float(v.x); z[4 * j + 1] = __uint_as_float(v.y);
                z[4 * j + 2] = __uint_as_float(v.z); z[4 * j + 3] = __uint_as_float(v.w);
            }
        }
    }
    __device__ __forceinline__ float reduce_max() {
#pragma unroll
        for (int j = 0; j < 4; ++j) vm[j] = fmaxf(fmaxf(z[4 * j], z[4 * j + 1]), fmaxf(z[4 * j + 2], z[4 * j + 3]));
        return fmaxf(fmaxf(vm[0], vm[1]), fmaxf(vm[2], vm[3]));
    }
    __device__ __forceinline__ float vec_max(int j) const { return vm[j]; }
    __device__ __forceinline__ void accumulate(LaneSum& s, float c) const {
        const float2 c2 = make_float2(c, c), negM2 = make_float2(-s.M, -s.M);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float2 t = __ffma2_rn(make_float2(z[2 * i], z[2 * i + 1]), c2, negM2);
            s.acc[i & 3] = __fadd2_rn(s.acc[i & 3], make_float2(ex2_approx(t.x), ex2_approx(t.y)));
        }
    }
    __device__ __forceinline__ float elem(int j, int e) const { return z[4 * j + e]; }
};

}  // namespace tslt
