// Per-lane arithmetic of the streaming pass.  A "lane tile" is the four 16-byte vectors a lane
// owns in one ring tile (32 bf16 or 16 fp32 logits).  All four are loaded before any math so
// the shared-memory latency overlaps, the running maximum is taken once per lane tile (on
// packed bf16x2 for bf16 input), and the exponent arithmetic uses the packed f32x2
// instructions of sm_100 so that one FMA-pipe instruction serves two logits.
#pragma once

#include "tslt_common.cuh"

namespace tslt {

// ---- packed f32x2 helpers (sm_100) ---------------------------------------------------------
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Online softmax state of one lane: sum of 2^(y - M) in four packed accumulators.
struct LaneSum {
    uint64_t acc[4];
    float M;     // reference exponent (base 2), -3e38 while the lane has seen nothing finite
    float zmax;  // largest logit seen
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = 0ull;
        M = -3.0e38f;
        zmax = -INFINITY;
    }
    // raise the reference to the exponent of a new maximum
    __device__ __forceinline__ void raise(float new_max, float chi, float clo) {
        zmax = new_max;
        const float Mn = fmaf(new_max, chi, new_max * clo);
        const float sc = ex2_approx(M - Mn);
        const uint64_t sc2 = pack2(sc, sc);
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = mul2(acc[i], sc2);
        M = Mn;
    }
    __device__ __forceinline__ float total() const {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float a, b;
            unpack2(acc[i], a, b);
            s += a + b;
        }
        return s;
    }
    __device__ __forceinline__ double total_f64() const {
        double s = 0.0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float a, b;
            unpack2(acc[i], a, b);
            s += (double)a + (double)b;
        }
        return s;
    }
};

template <typename T> struct LaneTile;

template <> struct LaneTile<bf16_t> {
    static constexpr int kElems = 32;
    uint32_t w[16];  // vector j holds words 4j..4j+3, each two bf16 (low half = lower index)

    __device__ __forceinline__ void load(const unsigned char* tile, int warp, int lane, uint32_t padded) {
#pragma unroll
        for (int j = 0; j < kVecsPerLane; ++j) {
            const uint32_t off = warp * kChunkBytes + (j * 32 + lane) * kVecBytes;
            uint4 v = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);  // -inf
            if (off < padded) v = lds_vec(tile + off);
            w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
        }
    }
    static __device__ __forceinline__ float lo(uint32_t x) { return __uint_as_float(x << 16); }
    static __device__ __forceinline__ float hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }
    // packed maximum of vector j (two bf16 lanes of one word)
    __device__ __forceinline__ uint32_t vec_max2(int j) const {
        return bf16x2_max(bf16x2_max(w[4 * j], w[4 * j + 1]), bf16x2_max(w[4 * j + 2], w[4 * j + 3]));
    }
    __device__ __forceinline__ float lane_max() const {
        const uint32_t m = bf16x2_max(bf16x2_max(vec_max2(0), vec_max2(1)), bf16x2_max(vec_max2(2), vec_max2(3)));
        return fmaxf(lo(m), hi(m));
    }
    __device__ __forceinline__ float vec_max(int j) const {
        const uint32_t m = vec_max2(j);
        return fmaxf(lo(m), hi(m));
    }
    // s += sum 2^(z * c - M) over the 32 logits
    __device__ __forceinline__ void accumulate(LaneSum& s, float chi, float clo) const {
        const uint64_t chi2 = pack2(chi, chi), clo2 = pack2(clo, clo), negM2 = pack2(-s.M, -s.M);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint64_t z2 = pack2(lo(w[i]), hi(w[i]));
            const uint64_t t2 = fma2(z2, chi2, fma2(z2, clo2, negM2));
            float a, b;
            unpack2(t2, a, b);
            s.acc[i & 3] = add2(s.acc[i & 3], pack2(ex2_approx(a), ex2_approx(b)));
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

    __device__ __forceinline__ void load(const unsigned char* tile, int warp, int lane, uint32_t padded) {
#pragma unroll
        for (int j = 0; j < kVecsPerLane; ++j) {
            const uint32_t off = warp * kChunkBytes + (j * 32 + lane) * kVecBytes;
            uint4 v = make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
            if (off < padded) v = lds_vec(tile + off);
            z[4 * j] = __uint_as_float(v.x); z[4 * j + 1] = __uint_as_float(v.y);
            z[4 * j + 2] = __uint_as_float(v.z); z[4 * j + 3] = __uint_as_float(v.w);
        }
    }
    __device__ __forceinline__ float vec_max(int j) const {
        return fmaxf(fmaxf(z[4 * j], z[4 * j + 1]), fmaxf(z[4 * j + 2], z[4 * j + 3]));
    }
    __device__ __forceinline__ float lane_max() const {
        return fmaxf(fmaxf(vec_max(0), vec_max(1)), fmaxf(vec_max(2), vec_max(3)));
    }
    __device__ __forceinline__ void accumulate(LaneSum& s, float chi, float clo) const {
        const uint64_t chi2 = pack2(chi, chi), clo2 = pack2(clo, clo), negM2 = pack2(-s.M, -s.M);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint64_t z2 = pack2(z[2 * i], z[2 * i + 1]);
            const uint64_t t2 = fma2(z2, chi2, fma2(z2, clo2, negM2));
            float a, b;
            unpack2(t2, a, b);
            s.acc[i & 3] = add2(s.acc[i & 3], pack2(ex2_approx(a), ex2_approx(b)));
        }
    }
    __device__ __forceinline__ float elem(int j, int e) const { return z[4 * j + e]; }
};

// Logit number e of a ring tile held in shared memory.
template <typename T> __device__ __forceinline__ float tile_elem(const unsigned char* tile, int e);
template <> __device__ __forceinline__ float tile_elem<float>(const unsigned char* tile, int e) {
    return reinterpret_cast<const float*>(tile)[e];
}
template <> __device__ __forceinline__ float tile_elem<bf16_t>(const unsigned char* tile, int e) {
    return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(tile)[e] << 16);
}

}  // namespace tslt
