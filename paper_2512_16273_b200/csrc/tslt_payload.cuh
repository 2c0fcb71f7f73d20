// Bit layout of the uplink payload shared by the codec kernels and by the verifier that reads packed
// records directly (Section 2.2 fixes the widths: b_idx = ceil(log2 |V|), b_prob = 32 or 16; the
// record layout is this library's and is stated in include/tslt.h).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tslt.h"

namespace tslt {

__host__ __device__ inline int index_bits_of(int V) {
    int b = 0;
    while (b < 31 && (1ll << b) < (long long)V) ++b;
    return b;
}
__host__ __device__ inline int prob_bits_of(int fmt) { return fmt == TSLT_PROB_F32 ? 32 : 16; }

inline bool payload_shape(int k, int V, int fmt, int* bi, int* bp, int* words) {
    if (fmt != TSLT_PROB_F32 && fmt != TSLT_PROB_BF16 && fmt != TSLT_PROB_F16) return false;
    *bi = index_bits_of(V);
    *bp = prob_bits_of(fmt);
    *words = 1 + (int)(((long long)k * (*bi + *bp) + 31) / 32);
    return true;
}

__device__ __forceinline__ float pattern_value(uint32_t p, int fmt) {
    if (fmt == TSLT_PROB_F32) return __uint_as_float(p);
    if (fmt == TSLT_PROB_BF16) return __uint_as_float(p << 16);
    return __half2float(__ushort_as_half((unsigned short)p));
}

// Entry e of a record from the three words it can touch (lo = word 1 + (e * w >> 5), then the next two;
// words past the record read as 0): its token index and its value.
__device__ __forceinline__ void decode_entry(unsigned long long lo, unsigned long long mid, unsigned long long hi, int e,
                                             int bi, int bp, int fmt, int* idx, float* value) {
    const int sh = (int)(((long long)e * (bi + bp)) & 31);
    unsigned long long entry = (lo | (mid << 32)) >> sh;
    if (sh) entry |= hi << (64 - sh);
    *idx = (int)(entry & ((1ull << bi) - 1ull));
    *value = pattern_value((uint32_t)((entry >> bi) & (bp == 32 ? 0xffffffffull : 0xffffull)), fmt);
}

}  // namespace tslt
