// Uplink payload of TSLT: bit-packed (token index, logit) records (Section 2.2 of the paper gives
// the bit widths; the record layout is stated in include/tslt.h).  Two small kernels, one CTA per
// row: the work is a few hundred entries per row, so the only things that matter are coalesced
// record traffic and not serialising the threads of a row on shared words.
#include "tslt_payload.cuh"

namespace tslt {

constexpr int kPayloadThreads = 128;

// fp32 -> bf16 bit pattern, round to nearest even; inf stays inf, NaN stays NaN.
__device__ __forceinline__ uint32_t bf16_pattern(float x) {
    const uint32_t u = __float_as_uint(x);
    if ((u & 0x7f800000u) == 0x7f800000u) {
        uint32_t hi = u >> 16;
        if ((u & 0x007fffffu) && !(hi & 0x7fu)) hi |= 1u;
        return hi;
    }
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ uint32_t value_pattern(float x, int fmt) {
    if (fmt == TSLT_PROB_F32) return __float_as_uint(x);
    if (fmt == TSLT_PROB_BF16) return bf16_pattern(x);
    return (uint32_t)__half_as_ushort(__float2half_rn(x));
}
// One CTA per row.  The record is assembled in shared memory: an entry of w <= 63 bits touches at
// most three words, each through atomicOr (neighbouring entries share words), then the record goes
// out with coalesced stores.
__global__ void __launch_bounds__(kPayloadThreads) pack_payload_kernel(const int* __restrict__ idx,
                                                                        const float* __restrict__ logit,
                                                                        const int* __restrict__ count, int k, int bi, int bp,
                                                                        int fmt, int words, uint32_t* __restrict__ payload,
                                                                        long long* __restrict__ payload_bits) {
    extern __shared__ uint32_t rec[];
    const int row = blockIdx.x, tid = threadIdx.x;
    int n = count[row];
    n = n < 0 ? 0 : (n > k ? k : n);
    for (int i = tid; i < words; i += kPayloadThreads) rec[i] = 0u;
    __syncthreads();
    if (tid == 0) rec[0] = (uint32_t)n;
    const int w = bi + bp;
    for (int e = tid; e < n; e += kPayloadThreads) {
        const unsigned long long entry = ((unsigned long long)(uint32_t)idx[(size_t)row * k + e] & ((1ull << bi) - 1ull)) |
                                         ((unsigned long long)value_pattern(logit[(size_t)row * k + e], fmt) << bi);
        const long long pos = (long long)e * w;
        const int word = 1 + (int)(pos >> 5), sh = (int)(pos & 31);
        // the entry, shifted into place, spans up to 96 bits
        const uint32_t lo = (uint32_t)(entry << sh);
        const uint32_t mid = (uint32_t)(sh ? (entry >> (32 - sh)) : (entry >> 32));
        const uint32_t hi = sh ? (uint32_t)(entry >> 32 >> (32 - sh)) : 0u;
        if (lo) atomicOr(&rec[word], lo);
        if (mid) atomicOr(&rec[word + 1], mid);
        if (hi) atomicOr(&rec[word + 2], hi);
    }
    __syncthreads();
    uint32_t* out = payload + (size_t)row * words;
    for (int i = tid; i < words; i += kPayloadThreads) out[i] = rec[i];
    if (payload_bits && tid == 0) payload_bits[row] = (long long)n * w;
}

__global__ void __launch_bounds__(kPayloadThreads) unpack_payload_kernel(const uint32_t* __restrict__ payload, int k, int bi,
                                                                          int bp, int fmt, int words, int* __restrict__ idx,
                                                                          float* __restrict__ logit, int* __restrict__ count,
                                                                          int* __restrict__ device_flag) {
    extern __shared__ uint32_t rec[];
    const int row = blockIdx.x, tid = threadIdx.x;
    const uint32_t* in = payload + (size_t)row * words;
    for (int i = tid; i < words; i += kPayloadThreads) rec[i] = in[i];
    if (tid == 0) rec[words] = rec[words + 1] = 0u;  // an entry may be read as three whole words
    __syncthreads();
    int n = (int)rec[0];
    if (n < 0 || n > k) {  // not a record this library wrote
        if (tid == 0 && device_flag) *device_flag = 1;
        n = 0;
    }
    const int w = bi + bp;
    for (int e = tid; e < k; e += kPayloadThreads) {
        int i_out = -1;
        float z_out = -INFINITY;
        if (e < n) {
            const int word = 1 + (int)(((long long)e * w) >> 5);
            decode_entry(rec[word], rec[word + 1], rec[word + 2], e, bi, bp, fmt, &i_out, &z_out);
        }
        idx[(size_t)row * k + e] = i_out;
        logit[(size_t)row * k + e] = z_out;
    }
    if (tid == 0) count[row] = n;
}

}  // namespace tslt

using namespace tslt;

extern "C" int tslt_payload_words(int k, int V, int prob_format, int* words, int* entry_bits) {
    if (k <= 0 || k > TSLT_MAX_K || V <= 0 || !words) return TSLT_ERR_INVALID_ARG;
    int bi, bp, w;
    if (!payload_shape(k, V, prob_format, &bi, &bp, &w)) return TSLT_ERR_UNSUPPORTED;
    *words = w;
    if (entry_bits) *entry_bits = bi + bp;
    return TSLT_OK;
}

extern "C" int tslt_pack_payload(const int* idx, const float* logit, const int* count, int rows, int k, int V,
                                 int prob_format, unsigned int* payload, long long* payload_bits, void* stream) {
    if (rows < 0 || k <= 0 || k > TSLT_MAX_K || V <= 0) return TSLT_ERR_INVALID_ARG;
    int bi, bp, words;
    if (!payload_shape(k, V, prob_format, &bi, &bp, &words)) return TSLT_ERR_UNSUPPORTED;
    if (rows == 0) return TSLT_OK;
    if (!idx || !logit || !count || !payload) return TSLT_ERR_INVALID_ARG;
    pack_payload_kernel<<<rows, kPayloadThreads, (size_t)(words + 2) * sizeof(uint32_t), (cudaStream_t)stream>>>(
        idx, logit, count, k, bi, bp, prob_format, words, payload, payload_bits);
    return cudaGetLastError() == cudaSuccess ? TSLT_OK : TSLT_ERR_CUDA;
}

extern "C" int tslt_unpack_payload(const unsigned int* payload, int rows, int k, int V, int prob_format, int* idx,
                                   float* logit, int* count, int* device_flag, void* stream) {
    if (rows < 0 || k <= 0 || k > TSLT_MAX_K || V <= 0) return TSLT_ERR_INVALID_ARG;
    int bi, bp, words;
    if (!payload_shape(k, V, prob_format, &bi, &bp, &words)) return TSLT_ERR_UNSUPPORTED;
    if (rows == 0) return TSLT_OK;
    if (!payload || !idx || !logit || !count) return TSLT_ERR_INVALID_ARG;
    unpack_payload_kernel<<<rows, kPayloadThreads, (size_t)(words + 2) * sizeof(uint32_t), (cudaStream_t)stream>>>(
        payload, k, bi, bp, prob_format, words, idx, logit, count, device_flag);
    return cudaGetLastError() == cudaSuccess ? TSLT_OK : TSLT_ERR_CUDA;
}
