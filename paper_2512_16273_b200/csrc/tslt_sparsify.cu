// tslt_sparsify: draft-side sparsify-then-sample (Section 3, Solution 1; the sampling steps
// of Algorithms 2 and 4) as one kernel.
//
// One CTA streams one segment of one logits row through the bulk-copy ring exactly once.
// While streaming, each consumer thread keeps an online (max, sum) for the softmax
// normaliser and pushes every logit above a running threshold tau into a shared candidate
// buffer.  tau is the exact k-th largest logit seen so far (radix select with ties broken
// toward the lower index), so the buffer always contains the row's top-k.  The CTA that
// holds the whole row (the only one, or the last of the row's segments to finish) then
// trims to the exact top-k, applies the top-rho cut, renormalises in fp64, draws the samples
// by inverse CDF and writes the (index, logit) pairs in ascending index.
#include <math.h>

#include "tslt_common.cuh"
#include "tslt_rowmath.cuh"
#include "tslt_select.cuh"
#include "tslt_stream.cuh"

namespace tslt {

struct SegStat {
    double S;  // sum of 2^(y - M) over the segment
    float M;   // reference exponent (base 2)
    int n;     // candidates written for the segment
};

struct SparsifyParams {
    const unsigned char* logits;
    long long row_stride_bytes;
    long long row_bytes;
    int V, rows, k;
    float top_p;
    ScaleC c;
    int num_samples;
    const float* uniforms;
    int* idx;
    float* logit;
    int* count;
    int* token;
    float* lse;
    float* mass;
    int nseg, tiles_per_seg, ntiles;
    int cap, high;
    int idx_hi_byte;
    int* status;
    int* tickets;
    SegStat* seg_stats;
    uint2* seg_entries;  // [rows, nseg, k] (key, idx)
};

struct SparsifyShared {
    RingBars bars;
    SelectScratch sel;
    double scratch[16];
    float tau;
    int cand_count;
    int overflow;
    int ticket;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// shared-memory carve-up (dynamic): ring | cand_key | cand_idx | tmp_key | tmp_idx | SparsifyShared
__host__ __device__ inline size_t sparsify_smem_bytes(int cap, int k) {
    return kRingBytes + (size_t)cap * 8 + (size_t)k * 8 + align_up(sizeof(SparsifyShared), 16) + 256;
}

// Sources for select_topk: the candidate buffer, one ring tile, or both.
struct BufferSrc {
    const uint32_t* k_;
    const int* i_;
    __device__ __forceinline__ bool valid(int) const { return true; }
    __device__ __forceinline__ uint32_t key(int i) const { return k_[i]; }
    __device__ __forceinline__ int idx(int i) const { return i_[i]; }
};
template <typename T> struct TileSrc {
    const unsigned char* tile;
    int elem0;
    __device__ __forceinline__ bool valid(int i) const { return tile_elem<T>(tile, i) > -INFINITY; }
    __device__ __forceinline__ uint32_t key(int i) const { return float_to_key(tile_elem<T>(tile, i)); }
    __device__ __forceinline__ int idx(int i) const { return elem0 + i; }
};
// entries of the buffer that precede the tile, followed by every logit of the tile above tau
template <typename T> struct UnionSrc {
    const uint32_t* k_;
    const int* i_;
    int nb;
    const unsigned char* tile;
    int elem0;
    float tau;
    __device__ __forceinline__ bool valid(int i) const {
        return i < nb ? i_[i] < elem0 : tile_elem<T>(tile, i - nb) > tau;
    }
    __device__ __forceinline__ uint32_t key(int i) const {
        return i < nb ? k_[i] : float_to_key(tile_elem<T>(tile, i - nb));
    }
    __device__ __forceinline__ int idx(int i) const { return i < nb ? i_[i] : elem0 + (i - nb); }
};

__device__ __forceinline__ int barrier_or(bool pred) {
    int any;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.s32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\tselp.s32 %0, 1, 0, p;\n\t}"
        : "=r"(any)
        : "r"((int)pred), "n"(kConsumerBarrier), "n"(kConsumerThreads)
        : "memory");
    return any;
}

// Trim the candidate buffer to its exact top-k and raise tau to the k-th logit once k exist.
template <bool kKeyHiOnly>
__device__ __forceinline__ void rebuild(Candidates cb, int k, int idx_hi_byte, SparsifyShared* sh, int tid) {
    const int n = min(*cb.count, 1 << 30);
    consumer_sync();
    if (n <= k) return;  // nothing to trim; tau unchanged (uniform: n is the same for every thread)
    uint32_t kth;
    BufferSrc src{cb.key, cb.idx};
    const bool full = select_topk<kKeyHiOnly>(src, n, k, idx_hi_byte, cb, &sh->sel, tid, &kth);
    if (full && tid == 0) sh->tau = key_to_float(kth);
    consumer_sync();
}

template <typename T>
__device__ __noinline__ void finalize_row(const SparsifyParams& p, int row, Candidates cb, SparsifyShared* sh,
                                          unsigned char* ring, double Mrow, double Srow, int tid);

template <typename T>
__global__ void __launch_bounds__(kBlockThreads, 3) sparsify_kernel(const SparsifyParams p) {
    constexpr bool kHiOnly = (Elt<T>::kBytes == 2);
    constexpr int kPer = Elt<T>::kPerVec;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>(align_up((size_t)smem_raw, 128));
    uint32_t* cand_key = reinterpret_cast<uint32_t*>(ring + kRingBytes);
    int* cand_idx = reinterpret_cast<int*>(cand_key + p.cap);
    uint32_t* tmp_key = reinterpret_cast<uint32_t*>(cand_idx + p.cap);
    int* tmp_idx = reinterpret_cast<int*>(tmp_key + p.k);
    SparsifyShared* sh = reinterpret_cast<SparsifyShared*>(align_up((size_t)(tmp_idx + p.k), 16));

    const int tid = threadIdx.x;
    const int row = blockIdx.x / p.nseg, seg = blockIdx.x % p.nseg;
    const unsigned char* rowp = p.logits + (long long)row * p.row_stride_bytes;
    const int tile_begin = seg * p.tiles_per_seg;
    const int tile_end = min(p.ntiles, tile_begin + p.tiles_per_seg);

    ring_init(&sh->bars, tid);
    if (tid == 0) {
        sh->tau = -INFINITY;
        sh->cand_count = 0;
        sh->overflow = 0;
    }
    __syncthreads();

    if (tid >= kConsumerThreads) {
        producer_loop<T>(rowp, p.row_bytes, tile_begin, tile_end, ring, &sh->bars, p.status);
        return;
    }

    Candidates cb{cand_key, cand_idx, tmp_key, tmp_idx, &sh->cand_count};
    const int lane = tid & 31, warp = tid >> 5;
    const int cap = p.cap, high = p.high, k = p.k;
    const float chi = p.c.hi, clo = p.c.lo;

    // ---- streaming pass ----------------------------------------------------------------
    LaneSum ls;
    ls.reset();
    bool live = true;

    for (int t = tile_begin; t < tile_end; ++t) {
        const int it = t - tile_begin, s = it % kStages;
        const bool arrived = mbar_wait(&sh->bars.full[s], (uint32_t)((it / kStages) & 1), &sh->bars.abort);
        const uint32_t padded = tile_padded_bytes(p.row_bytes, t);
        const unsigned char* tile = ring + s * kTileBytes;
        const float tau = sh->tau;
        const int tile_elem0 = t * (kTileBytes / Elt<T>::kBytes);
        // the first tile of a segment is not filtered: its exact top-k is selected in place below
        bool want_action = !arrived || it == 0;
        if (arrived) {
            LaneTile<T> lt;
            lt.load(tile, warp, lane, padded);
            const float lm = lt.lane_max();
            if (lm > ls.zmax) ls.raise(lm, chi, clo);
            lt.accumulate(ls, chi, clo);
            if (it != 0 && lm > tau) {
#pragma unroll
                for (int j = 0; j < kVecsPerLane; ++j) {
                    if (lt.vec_max(j) > tau) {
                        const int e0 = tile_elem0 + (warp * kChunkBytes + (j * 32 + lane) * kVecBytes) / Elt<T>::kBytes;
#pragma unroll
                        for (int e = 0; e < kPer; ++e) {
                            const float z = lt.elem(j, e);
                            if (z > tau) {
                                const int pos = atomicAdd(&sh->cand_count, 1);
                                if (pos < cap) {
                                    cand_key[pos] = float_to_key(z);
                                    cand_idx[pos] = e0 + e;
                                } else {
                                    sh->overflow = 1;
                                }
                                if (pos + 1 > high) want_action = true;
                            }
                        }
                    }
                }
            }
        }
        // one barrier per tile: it also tells everyone whether the buffer needs attention
        if (barrier_or(want_action)) {
            // a wait that ran out is decided collectively, so that nobody is left at a barrier
            if (barrier_or(!arrived)) {
                if (!arrived) raise_abort(&sh->bars, p.status);
                live = false;
                break;
            }
            const int tile_elems = (int)(padded / Elt<T>::kBytes);
            uint32_t kth;
            bool full;
            if (it == 0) {
                TileSrc<T> src{tile, tile_elem0};
                full = select_topk<kHiOnly>(src, tile_elems, k, p.idx_hi_byte, cb, &sh->sel, tid, &kth);
            } else {
                const int ovf = sh->overflow;
                const int nb = min(sh->cand_count, cap);
                consumer_sync();
                if (!ovf) {
                    BufferSrc src{cand_key, cand_idx};
                    full = select_topk<kHiOnly>(src, nb, k, p.idx_hi_byte, cb, &sh->sel, tid, &kth);
                } else {
                    // this tile brought more candidates than fit: redo it from shared memory, selecting
                    // over the earlier entries of the buffer and every logit of the tile above tau
                    if (tid == 0) sh->overflow = 0;
                    UnionSrc<T> src{cand_key, cand_idx, nb, tile, tile_elem0, tau};
                    full = select_topk<kHiOnly>(src, nb + tile_elems, k, p.idx_hi_byte, cb, &sh->sel, tid, &kth);
                }
            }
            if (full && tid == 0) sh->tau = key_to_float(kth);
            consumer_sync();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->bars.empty[s]);
    }
    if (!live) return;  // status word already set; outputs left untouched
    consumer_sync();

    // ---- row statistics ------------------------------------------------------------------
    float Mrow_f = warp_max(ls.M);
    if (lane == 0) sh->scratch[warp] = (double)Mrow_f;
    consumer_sync();
    double Mrow = sh->scratch[0];
    for (int w = 1; w < kConsumerWarps; ++w) Mrow = fmax(Mrow, sh->scratch[w]);
    consumer_sync();
    double Srow = block_sum(ls.total_f64() * exp2((double)ls.M - Mrow), tid, sh->scratch);

    // ---- segments of a split row meet through the workspace; the last to arrive goes on ------
    if (p.nseg > 1) {
        rebuild<kHiOnly>(cb, k, p.idx_hi_byte, sh, tid);  // <= k entries per segment
        const int n = sh->cand_count;
        uint2* my_entries = p.seg_entries + ((size_t)row * p.nseg + seg) * (size_t)k;
        for (int i = tid; i < n; i += kConsumerThreads) my_entries[i] = make_uint2(cand_key[i], (uint32_t)cand_idx[i]);
        if (tid == 0) {
            SegStat st;
            st.S = Srow;
            st.M = (float)Mrow;
            st.n = n;
            p.seg_stats[(size_t)row * p.nseg + seg] = st;
        }
        __threadfence();
        consumer_sync();
        if (tid == 0) sh->ticket = atomicAdd(&p.tickets[row], 1);
        consumer_sync();
        if (sh->ticket != p.nseg - 1) return;
        __threadfence();
        // gather every segment's candidates and statistics
        if (tid == 0) sh->cand_count = 0;
        consumer_sync();
        double Mall = -INFINITY;
        for (int g = 0; g < p.nseg; ++g) {
            const SegStat* st = &p.seg_stats[(size_t)row * p.nseg + g];
            Mall = fmax(Mall, (double)__ldcg(&st->M));
        }
        double Sall = 0.0;
        for (int g = 0; g < p.nseg; ++g) {
            const SegStat* st = &p.seg_stats[(size_t)row * p.nseg + g];
            const double Sg = __ldcg(&st->S);
            const double Mg = (double)__ldcg(&st->M);
            Sall += Sg * exp2(Mg - Mall);
            const int ng = __ldcg(&st->n);
            const uint2* ent = p.seg_entries + ((size_t)row * p.nseg + g) * (size_t)k;
            const int base = sh->cand_count;
            for (int i = tid; i < ng; i += kConsumerThreads) {
                uint2 e2 = __ldcg(&ent[i]);
                cand_key[base + i] = e2.x;
                cand_idx[base + i] = (int)e2.y;
            }
            consumer_sync();
            if (tid == 0) sh->cand_count = base + ng;
            consumer_sync();
        }
        Mrow = Mall;
        Srow = Sall;
    }

    finalize_row<T>(p, row, cb, sh, ring, Mrow, Srow, tid);
}

// Exact top-k of the row, nucleus cut, renormalisation, sampling and the ascending-index payload.
template <typename T>
__device__ __noinline__ void finalize_row(const SparsifyParams& p, int row, Candidates cb, SparsifyShared* sh,
                                          unsigned char* ring, double Mrow, double Srow, int tid) {
    constexpr bool kHiOnly = (Elt<T>::kBytes == 2);
    const int k = p.k;
    uint32_t* cand_key = cb.key;
    int* cand_idx = cb.idx;
    rebuild<kHiOnly>(cb, k, p.idx_hi_byte, sh, tid);
    const int n0 = min(sh->cand_count, k);
    const double L2 = Mrow + log2(Srow);  // base-2 log of the softmax normaliser
    const double cd = p.c.d;
    // the ring is idle now: reuse it for the fp64 work arrays
    unsigned long long* comp = reinterpret_cast<unsigned long long*>(ring);           // 1024 * 8
    double* wv = reinterpret_cast<double*>(ring + 8192);                              // 1024 * 8
    double* cum = reinterpret_cast<double*>(ring + 16384);                            // 1024 * 8
    int n = n0;
    double mass = 0.0;
    if (n0 > 0 && p.top_p < 1.0f) {
        // order the candidates by (logit descending, index ascending) and cut at the nucleus
        const int P = next_pow2(n0);
        for (int i = tid; i < P; i += kConsumerThreads)
            comp[i] = i < n0 ? (((unsigned long long)cand_key[i] << 32) | (unsigned long long)(0xffffffffu - (uint32_t)cand_idx[i])) : 0ull;
        consumer_sync();
        bitonic_sort<true>(comp, P, tid);
        for (int i = tid; i < n0; i += kConsumerThreads) {
            const float z = key_to_float((uint32_t)(comp[i] >> 32));
            cum[i] = exp2((double)z * cd - L2);
        }
        consumer_sync();
        block_inclusive_scan(cum, n0, tid, sh->scratch);
        // n* = first n with c_n >= top_p
        const double tp = (double)p.top_p;
        int lo = 0, hi = n0;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (cum[mid] >= tp) hi = mid; else lo = mid + 1;
        }
        n = lo < n0 ? lo + 1 : n0;
        mass = cum[n - 1];
        consumer_sync();
        for (int i = tid; i < n; i += kConsumerThreads) {
            cand_key[i] = (uint32_t)(comp[i] >> 32);
            cand_idx[i] = (int)(0xffffffffu - (uint32_t)(comp[i] & 0xffffffffull));
        }
        consumer_sync();
    }
    // ascending index order
    if (n > 0) {
        const int P = next_pow2(n);
        for (int i = tid; i < P; i += kConsumerThreads)
            comp[i] = i < n ? (((unsigned long long)(uint32_t)cand_idx[i] << 32) | (unsigned long long)cand_key[i]) : ~0ull;
        consumer_sync();
        bitonic_sort<false>(comp, P, tid);
    }
    // renormalised truncated distribution in fp64: w_i = 2^(y_i - m_S), CDF by inclusive scan
    double my_max = -INFINITY;
    for (int i = tid; i < n; i += kConsumerThreads) {
        const float z = key_to_float((uint32_t)(comp[i] & 0xffffffffull));
        const double y = (double)z * cd;
        wv[i] = y;
        my_max = fmax(my_max, y);
    }
    const double mS = block_max(my_max, tid, sh->scratch);
    double my_mass = 0.0;
    for (int i = tid; i < n; i += kConsumerThreads) {
        const double y = wv[i];
        if (!(p.top_p < 1.0f)) my_mass += exp2(y - L2);
        const double w = exp2(y - mS);
        wv[i] = w;
        cum[i] = w;
    }
    if (!(p.top_p < 1.0f)) mass = block_sum(my_mass, tid, sh->scratch);
    else consumer_sync();
    block_inclusive_scan(cum, n, tid, sh->scratch);

    // ---- outputs ------------------------------------------------------------------------------
    int* o_idx = p.idx + (size_t)row * k;
    float* o_logit = p.logit + (size_t)row * k;
    for (int i = tid; i < k; i += kConsumerThreads) {
        if (i < n) {
            o_idx[i] = (int)(comp[i] >> 32);
            o_logit[i] = key_to_float((uint32_t)(comp[i] & 0xffffffffull));
        } else {
            o_idx[i] = -1;
            o_logit[i] = -INFINITY;
        }
    }
    if (tid == 0) {
        p.count[row] = n;
        if (p.lse) p.lse[row] = n0 > 0 ? (float)(L2 * 0.6931471805599453) : -INFINITY;
        if (p.mass) p.mass[row] = n0 > 0 ? (float)mass : 0.f;
    }
    const double W = n > 0 ? cum[n - 1] : 0.0;
    for (int sidx = tid; sidx < p.num_samples; sidx += kConsumerThreads) {
        int tok = -1;
        if (n > 0) {
            const float u = clamp_uniform(p.uniforms[(size_t)row * p.num_samples + sidx]);
            int pos = first_greater(cum, n, (double)u * W);
            if (pos >= n) {
                pos = n - 1;
                while (pos > 0 && !(wv[pos] > 0.0)) --pos;
            }
            tok = (int)(comp[pos] >> 32);
        }
        p.token[(size_t)row * p.num_samples + sidx] = tok;
    }
}

// ---- host side -------------------------------------------------------------------------------

struct SparsifyPlan {
    int nseg, tiles_per_seg, ntiles, cap, high;
    size_t smem;
    size_t ws_tickets_off, ws_stats_off, ws_entries_off, ws_bytes;
};

static int sm_count_cached() {
    static int sms = 0;
    if (sms == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
        sms = v;
    }
    return sms;
}

static SparsifyPlan make_sparsify_plan(int rows, int V, int k, int elt_bytes) {
    SparsifyPlan pl;
    const long long row_bytes = (long long)V * elt_bytes;
    pl.ntiles = (int)((row_bytes + kTileBytes - 1) / kTileBytes);
    pl.cap = 4 * k;
    if (pl.cap < 2048) pl.cap = 2048;
    if (pl.cap > 4096) pl.cap = 4096;
    pl.high = pl.cap - pl.cap / 4;
    // Split a row over several CTAs when there are too few rows to fill the machine.
    const int sms = sm_count_cached();
    int nseg = 1;
    const int max_seg_by_cap = pl.cap / k;
    while (nseg < 16 && nseg * 2 <= max_seg_by_cap && (long long)rows * nseg < 4LL * sms &&
           pl.ntiles / (nseg * 2) >= 2)
        nseg *= 2;
    pl.tiles_per_seg = (pl.ntiles + nseg - 1) / nseg;
    pl.nseg = (pl.ntiles + pl.tiles_per_seg - 1) / pl.tiles_per_seg;
    if (pl.nseg < 1) pl.nseg = 1;
    pl.smem = sparsify_smem_bytes(pl.cap, k);
    size_t off = kWsHeaderBytes;
    pl.ws_tickets_off = off;
    off = align_up(off + (size_t)rows * sizeof(int), 256);
    pl.ws_stats_off = off;
    off = align_up(off + (size_t)rows * pl.nseg * sizeof(SegStat), 256);
    pl.ws_entries_off = off;
    off = align_up(off + (pl.nseg > 1 ? (size_t)rows * pl.nseg * k * sizeof(uint2) : 0), 256);
    pl.ws_bytes = off;
    return pl;
}

ScaleC make_scale(float temperature) {
    const double c = 1.4426950408889634 / (double)temperature;
    ScaleC s;
    float hi = (float)c;
    if ((double)hi > c) hi = nextafterf(hi, 0.0f);
    float lo = (float)(c - (double)hi);
    if (!(lo > 0.0f)) lo = 1e-30f;
    s.hi = hi;
    s.lo = lo;
    s.d = (double)hi + (double)lo;
    return s;
}

}  // namespace tslt

using namespace tslt;

extern "C" int tslt_sparsify_workspace_bytes(int rows, int V, int k, int num_samples, size_t* bytes) {
    if (!bytes || rows < 0 || V <= 0 || k <= 0 || k > V || k > TSLT_MAX_K || num_samples < 0)
        return TSLT_ERR_INVALID_ARG;
    SparsifyPlan a = make_sparsify_plan(rows, V, k, 2), b = make_sparsify_plan(rows, V, k, 4);
    *bytes = a.ws_bytes > b.ws_bytes ? a.ws_bytes : b.ws_bytes;
    return TSLT_OK;
}

extern "C" int tslt_sparsify(const void* logits, int dtype, int B, int gamma, int V,
                             long long row_stride_elems, int k, float top_p, float temperature,
                             int num_samples, const float* uniforms, int* idx, float* logit, int* count,
                             int* token, float* lse, float* mass, void* workspace, size_t workspace_bytes,
                             void* stream) {
    if (dtype != TSLT_F32 && dtype != TSLT_BF16) return TSLT_ERR_UNSUPPORTED;
    const int eb = dtype == TSLT_F32 ? 4 : 2;
    if (B < 0 || gamma < 0 || V <= 0 || k <= 0 || k > V || !(top_p > 0.0f) || !(temperature > 0.0f) ||
        !isfinite(temperature) || num_samples < 0)
        return TSLT_ERR_INVALID_ARG;
    if (k > TSLT_MAX_K) return TSLT_ERR_UNSUPPORTED;
    const long long rows_ll = (long long)B * gamma;
    if (rows_ll > 0x7fffffffLL / 16) return TSLT_ERR_UNSUPPORTED;
    const int rows = (int)rows_ll;
    if (rows == 0) return TSLT_OK;
    if (!logits || !idx || !logit || !count || !workspace || (num_samples > 0 && (!uniforms || !token)))
        return TSLT_ERR_INVALID_ARG;
    if (row_stride_elems < V || ((uintptr_t)logits & 15) || ((row_stride_elems * eb) & 15) ||
        ((uintptr_t)workspace & 255))
        return TSLT_ERR_INVALID_ARG;
    SparsifyPlan pl = make_sparsify_plan(rows, V, k, eb);
    if (workspace_bytes < pl.ws_bytes) return TSLT_ERR_WORKSPACE;

    SparsifyParams p;
    p.logits = (const unsigned char*)logits;
    p.row_stride_bytes = row_stride_elems * eb;
    p.row_bytes = (long long)V * eb;
    p.V = V; p.rows = rows; p.k = k;
    p.top_p = top_p;
    p.c = make_scale(temperature);
    p.num_samples = num_samples;
    p.uniforms = uniforms;
    p.idx = idx; p.logit = logit; p.count = count; p.token = token; p.lse = lse; p.mass = mass;
    p.nseg = pl.nseg; p.tiles_per_seg = pl.tiles_per_seg; p.ntiles = pl.ntiles;
    p.cap = pl.cap; p.high = pl.high;
    p.idx_hi_byte = (V - 1) >= (1 << 24) ? 3 : (V - 1) >= (1 << 16) ? 2 : (V - 1) >= (1 << 8) ? 1 : 0;
    unsigned char* ws = (unsigned char*)workspace;
    p.status = (int*)ws;
    p.tickets = (int*)(ws + pl.ws_tickets_off);
    p.seg_stats = (SegStat*)(ws + pl.ws_stats_off);
    p.seg_entries = (uint2*)(ws + pl.ws_entries_off);

    cudaStream_t st = (cudaStream_t)stream;
    // status word and tickets start at zero
    if (cudaMemsetAsync(ws, 0, pl.ws_stats_off, st) != cudaSuccess) return TSLT_ERR_CUDA;
    auto kern = dtype == TSLT_F32 ? sparsify_kernel<float> : sparsify_kernel<bf16_t>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem) != cudaSuccess)
        return TSLT_ERR_CUDA;
    kern<<<rows * pl.nseg, kBlockThreads, pl.smem, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? TSLT_OK : TSLT_ERR_CUDA;
}
