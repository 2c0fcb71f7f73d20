// tslt_sparsify: draft-side sparsify-then-sample (Section 3, Solution 1; the sampling steps
// of Algorithms 2 and 4) as two kernels on the caller's stream.
//
// Streaming kernel.  One CTA reads one segment of one logits row from HBM exactly once, with
// 16-byte loads that go straight to registers (each warp instruction covers 512 contiguous
// bytes).  Warps run freely: there is no barrier in the steady state.  Each lane keeps an online
// (max, sum) for the softmax normaliser and stages every lane tile (its four 16-byte vectors of a
// 2 KB chunk) that holds a logit at or above a running threshold: 8 bytes (where the tile is,
// which of its vectors hold a candidate, the key of its largest logit), no data.  The test is on
// the tile's packed maximum, so a tile without a candidate costs a handful of instructions and
// nothing is searched inside a vector while streaming.  The threshold comes from a 4096-bin
// histogram of the order-preserving keys (top 12 bits) of what is staged: the highest bin above
// which at least k distinct logits have been counted is a lower bound on the row's k-th largest
// logit, so no member of the top-k is ever skipped, whatever the order in which the warps run.
// The warps take turns at checking whether enough has been counted for the threshold to rise,
// and rescan the histogram then.  At the end the segment hands over its per-warp (max, sum)
// pairs and either the staged tiles as they are (k <= 256, the usual case) or the (key, index)
// candidates it expanded from them by reading the marked vectors back.
//
// Finish kernel (launched with programmatic stream serialization, so that it is in place when
// the streaming kernel ends).  One CTA per row: candidates from the hand-over, the bin that holds
// the k-th largest logit, everything above it, the tie inside it broken exactly (logit
// descending, index ascending), the top-rho cut, renormalisation in fp64, the samples by inverse
// CDF, the (index, logit) pairs in ascending index.
//
// Rare paths: a staging buffer that fills up is expanded early by all warps together (and the
// candidate list compacted to the current threshold); a buffer that overflows before they can
// meet (adversarial rows: sorted ascending, all equal) is abandoned and the segment is read a
// second time against the final threshold; a candidate list that overflows even then is selected
// again from global memory with a radix select.
#include <math.h>

#include "tslt_common.cuh"
#include "tslt_rowmath.cuh"
#include "tslt_select.cuh"

namespace tslt {

constexpr int kHistBins = 4096;   // fine bins: key >> 20 (sign, exponent and three mantissa bits)
constexpr int kHistShift = 20;
constexpr int kCoarseBins = 128;  // coarse bin = fine bin >> 5: lets a scan find the right 32 fine bins in one step
constexpr int kLowestFiniteBin = 0x00800000u >> kHistShift;  // bin of -FLT_MAX: every finite logit passes
constexpr int kBoundaryCap = 960;   // entries of the k-th logit's bin that the direct tie-break handles
constexpr int kArenaBytes = 24576;  // histograms (16.5 KB) + boundary list (7.5 KB); fp64 work arrays afterwards
constexpr int kSparsifyCtasPerSm = 4;  // 64 registers per thread
constexpr int kPrefetchSteps = 1;      // how many of its own steps ahead a warp asks L2 for its chunk
constexpr int kRankSortMax = 256;   // up to this many entries are ordered by counting, more by a bitonic sort

struct SegStat {
    double S[kWarps];  // per warp: sum of 2^(y - M) over the warp's chunks of the segment
    float M[kWarps];   // per warp: reference exponent (base 2)
    int n;             // entries written for the segment
    int raw_bin;       // -1: the entries are (key, idx) candidates; else they are staged lane tiles (first vector
                       // and vector mask, relative key of the largest logit) and this is the segment's final
                       // threshold bin
    float z0;          // the segment's offset: bins are over z - z0 (see rel_key)
    int pad;
};

struct SparsifyParams {
    const unsigned char* logits;
    long long row_stride_bytes;
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
    int nchunks;
    RowSplit split;
    int cap, high;      // candidate (key, index) list of the streaming kernel: capacity and compaction mark
    int fin_cap;        // candidate list of the finish kernel: what the row's segments can hand over
    int vcap, vhigh;    // staged lane tiles: capacity and early-expansion mark
    int idx_hi_byte;
    int* status;
    SegStat* seg_stats;
    uint2* seg_entries;  // [rows, nseg, seg_stride]: (key, idx) candidates, or staged lane tiles handed over raw
    int seg_cap;         // most candidates a segment hands over
    int seg_stride;      // entries reserved per segment
    int raw_cap;         // > 0: a segment whose staging buffer never filled hands its staged tiles over unexpanded
    int* row_ready;      // [rows] (rows of one segment only, else NULL): set to 1 when the row has been handed over
};

struct SparsifyShared {
    // ---- written by stage_tile through their shared-space addresses ----------------------------------
    int vec_count;   // staged lane tiles
    int overflow;    // a buffer was found full: its contents are no longer complete
    int trim_request;
    int n_above;     // logits counted in bins above thr_bin since it last rose (may lag, never leads a rise)
    // --------------------------------------------------------------------------------------------
    int n_list;      // expand_staged: vectors listed for reading back
    int cand_count;  // expanded (key, index) candidates
    int thr_bin;     // candidates are the logits whose relative key's bin is >= thr_bin; only ever rises
    float z0;        // the segment's offset (see rel_key); fixed once the first chunks have been looked at
    uint32_t thr_edge_key;  // fp32 rows: order-preserving key of the raw-domain threshold the lane-tile test uses
    uint32_t thr_word;  // thr_bin << 16 | the bf16 pattern the packed lane-tile test compares with; only ever rises
    int sel_bin, sel_above;  // bin of the k-th largest logit and the number of logits in higher bins
    int n_win, n_bnd;
    int warp_tot[kWarps];
    double scratch[16];
    SelectScratch sel;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// shared-memory carve-up (dynamic):
//   SparsifyShared | arena | staged[vcap] | cand_key[cap] | cand_idx[cap] | tmp_key[k] | tmp_idx[k]
// The control block, the histograms and the staging buffer sit at compile-time offsets of the
// CTA's shared memory, so the streaming loop holds no address of them in a register.
constexpr uint32_t kSharedBlockBytes = (sizeof(SparsifyShared) + 127) / 128 * 128;
constexpr uint32_t kHistOff = kSharedBlockBytes;
constexpr uint32_t kCoarseOff = kHistOff + 4u * kHistBins;
constexpr uint32_t kStagedOff = kHistOff + kArenaBytes;
__host__ __device__ inline size_t sparsify_smem_bytes(int cap, int vcap, int k) {
    return align_up((size_t)kStagedOff + (size_t)vcap * 8 + (size_t)cap * 8 + (size_t)k * 8, 16);
}

// Sources for select_topk: the candidate buffer, or a run of logits in global memory.
struct BufferSrc {
    const uint32_t* k_;
    const int* i_;
    __device__ __forceinline__ bool valid(int) const { return true; }
    __device__ __forceinline__ uint32_t key(int i) const { return k_[i]; }
    __device__ __forceinline__ int idx(int i) const { return i_[i]; }
};
template <typename T> struct GlobalSrc {
    const unsigned char* row;
    int elem0;
    __device__ __forceinline__ bool valid(int i) const { return Elt<T>::load(row, elem0 + i) > -INFINITY; }
    __device__ __forceinline__ uint32_t key(int i) const { return float_to_key(Elt<T>::load(row, elem0 + i)); }
    __device__ __forceinline__ int idx(int i) const { return elem0 + i; }
};

__device__ __forceinline__ float bin_lower_edge(int bin) { return key_to_float((uint32_t)bin << kHistShift); }

// The histogram's bins are over the logits RELATIVE to an offset z0 taken from the segment's first
// chunks (their largest logit): a bin is the top 12 bits of the order-preserving key of z - z0.
// Float keys are relative (three mantissa bits: 12.5 % of the value), so bins over the raw logits
// would be as wide as the logits are large: a row of N(20, 1) logits put thousands of them in the
// threshold's bin and fell off every fast path (5.7 ms for 2048 rows of 256 000 bf16 logits instead of 0.23).
// Relative to a value near the row's maximum the bins are finest exactly where the top-k lives,
// whatever the offset and scale of the logits.  z - z0 is monotone in z (rounding is), which is all
// the threshold argument needs.  Candidates always carry their RAW keys: exact selection and
// ordering never see z0.
// (A finite z keeps a finite relative value, so that the lowest finite bin still admits every finite
// logit: -3e38 relative to +3e38 would otherwise round to -inf.)
__device__ __forceinline__ uint32_t rel_key(float z, float z0) { return float_to_key(fmaxf(z - z0, -3.4028234e38f)); }

// A raw-domain value that every logit whose relative bin is >= bin is at or above: the bin's lower
// edge moved back by z0, less a margin that covers the roundings of z - z0, of edge + z0 and of the
// subtraction itself (2^-21 of the magnitudes involved; each rounding is at most 2^-24 of one).
// Being low only lets a few more tiles through the streaming test; what they hold is then judged
// by its relative key.
__device__ __forceinline__ float raw_edge_below(int bin, float z0) {
    const float es = bin_lower_edge(bin);
    const float er = es + z0;
    return er - 4.76837158e-7f * (fabsf(es) + fabsf(z0) + fabsf(er));
}

// ---- shared memory by address: one out-of-line copy of the rare paths, still shared-space code ----
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float lds_f32(uint32_t addr) { return __uint_as_float(lds_u32(addr)); }
__device__ __forceinline__ void sts_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t atoms_add(uint32_t addr, uint32_t v) {
    uint32_t old;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void reds_add(uint32_t addr, uint32_t v) {
    asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// Count one logit in both histogram levels (fine first: a scan that sees the coarse count also
// finds the fine one).
__device__ __forceinline__ void hist_count(uint32_t hist_addr, uint32_t coarse_addr, int bin, uint32_t delta) {
    reds_add(hist_addr + 4u * (uint32_t)bin, delta);
    reds_add(coarse_addr + 4u * (uint32_t)(bin >> 5), delta);
}

__device__ __forceinline__ void sts_v2(uint32_t addr, uint32_t x, uint32_t y) {
    asm volatile("st.volatile.shared.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(x), "r"(y) : "memory");
}
// A warp hands out list positions with one atomic: returns where this lane's cnt entries start.
__device__ __forceinline__ int warp_reserve(int* counter, int cnt, int lane) {
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    int start = 0;
    if (lane == 31 && incl > 0) start = atomicAdd(counter, incl);
    return __shfl_sync(0xffffffffu, start, 31) + incl - cnt;
}


// Stage a lane tile (the four 16-byte vectors vec0, vec0 + 32, vec0 + 64, vec0 + 96 of the row)
// whose largest logit is vmax: only vec0, which of the four vectors hold a candidate, and the key
// of that logit are kept (8 bytes), and the logit is counted.  The tile's data is read again from
// global memory when the staged tiles are expanded, and only if its largest logit still passes
// the threshold of that moment: a fraction of what is staged.  `base` is the shared-space address
// of the CTA's dynamic shared memory.
constexpr int kTileMaskShift = 28;  // a staged tile's word: first vector (below 2^18) | mask of its four vectors << 28
// Count one logit of the row in the histogram, and towards the next rise of the threshold.
__device__ __forceinline__ void count_logit(uint32_t base, int thr_bin, uint32_t key) {
    hist_count(base + kHistOff, base + kCoarseOff, (int)(key >> kHistShift), 1u);
    if ((int)(key >> kHistShift) > thr_bin) reds_add(base + (uint32_t)offsetof(SparsifyShared, n_above), 1u);
}
// Small k counts the tile's largest logit only (two candidates seldom share a tile); large k, where
// most tiles hold some, counts the largest logit of every marked vector (count_tile false, the
// caller does it), or the threshold would sit too low.
constexpr int kCountPerVectorAboveK = 128;
__device__ __forceinline__ void stage_tile(uint32_t base, const SparsifyParams& p, int thr_bin, uint32_t tile_word,
                                           float vmax, bool count_tile) {
    const uint32_t pos = atoms_add(base + (uint32_t)offsetof(SparsifyShared, vec_count), 1u);
    const uint32_t key = rel_key(vmax, lds_f32(base + (uint32_t)offsetof(SparsifyShared, z0)));
    if (count_tile) count_logit(base, thr_bin, key);
    if (pos < (uint32_t)p.vcap) sts_v2(base + kStagedOff + 8u * pos, tile_word, key);
    else sts_u32(base + (uint32_t)offsetof(SparsifyShared, overflow), 1u);
    if (pos + 1u == (uint32_t)p.vhigh) sts_u32(base + (uint32_t)offsetof(SparsifyShared, trim_request), 1u);
}

// One warp: the highest fine bin b with (number of counted logits in bins >= b) >= k, or -1 if
// fewer than k are counted; *above gets the count in the bins above b (the total if none).
// Two steps whatever the values: the 128 coarse counts, then the 32 fine bins of the coarse bin
// in which the running count crosses k.
__device__ __noinline__ int scan_boundary(uint32_t hist_addr, uint32_t coarse_addr, int k, uint32_t* above_out) {
    const int lane = threadIdx.x & 31;
    // lane l owns coarse bins 127-4l .. 124-4l (descending)
    uint32_t c[4], tot = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        c[i] = lds_u32(coarse_addr + 4u * (uint32_t)(127 - 4 * lane - i));
        tot += c[i];
    }
    uint32_t incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, incl >= (uint32_t)k);
    if (!hit) {
        *above_out = __shfl_sync(0xffffffffu, incl, 31);
        return -1;
    }
    const int l = __ffs(hit) - 1;
    uint32_t run = incl - tot;  // counted above this lane's bins
    int cbin = 0;
    bool done = false;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (!done) {
            if (run + c[i] >= (uint32_t)k) {
                cbin = 127 - 4 * lane - i;
                done = true;
            } else {
                run += c[i];
            }
        }
    }
    cbin = __shfl_sync(0xffffffffu, cbin, l);
    const uint32_t above_c = __shfl_sync(0xffffffffu, run, l);
    // fine bins of that coarse bin, lane 0 the highest
    const int fb = cbin * 32 + 31 - lane;
    const uint32_t f = lds_u32(hist_addr + 4u * (uint32_t)fb);
    uint32_t fincl = f;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, fincl, o);
        if (lane >= o) fincl += t;
    }
    const unsigned fhit = __ballot_sync(0xffffffffu, above_c + fincl >= (uint32_t)k);
    if (!fhit) {  // the fine counts lag the coarse one (another warp is mid-push): nothing to report yet
        *above_out = 0;
        return -2;
    }
    const int fl = __ffs(fhit) - 1;
    *above_out = above_c + __shfl_sync(0xffffffffu, fincl - f, fl);
    return cbin * 32 + 31 - fl;
}

// The bf16 side of the threshold word: P = the largest bf16 value below raw_edge_below(bin, z0),
// never below -inf (the pattern that lets every finite logit through).
__device__ __forceinline__ uint32_t threshold_word(int bin, float z0) {
    uint32_t k16 = float_to_key(raw_edge_below(bin, z0)) >> 16;  // bf16 key at or below the edge ...
    k16 = k16 > 0x80u ? k16 - 1u : 0x7fu;                       // ... then strictly below; 0x7f is -inf
    if (k16 == 0x7fffu) k16 = 0x7ffeu;                           // -0 shares +0's key: step past it
    const uint32_t b16 = (k16 & 0x8000u) ? (k16 & 0x7fffu) : (~k16 & 0xffffu);
    return ((uint32_t)bin << 16) | b16;
}

// One warp: raise thr_bin to the bin scan_boundary finds.  Counts that other warps are still adding
// can only be missed, never invented, so the result is always a valid lower bound.
__device__ __forceinline__ void raise_threshold(SparsifyShared* sh, int k) {
    uint32_t above;
    const int found = scan_boundary(smem_u32(sh) + kHistOff, smem_u32(sh) + kCoarseOff, k, &above);
    if ((threadIdx.x & 31) == 0) {
        const int cur = *(volatile int*)&sh->thr_bin;
        if (found > cur) {
            const float z0 = sh->z0;
            atomicMax(&sh->thr_bin, found);
            atomicMax(&sh->thr_word, threshold_word(found, z0));
            atomicMax(&sh->thr_edge_key, float_to_key(raw_edge_below(found, z0)));
        }
        // what is counted above the boundary bin starts the count towards the next rise (a stale
        // value only costs or delays a rescan)
        if (found >= cur) *(volatile int*)&sh->n_above = (int)above;
    }
}

// The running threshold in the form the lane-tile test wants: a raw-domain bound that lets through
// every logit whose relative bin is >= thr_bin (and a few more, see raw_edge_below).
//   fp32 rows: the bound itself, compared as floats.
//   bf16 rows: P = the largest bf16 value below the bound, in both halves of a word; a packed
//              word w holds a candidate iff max.bf16x2(w, P) != P (NaN halves never differ).
template <typename T> struct Threshold;
template <> struct Threshold<float> {
    int bin;
    float edge;
    __device__ __forceinline__ explicit Threshold(const SparsifyShared* sh)
        : bin(*(const volatile int*)&sh->thr_bin), edge(key_to_float(*(const volatile uint32_t*)&sh->thr_edge_key)) {}
    __device__ __forceinline__ int bin_value() const { return bin; }
};
template <> struct Threshold<bf16_t> {
    uint32_t word, P2;
    __device__ __forceinline__ explicit Threshold(const SparsifyShared* sh) {
        word = *(const volatile uint32_t*)&sh->thr_word;
        P2 = __byte_perm(word, 0u, 0x1010);
    }
    __device__ __forceinline__ int bin_value() const { return (int)(word >> 16); }
};

// Stage the lane tile if it holds a candidate (reduce_max() already called, lm its result): one
// test on the lane's packed maximum, one staging step for all the lanes of the warp that pass.
__device__ __forceinline__ void filter_push(const LaneTile<bf16_t>& lt, const Threshold<bf16_t>& th, float lm, int vec0,
                                            uint32_t base, const SparsifyParams& p) {
    const uint32_t P2 = th.P2;
    if (bf16x2_max(lt.m2, P2) != P2) {
        uint32_t word = (uint32_t)vec0;
#pragma unroll
        for (int j = 0; j < kVecsPerLane; ++j)
            if (bf16x2_max(lt.vm[j], P2) != P2) word |= 1u << (kTileMaskShift + j);
        const bool per_vector = p.k > kCountPerVectorAboveK;
        stage_tile(base, p, th.bin_value(), word, lm, !per_vector);
        if (per_vector) {
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j)
                if ((word >> (kTileMaskShift + j)) & 1u)
                    count_logit(base, th.bin_value(),
                                rel_key(lt.vec_max(j), lds_f32(base + (uint32_t)offsetof(SparsifyShared, z0))));
        }
    }
}
__device__ __forceinline__ void filter_push(const LaneTile<float>& lt, const Threshold<float>& th, float lm, int vec0,
                                            uint32_t base, const SparsifyParams& p) {
    if (lm >= th.edge) {
        uint32_t word = (uint32_t)vec0;
#pragma unroll
        for (int j = 0; j < kVecsPerLane; ++j)
            if (lt.vec_max(j) >= th.edge) word |= 1u << (kTileMaskShift + j);
        const bool per_vector = p.k > kCountPerVectorAboveK;
        stage_tile(base, p, th.bin_value(), word, lm, !per_vector);
        if (per_vector) {
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j)
                if ((word >> (kTileMaskShift + j)) & 1u)
                    count_logit(base, th.bin_value(),
                                rel_key(lt.vec_max(j), lds_f32(base + (uint32_t)offsetof(SparsifyShared, z0))));
        }
    }
}

// One 16-byte vector of a row as kPer logits; the row's ragged last vector element by element,
// -inf beyond the row.
template <typename T>
__device__ __forceinline__ void load_row_vector(const unsigned char* rowp, int vi, const RowExtent& ext, int V,
                                                float (&z)[Elt<T>::kPerVec]) {
    constexpr int kPer = Elt<T>::kPerVec;
    if (vi < ext.nvec_full) {
        unpack_vec<T>(__ldcg(reinterpret_cast<const uint4*>(rowp) + vi), z);
    } else {
#pragma unroll
        for (int e = 0; e < kPer; ++e) z[e] = vi * kPer + e < V ? Elt<T>::load(rowp, vi * kPer + e) : -INFINITY;
    }
}

// All threads: turn the staged lane tiles whose largest logit is in a bin >= bin into (key, index)
// candidates, keeping the logits whose bin is >= bin, and empty the staging buffer.  First the
// marked vectors of the tiles that pass are listed (over the staging buffer itself, its entries
// held in registers meanwhile), then one thread per listed vector reads it back from global
// memory (L2 or HBM), four loads in flight per thread: no load is spent on a tile that fails.
// A full candidate list raises the overflow flag.
constexpr int kMaxStagedTiles = 4096;  // largest vcap
template <typename T>
__device__ __noinline__ void expand_staged(uint2* staged, int vcap, const unsigned char* rowp, const RowExtent ext,
                                           Candidates cb, int cap, int bin, int V, SparsifyShared* sh, int tid) {
    constexpr int kPer = Elt<T>::kPerVec;
    constexpr int kInFlight = 4;
    constexpr int kMine = kMaxStagedTiles / kBlockThreads;
    constexpr uint32_t kVecMask = (1u << kTileMaskShift) - 1u;
    const int nv = min(sh->vec_count, vcap);
    const uint32_t min_key = (uint32_t)bin << kHistShift;
    const float z0 = sh->z0;
    const int lane = tid & 31;
    uint2 mine[kMine];
    int cnt = 0;
#pragma unroll
    for (int c = 0; c < kMine; ++c) {
        const int i = tid + c * kBlockThreads;
        mine[c] = i < nv ? staged[i] : make_uint2(0u, 0u);  // key 0 never passes
        if (mine[c].y >= min_key) cnt += __popc(mine[c].x >> kTileMaskShift);
    }
    if (tid == 0) sh->n_list = 0;
    consumer_sync();  // every entry is in a register: the buffer can take the list
    uint32_t* list = reinterpret_cast<uint32_t*>(staged);
    const int list_cap = 2 * vcap;
    int pos = warp_reserve(&sh->n_list, cnt, lane);
#pragma unroll
    for (int c = 0; c < kMine; ++c) {
        if (mine[c].y >= min_key) {
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                if ((mine[c].x >> (kTileMaskShift + j)) & 1u) {
                    if (pos < list_cap) list[pos] = (mine[c].x & kVecMask) + 32u * j;
                    ++pos;
                }
            }
        }
    }
    consumer_sync();
    int nlist = sh->n_list;
    if (nlist > list_cap) {  // more than two marked vectors per staged tile: take the second pass over the row
        if (tid == 0) sh->overflow = 1;
        nlist = 0;
    }
    for (int base = 0; base < nlist; base += kInFlight * kBlockThreads) {
        uint4 d[kInFlight];
        int vi[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int i = base + u * kBlockThreads + tid;
            vi[u] = i < nlist ? (int)list[i] : -1;
            if (vi[u] >= 0 && vi[u] < ext.nvec_full) d[u] = __ldcg(reinterpret_cast<const uint4*>(rowp) + vi[u]);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            if (vi[u] < 0) continue;
            const int e0 = vi[u] * kPer;
            float z[kPer];
            if (vi[u] < ext.nvec_full) unpack_vec<T>(d[u], z);
            else load_row_vector<T>(rowp, vi[u], ext, V, z);  // the ragged last vector; nothing beyond it
#pragma unroll
            for (int e = 0; e < kPer; ++e) {
                if (z[e] >= -3.4028234e38f) {
                    if (rel_key(z[e], z0) >= min_key) {
                        const int pos2 = atomicAdd(cb.count, 1);
                        if (pos2 < cap) {
                            cb.key[pos2] = float_to_key(z[e]);
                            cb.idx[pos2] = e0 + e;
                        } else {
                            sh->overflow = 1;
                        }
                    }
                }
            }
        }
    }
    consumer_sync();
    if (tid == 0) {
        sh->vec_count = 0;
        if (*cb.count > cap) *cb.count = cap;
    }
    consumer_sync();
}

// All threads: drop the buffer entries whose bin is below `bin` (entries are held in registers
// between the read and the write phase, so the compaction is in place).
__device__ __noinline__ void compact_buffer(Candidates cb, int bin, SparsifyShared* sh, int tid) {
    constexpr int E = 16;  // cap <= 4096 = 16 * 256
    const int n = min(*cb.count, E * kBlockThreads);
    const float z0 = sh->z0;
    uint32_t ek[E];
    int ei[E];
    unsigned keep = 0;
    int cnt = 0;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int i = tid * E + e;
        ek[e] = 0u;
        ei[e] = 0;
        if (i < n) {
            ek[e] = cb.key[i];
            ei[e] = cb.idx[i];
            if ((int)(rel_key(key_to_float(ek[e]), z0) >> kHistShift) >= bin) {
                keep |= 1u << e;
                ++cnt;
            }
        }
    }
    const int lane = tid & 31, warp = tid >> 5;
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) sh->warp_tot[warp] = incl;
    consumer_sync();  // every entry has been read, warp totals are in place
    int off = incl - cnt, total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const int t = sh->warp_tot[w];
        if (w < warp) off += t;
        total += t;
    }
#pragma unroll
    for (int e = 0; e < E; ++e)
        if (keep & (1u << e)) {
            cb.key[off] = ek[e];
            cb.idx[off] = ei[e];
            ++off;
        }
    consumer_sync();
    if (tid == 0) *cb.count = total;
    consumer_sync();
}

template <typename T>
__device__ __noinline__ void finalize_row(const SparsifyParams& p, int row, Candidates cb, SparsifyShared* sh,
                                          unsigned char* arena, double Mrow, double Srow, int tid);

// All threads: second pass over a segment whose buffers overflowed.  The histogram went on counting,
// so the final threshold is as tight as ever: read the segment again and append every logit whose
// bin is >= bin straight to the (emptied) candidate list.  A list that fills up again (a huge tie)
// leaves the overflow flag set for the radix select.
template <typename T>
__device__ __noinline__ void recollect_from_global(const unsigned char* rowp, int chunk_begin, int chunk_end, int bin,
                                                   const RowExtent ext, Candidates cb, int cap, SparsifyShared* sh,
                                                   int tid) {
    constexpr int kPer = Elt<T>::kPerVec;
    const int lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        *cb.count = 0;
        sh->overflow = 0;
    }
    consumer_sync();
    const float z0 = sh->z0;
    const float edge = raw_edge_below(bin, z0);  // for the tile and vector tests; a logit is judged by its relative key
    const uint32_t min_key = (uint32_t)bin << kHistShift;
    for (int ch = chunk_begin + warp; ch < chunk_end; ch += kWarps) {
        LaneTile<T> lt;
        lt.load(rowp, ch * kVecsPerChunk, lane, ext);
        if (lt.reduce_max() >= edge) {
#pragma unroll 1
            for (int j = 0; j < kVecsPerLane; ++j) {
                if (!(lt.vec_max(j) >= edge)) continue;
#pragma unroll
                for (int e = 0; e < kPer; ++e) {
                    const float z = lt.elem(j, e);
                    if (z >= -3.4028234e38f && rel_key(z, z0) >= min_key) {
                        const int pos = atomicAdd(cb.count, 1);
                        if (pos < cap) {
                            cb.key[pos] = float_to_key(z);
                            cb.idx[pos] = (ch * kVecsPerChunk + j * 32 + lane) * kPer + e;
                        } else {
                            sh->overflow = 1;
                        }
                    }
                }
            }
        }
    }
    consumer_sync();
    if (tid == 0 && *cb.count > cap) *cb.count = cap;
    consumer_sync();
}

// Radix-select fallbacks, out of line (one copy each).
template <typename T>
__device__ __noinline__ void reselect_from_global(const unsigned char* rowp, int e0, int n, int k, int idx_hi_byte,
                                                  Candidates cb, SparsifyShared* sh, int tid) {
    uint32_t kth;
    GlobalSrc<T> src{rowp, e0};
    select_topk<(Elt<T>::kBytes == 2)>(src, n, k, idx_hi_byte, cb, &sh->sel, tid, &kth);
}
template <bool kKeyHiOnly>
__device__ __noinline__ void reselect_from_buffer(int n, int k, int idx_hi_byte, Candidates cb, SparsifyShared* sh,
                                                  int tid) {
    uint32_t kth;
    BufferSrc src{cb.key, cb.idx};
    select_topk<kKeyHiOnly>(src, n, k, idx_hi_byte, cb, &sh->sel, tid, &kth);
}

// All threads: bring every segment's candidates and statistics of a row into the candidate list.
__device__ __forceinline__ void gather_segments(const SparsifyParams& p, int row, int nseg, Candidates cb,
                                                SparsifyShared* sh, int tid, double* Mrow, double* Srow) {
    const size_t slot0 = (size_t)row * nseg;
    if (nseg == 1 && p.seg_cap <= 8 * kBlockThreads) {
        // one segment: every load is issued before anything is used, so the row costs one trip to memory
        const SegStat* st = &p.seg_stats[slot0];
        const uint2* ent = p.seg_entries + slot0 * (size_t)p.seg_stride;
        uint2 e[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = tid + j * kBlockThreads;
            e[j] = i < p.seg_cap ? __ldcg(&ent[i]) : make_uint2(0u, 0u);
        }
        const int n = __ldcg(&st->n);
        // fp64 is scarce (two warp instructions per clock per SM): one warp combines the eight
        // per-warp pairs, one pair per lane, and leaves (M, S) in shared memory for the others
        if (tid < 32) {
            const double Sw = tid < kWarps ? __ldcg(&st->S[tid]) : 0.0;
            const double Mw = tid < kWarps ? (double)__ldcg(&st->M[tid]) : -INFINITY;
            const double Mall = warp_max(Sw > 0.0 ? Mw : -INFINITY);
            const double Sall = warp_sum(Sw > 0.0 ? Sw * exp2(Mw - Mall) : 0.0);
            if (tid == 0) {
                sh->scratch[0] = Mall;
                sh->scratch[1] = Sall;
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = tid + j * kBlockThreads;
            if (i < n) {
                cb.key[i] = e[j].x;
                cb.idx[i] = (int)e[j].y;
            }
        }
        if (tid == 0) sh->cand_count = n;
        consumer_sync();
        *Mrow = sh->scratch[0];
        *Srow = sh->scratch[1];
        consumer_sync();
        return;
    }
    if (tid == 0) sh->cand_count = 0;
    consumer_sync();
    if (tid < 32) {  // one warp combines the nseg * 8 per-warp pairs (fp64 is scarce)
        double Mall = -INFINITY;
        for (int i = tid; i < nseg * kWarps; i += 32) {
            const SegStat* st = &p.seg_stats[slot0 + i / kWarps];
            if (__ldcg(&st->S[i % kWarps]) > 0.0) Mall = fmax(Mall, (double)__ldcg(&st->M[i % kWarps]));
        }
        Mall = warp_max(Mall);
        double Sall = 0.0;
        for (int i = tid; i < nseg * kWarps; i += 32) {
            const SegStat* st = &p.seg_stats[slot0 + i / kWarps];
            const double Sw = __ldcg(&st->S[i % kWarps]);
            if (Sw > 0.0) Sall += Sw * exp2((double)__ldcg(&st->M[i % kWarps]) - Mall);
        }
        Sall = warp_sum(Sall);
        if (tid == 0) {
            sh->scratch[0] = Mall;
            sh->scratch[1] = Sall;
        }
    }
    for (int g = 0; g < nseg; ++g) {
        const SegStat* st = &p.seg_stats[slot0 + g];
        const int ng = __ldcg(&st->n);
        const uint2* ent = p.seg_entries + (slot0 + g) * (size_t)p.seg_stride;
        const int base = sh->cand_count;
        for (int i = tid; i < ng; i += kBlockThreads) {
            const uint2 e2 = __ldcg(&ent[i]);
            cb.key[base + i] = e2.x;
            cb.idx[base + i] = (int)e2.y;
        }
        consumer_sync();
        if (tid == 0) sh->cand_count = base + ng;
        consumer_sync();
    }
    *Mrow = sh->scratch[0];
    *Srow = sh->scratch[1];
    consumer_sync();
}

// First launch: every segment streams, hands its candidates and statistics over and ends; the
// rows are finished by sparsify_finish_kernel, launched next on the stream.
template <typename T>
__global__ void __launch_bounds__(kBlockThreads, kSparsifyCtasPerSm) sparsify_kernel(const SparsifyParams p) {
    constexpr bool kHiOnly = (Elt<T>::kBytes == 2);
    constexpr int kPer = Elt<T>::kPerVec;
    constexpr int kChunkElems = kChunkBytes / Elt<T>::kBytes;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // every pointer below is derived from smem_raw by plain offsets, so that the compiler keeps
    // them in the shared address space (shared-memory atomics and loads, not generic ones)
    SparsifyShared* sh = reinterpret_cast<SparsifyShared*>(smem_raw);
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw + kHistOff);
    uint2* staged = reinterpret_cast<uint2*>(smem_raw + kStagedOff);
    uint32_t* cand_key = reinterpret_cast<uint32_t*>(staged + p.vcap);
    int* cand_idx = reinterpret_cast<int*>(cand_key + p.cap);
    uint32_t* tmp_key = reinterpret_cast<uint32_t*>(cand_idx + p.cap);
    int* tmp_idx = reinterpret_cast<int*>(tmp_key + p.k);
    const uint32_t base = smem_u32(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const RowWork wk = locate_work(p.split, blockIdx.x, p.nchunks);
    const int row = wk.row, chunk_begin = wk.chunk_begin, chunk_end = wk.chunk_end;
    const unsigned char* rowp = p.logits + (long long)row * p.row_stride_bytes;
    const RowExtent ext = row_extent<T>(p.V);
    const int k = p.k;
    const float c = p.c.f;

    // the first chunk's loads go out before anything else: their latency covers the set-up below
    const int ch0 = chunk_begin + warp;
    LaneTile<T> first;
    if (ch0 < chunk_end) first.load(rowp, ch0 * kVecsPerChunk, lane, ext);
    static_assert((kHistBins + kCoarseBins) % 4 == 0, "the histograms are cleared 16 bytes at a time");
    uint4* hist4 = reinterpret_cast<uint4*>(hist);
    for (int i = tid; i < (kHistBins + kCoarseBins) / 4; i += kBlockThreads) hist4[i] = make_uint4(0u, 0u, 0u, 0u);
    if (tid == 0) {
        sh->thr_bin = kLowestFiniteBin;
        sh->thr_word = threshold_word(kLowestFiniteBin, 0.f);  // P = -inf: every finite logit passes
        sh->thr_edge_key = float_to_key(-3.4028234e38f);
        sh->cand_count = 0;
        sh->vec_count = 0;
        sh->overflow = 0;
        sh->trim_request = 0;
        sh->n_above = 0;
        // The row's ready flag is cleared here, by the CTA that will set it, and the store is fenced
        // before the barrier after which the first thread of this CTA lets the finish kernel be
        // scheduled.  A finish CTA runs only after every streaming CTA has passed that point, so it
        // never sees a flag left by an earlier call, and the workspace needs no clearing between calls.
        if (p.row_ready) {
            *(volatile int*)&p.row_ready[row] = 0;
            __threadfence();
        }
    }
    // the segment's offset for the histogram's bins: the largest logit of its first chunks (see rel_key)
    float first_max = -INFINITY;
    if (ch0 < chunk_end) first_max = first.reduce_max();
    first_max = warp_max(first_max);
    if (lane == 0) sh->scratch[warp] = (double)first_max;
    __syncthreads();
    allow_dependent_launch();
    float z0 = (float)sh->scratch[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) z0 = fmaxf(z0, (float)sh->scratch[w]);
    if (!(z0 >= -3.4028234e38f && z0 <= 3.4028234e38f)) z0 = 0.f;  // nothing finite there: no offset
    if (tid == 0) sh->z0 = z0;  // read by others only after the barriers below
    Candidates cb{cand_key, cand_idx, tmp_key, tmp_idx, &sh->cand_count};

    // ---- first threshold, from the segment's first chunks (one per warp) ---------------------------
    // For k <= 256 the histogram takes only the maxima of the 1024 16-byte vectors of these chunks:
    // the k-th largest of them is a lower bound on the k-th largest logit, and close to it while k
    // is small against 1024.  Larger k counts every logit of the chunks.  The counts are wiped
    // afterwards: the streaming loop below starts again at the first chunk (an L2 hit) and counts
    // what it pushes.
    {
        if (ch0 < chunk_end) {
            LaneTile<T>& lt = first;  // (reduce_max() already called)
            if (k <= 256) {
#pragma unroll
                for (int j = 0; j < kVecsPerLane; ++j) {
                    const float z = lt.vec_max(j);
                    if (z >= -3.4028234e38f) hist_count(base + kHistOff, base + kCoarseOff, (int)(rel_key(z, z0) >> kHistShift), 1u);
                }
            } else {
#pragma unroll 4
                for (int e = 0; e < kVecsPerLane * kPer; ++e) {
                    const float z = lt.elem(e / kPer, e % kPer);
                    if (z >= -3.4028234e38f) hist_count(base + kHistOff, base + kCoarseOff, (int)(rel_key(z, z0) >> kHistShift), 1u);
                }
            }
        }
        __syncthreads();
        if (warp == 0) raise_threshold(sh, k);
        __syncthreads();
        for (int i = tid; i < (kHistBins + kCoarseBins) / 4; i += kBlockThreads) hist4[i] = make_uint4(0u, 0u, 0u, 0u);
        if (tid == 0) sh->n_above = 0;
        __syncthreads();
    }

    // ---- streaming: no barriers; warp w rescans the histogram on its turn --------------------------
    LaneSum ls;
    ls.reset();
    // chunks below pf_end are whole and inside the segment: the only ones asked of L2 ahead of time
    const int pf_end = min(chunk_end, ext.nvec_full / kVecsPerChunk);
    const unsigned char* lane_rowp = rowp + lane * kVecBytes;  // the loop's loads need no lane number
    int ch = chunk_begin + warp;
    for (;;) {
        while (ch < chunk_end) {
            __syncwarp();
            if (__shfl_sync(0xffffffffu, *(volatile int*)&sh->trim_request, 0)) break;
            LaneTile<T> lt;
            lt.load_lane(lane_rowp, ch * kVecsPerChunk, ext);
            if (ch + kPrefetchSteps * kWarps < pf_end && lane == 0)
                prefetch_l2(rowp + (size_t)(ch + kPrefetchSteps * kWarps) * kChunkBytes, kChunkBytes);
            const float lm = lt.reduce_max();
            const Threshold<T> th(sh);
            filter_push(lt, th, lm, ch * kVecsPerChunk + lane, base, p);  // while the vector maxima are at hand
            ls.raise_to(lm, c);
            lt.accumulate(ls, c);
            // The warps take turns at looking whether enough has been counted above the threshold
            // bin for it to rise (ch mod 8 is the warp's own, so the turns differ), and rescan then.
            if ((((ch >> 3) ^ ch) & (kWarps - 1)) == 0) {
                __syncwarp();
                if (__shfl_sync(0xffffffffu, *(volatile int*)&sh->n_above, 0) >= k) raise_threshold(sh, k);
            }
            ch += kWarps;
        }
        const int all_done = __syncthreads_and(ch >= chunk_end);
        const int want_trim = sh->trim_request;
        __syncthreads();
        if (all_done) break;
        if (want_trim) {
            if (!sh->overflow) {
                if (warp == 0) raise_threshold(sh, k);
                consumer_sync();
                const int bin = sh->thr_bin;
                expand_staged<T>(staged, p.vcap, rowp, ext, cb, p.cap, bin, p.V, sh, tid);
                if (sh->cand_count > p.high) compact_buffer(cb, bin, sh, tid);
            }
            if (tid == 0) sh->trim_request = 0;
            __syncthreads();
        }
    }

    // ---- hand-over: one (M, S) pair per warp and the segment's entries; the kernel boundary publishes
    // them to the finish kernel
    const float Mw = warp_max(ls.M);
    const double Sw = warp_sum(ls.total_f64() * exp2((double)ls.M - (double)Mw));
    const size_t slot = (size_t)row * wk.nseg + wk.seg;
    uint2* my_entries = p.seg_entries + slot * (size_t)p.seg_stride;
    SegStat* st = &p.seg_stats[slot];
    if (lane == 0) {
        st->S[warp] = Sw;
        st->M[warp] = Mw;
    }
    // (the loop's last barrier ordered every write of the flags read here)
    if (p.raw_cap > 0 && !sh->overflow && sh->cand_count == 0) {
        // The staging buffer never filled: its tiles go over as they are, with the final threshold
        // bin, and the finish kernel reads the few that still pass back from global memory, all
        // rows at once, instead of this CTA waiting on them now.
        const int n = sh->vec_count;
        for (int i = tid; i < n; i += kBlockThreads) my_entries[i] = staged[i];
        if (tid == 0) {
            st->n = n;
            st->raw_bin = sh->thr_bin;
            st->z0 = sh->z0;
        }
        __syncthreads();  // every thread's part of the hand-over is written
        if (tid == 0 && p.row_ready) publish_row_ready(&p.row_ready[row]);
        return;
    }

    // ---- what is still staged becomes candidates; a buffer that overflowed is rebuilt from global memory
    if (!sh->overflow) expand_staged<T>(staged, p.vcap, rowp, ext, cb, p.cap, sh->thr_bin, p.V, sh, tid);
    if (sh->overflow) {
        if (warp == 0) raise_threshold(sh, k);
        consumer_sync();
        recollect_from_global<T>(rowp, chunk_begin, chunk_end, sh->thr_bin, ext, cb, p.cap, sh, tid);
    }
    if (sh->overflow) {
        const int e0 = chunk_begin * kChunkElems;
        const int n = min(p.V, chunk_end * kChunkElems) - e0;
        reselect_from_global<T>(rowp, e0, n, k, p.idx_hi_byte, cb, sh, tid);
        if (tid == 0) sh->overflow = 0;
        consumer_sync();
    }
    // candidates: all at or above this segment's final threshold
    int n = sh->cand_count;
    if (n > p.seg_cap) {  // earlier expansions used looser thresholds: keep what the final one admits
        compact_buffer(cb, sh->thr_bin, sh, tid);
        n = sh->cand_count;
    }
    if (n > p.seg_cap) {  // heavy ties at the boundary: hand over the exact k
        reselect_from_buffer<kHiOnly>(n, k, p.idx_hi_byte, cb, sh, tid);
        n = sh->cand_count;
    }
    for (int i = tid; i < n; i += kBlockThreads) my_entries[i] = make_uint2(cand_key[i], (uint32_t)cand_idx[i]);
    if (tid == 0) {
        st->n = n;
        st->raw_bin = -1;
    }
    __syncthreads();  // every thread's part of the hand-over is written
    if (tid == 0 && p.row_ready) publish_row_ready(&p.row_ready[row]);
}

// Second launch: one CTA per row merges the row's segments and finishes it.
// Same shared-memory carve-up as the streaming kernel, with no staging buffer (vcap = 0).
template <typename T>
__global__ void __launch_bounds__(kBlockThreads, 6) sparsify_finish_kernel(const SparsifyParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    SparsifyShared* sh = reinterpret_cast<SparsifyShared*>(smem_raw);
    unsigned char* arena = smem_raw + kHistOff;
    uint32_t* cand_key = reinterpret_cast<uint32_t*>(smem_raw + kStagedOff);
    int* cand_idx = reinterpret_cast<int*>(cand_key + p.fin_cap);
    uint32_t* tmp_key = reinterpret_cast<uint32_t*>(cand_idx + p.fin_cap);
    int* tmp_idx = reinterpret_cast<int*>(tmp_key + p.k);
    const int tid = threadIdx.x, row = blockIdx.x;
    // the uniforms are needed last: ask for their cache line now
    if (tid == 0 && p.num_samples > 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.uniforms + (size_t)row * p.num_samples));
    if (tid == 0) sh->overflow = 0;
    // Nothing the streaming kernel wrote is read before this point.  A row of one segment goes on
    // as soon as its own ready flag is set (see poll_row_ready); rows cut into segments, and a
    // flag that does not come, wait for the end of the streaming kernel.
    if (p.row_ready) {
        if (tid == 0) sh->n_list = poll_row_ready(&p.row_ready[row]) ? 1 : 0;
        __syncthreads();
        if (!sh->n_list) wait_for_primary_kernel();
        __syncthreads();
    } else {
        wait_for_primary_kernel();
    }
    if (row == 0 && tid == 0) *p.status = 0;
    Candidates cb{cand_key, cand_idx, tmp_key, tmp_idx, &sh->cand_count};
    double Mrow, Srow;
    gather_segments(p, row, p.split.nseg, cb, sh, tid, &Mrow, &Srow);
    finalize_row<T>(p, row, cb, sh, arena, Mrow, Srow, tid);
    // this kernel's completion must imply the streaming kernel's: one CTA sees to that
    if (row == 0 && p.row_ready) wait_for_primary_kernel();
}

// Position of entry (key, idx) of the buffer in the order (key descending, idx ascending) /
// (idx ascending), by counting the entries that precede it.
__device__ __forceinline__ int rank_by_key(const uint32_t* key, const int* idx, int n, uint32_t my_key, int my_idx) {
    int r = 0;
    for (int j = 0; j < n; ++j) {
        const uint32_t kj = key[j];
        const int ij = idx[j];
        r += (kj > my_key || (kj == my_key && ij < my_idx)) ? 1 : 0;
    }
    return r;
}
__device__ __forceinline__ int rank_by_idx(const int* idx, int n, int my_idx) {
    int r = 0;
    for (int j = 0; j < n; ++j) r += idx[j] < my_idx ? 1 : 0;
    return r;
}

// Exact top-k of the row, nucleus cut, renormalisation, sampling and the ascending-index payload.
template <typename T>
__device__ __noinline__ void finalize_row(const SparsifyParams& p, int row, Candidates cb, SparsifyShared* sh,
                                          unsigned char* arena, double Mrow, double Srow, int tid) {
    constexpr bool kHiOnly = (Elt<T>::kBytes == 2);
    const int k = p.k;
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t* cand_key = cb.key;
    int* cand_idx = cb.idx;
    uint32_t* hist = reinterpret_cast<uint32_t*>(arena);
    uint2* bnd = reinterpret_cast<uint2*>(arena + (kHistBins + kCoarseBins) * 4);
    const int nc = sh->cand_count;

    // ---- the bin of the k-th largest logit ------------------------------------------------------
    // exact counts of the candidates (the streaming histogram only counted vector maxima)
    for (int i = tid; i < kHistBins + kCoarseBins; i += kBlockThreads) hist[i] = 0u;
    consumer_sync();
    for (int i = tid; i < nc; i += kBlockThreads)
        hist_count(smem_u32(sh) + kHistOff, smem_u32(sh) + kCoarseOff, (int)(cand_key[i] >> kHistShift), 1u);
    consumer_sync();
    if (warp == 0) {
        uint32_t above;
        const int b = scan_boundary(smem_u32(sh) + kHistOff, smem_u32(sh) + kCoarseOff, k, &above);
        if (lane == 0) {
            sh->sel_bin = b;  // -1: fewer than k candidates exist, all of them are kept
            sh->sel_above = (int)above;
            sh->n_win = 0;
            sh->n_bnd = 0;
        }
    }
    consumer_sync();
    const int sel_bin = sh->sel_bin;
    // ---- everything above that bin is in; the bin itself goes to the boundary list ---------------
    for (int i = tid; i < nc; i += kBlockThreads) {
        const uint32_t kk = cand_key[i];
        const int bin = (int)(kk >> kHistShift);
        if (bin > sel_bin) {
            const int pos = atomicAdd(&sh->n_win, 1);
            if (pos < k) {
                cb.tmp_key[pos] = kk;
                cb.tmp_idx[pos] = cand_idx[i];
            }
        } else if (bin == sel_bin) {
            const int pos = atomicAdd(&sh->n_bnd, 1);
            if (pos < kBoundaryCap) bnd[pos] = make_uint2(kk, (uint32_t)cand_idx[i]);
        }
    }
    consumer_sync();
    const int n_above = min(sh->n_win, k), nb = sh->n_bnd;
    int n0;
    if (nb > kBoundaryCap) {
        // heavy ties: radix select over the whole buffer (leaves its winners at the front of the buffer)
        reselect_from_buffer<kHiOnly>(nc, k, p.idx_hi_byte, cb, sh, tid);
        n0 = min(sh->cand_count, k);
    } else {
        const int need = min(k - n_above, nb);
        for (int t = tid; t < nb; t += kBlockThreads) {
            const uint2 me = bnd[t];
            int r = t;
            if (nb > need) {
                r = 0;
                for (int j = 0; j < nb; ++j) {
                    const uint2 o = bnd[j];
                    r += (o.x > me.x || (o.x == me.x && (int)o.y < (int)me.y)) ? 1 : 0;
                }
            }
            if (r < need) {
                cb.tmp_key[n_above + r] = me.x;
                cb.tmp_idx[n_above + r] = (int)me.y;
            }
        }
        consumer_sync();
        n0 = n_above + need;
        for (int i = tid; i < n0; i += kBlockThreads) {
            cand_key[i] = cb.tmp_key[i];
            cand_idx[i] = cb.tmp_idx[i];
        }
        consumer_sync();
    }

    if (tid == 0) sh->scratch[2] = Mrow + log2(Srow);  // base-2 log of the softmax normaliser (once: fp64 is scarce)
    consumer_sync();
    const double L2 = sh->scratch[2];
    const double cd = p.c.d;
    // the histogram and the boundary list are no longer needed: their arena holds the fp64 work arrays
    unsigned long long* comp = reinterpret_cast<unsigned long long*>(arena);          // 1024 * 8
    double* wv = reinterpret_cast<double*>(arena + 8192);                             // 1024 * 8
    double* cum = reinterpret_cast<double*>(arena + 16384);                           // 1024 * 8
    int n = n0;
    double mass = 0.0;
    if (n0 > 0 && p.top_p < 1.0f) {
        // order the candidates by (logit descending, index ascending) and cut at the nucleus
        if (n0 <= kRankSortMax) {
            if (tid < n0) {
                const uint32_t kk = cand_key[tid];
                const int ii = cand_idx[tid];
                const int r = rank_by_key(cand_key, cand_idx, n0, kk, ii);
                comp[r] = ((unsigned long long)kk << 32) | (unsigned long long)(0xffffffffu - (uint32_t)ii);
            }
            consumer_sync();
        } else {
            const int P = next_pow2(n0);
            for (int i = tid; i < P; i += kBlockThreads)
                comp[i] = i < n0 ? (((unsigned long long)cand_key[i] << 32) | (unsigned long long)(0xffffffffu - (uint32_t)cand_idx[i])) : 0ull;
            consumer_sync();
            bitonic_sort<true>(comp, P, tid);
        }
        for (int i = tid; i < n0; i += kBlockThreads) {
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
        for (int i = tid; i < n; i += kBlockThreads) {
            cand_key[i] = (uint32_t)(comp[i] >> 32);
            cand_idx[i] = (int)(0xffffffffu - (uint32_t)(comp[i] & 0xffffffffull));
        }
        consumer_sync();
    }
    // ascending index order
    if (n > 0) {
        if (n <= kRankSortMax) {
            if (tid < n) {
                const int ii = cand_idx[tid];
                comp[rank_by_idx(cand_idx, n, ii)] = ((unsigned long long)(uint32_t)ii << 32) | (unsigned long long)cand_key[tid];
            }
            consumer_sync();
        } else {
            const int P = next_pow2(n);
            for (int i = tid; i < P; i += kBlockThreads)
                comp[i] = i < n ? (((unsigned long long)(uint32_t)cand_idx[i] << 32) | (unsigned long long)cand_key[i]) : ~0ull;
            consumer_sync();
            bitonic_sort<false>(comp, P, tid);
        }
    }
    // renormalised truncated distribution in fp64: w_i = 2^(y_i - m_S), CDF by inclusive scan
    double my_max = -INFINITY;
    for (int i = tid; i < n; i += kBlockThreads) {
        const float z = key_to_float((uint32_t)(comp[i] & 0xffffffffull));
        const double y = (double)z * cd;
        wv[i] = y;
        my_max = fmax(my_max, y);
    }
    const double mS = block_max(my_max, tid, sh->scratch);
    double my_mass = 0.0;
    for (int i = tid; i < n; i += kBlockThreads) {
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
    for (int i = tid; i < k; i += kBlockThreads) {
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
    for (int sidx = tid; sidx < p.num_samples; sidx += kBlockThreads) {
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

// ---- finish kernel for small k --------------------------------------------------------------------
// Rows of one segment with k <= 256 are finished by a CTA of 64, 96, 128 or 256 threads (at least
// k) with 6 to 21 KB of shared memory, so that every row of a large batch is resident at once:
// finishing a row is a chain of dependent steps (trips to memory, rank counting, two scans), and
// what it costs machine-wide is the length of that chain times the number of waves.
constexpr int kSmallMaxThreads = 256;  // and so the largest k of this kernel
// candidates a row may bring as (key, index) entries: 2 k at most (seg_cap)
__host__ __device__ constexpr int small_cand_cap(int nt) { return nt > 128 ? 512 : 256; }
// Candidates the kernel may make from a row's staged tiles: 256, and 512 for k above 96, where
// 256 is only 2 k and the threshold bin's share can exceed it on ordinary rows.  (512 everywhere
// cost the 64-thread kernel 9 us on 2048 rows of 256 000 logits: fewer finish CTAs fit beside the streaming
// CTAs of the last wave.)
__host__ __device__ constexpr int small_list_cap(int nt) { return nt > 128 ? 1024 : nt > 96 ? 512 : 256; }
// marked vectors in the staged tiles of a row that pass its final threshold
__host__ __device__ constexpr int small_pass_cap(int nt) { return nt > 128 ? 1024 : 512; }

template <int kList, int kK, int kPass> struct SmallShared {
    unsigned long long comp[kList];  // candidates as key << 32 | ~index: larger is earlier in the top-k order
    uint32_t wkey[kK];  // winners in (key descending, index ascending) order, then in ascending index
    int widx[kK];
    uint32_t okey[kK];
    int oidx[kK];
    double cum[kK];
    double wv[kK];
    double red[8];   // one slot per warp for the block scans
    double lrow;     // the row's log2-normaliser
    int n_cut;
    // rows handed over as staged lane tiles
    uint32_t pass[kPass];  // marked vectors of the tiles whose largest logit passes the final threshold
    int n_pass, n_cand;
    unsigned long long best[kSmallMaxThreads / 32];
};
template <int NT> using SmallSharedFor = SmallShared<small_list_cap(NT), NT, small_pass_cap(NT)>;

template <int NT> __device__ __forceinline__ void small_sync() { asm volatile("bar.sync 2, %0;" ::"n"(NT) : "memory"); }

// inclusive scan of one value per thread over the NT threads; returns this thread's inclusive sum
template <int NT> __device__ __forceinline__ double small_scan(double v, int tid, double* red, double* total) {
    const int lane = tid & 31, warp = tid >> 5;
    double incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) red[warp] = incl;
    small_sync<NT>();
    double base = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) {
        const double t = red[w];
        if (w < warp) base += t;
        tot += t;
    }
    small_sync<NT>();
    *total = tot;
    return base + incl;
}
template <int NT> __device__ __forceinline__ double small_max(double v, int tid, double* red) {
    v = warp_max(v);
    if ((tid & 31) == 0) red[tid >> 5] = v;
    small_sync<NT>();
    double m = red[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) m = fmax(m, red[w]);
    small_sync<NT>();
    return m;
}

// The slow way to a row's k winners from its staged tiles: one winner per round, each round a pass
// over the marked vectors of the passing tiles (the kernel's list of them if it held them all).
// Only there to be correct when a row has more tied candidates around its k-th logit than the
// lists of the kernel below hold.
// composite = key << 32 | ~index: larger is earlier in (logit descending, index ascending)
template <typename T, int NT>
__device__ __noinline__ int winners_one_by_one(const SparsifyParams& p, int row, const uint2* ent, int n_tiles, int bin,
                                               float z0, int n_listed, SmallSharedFor<NT>* sm, int tid) {
    constexpr int kPer = Elt<T>::kPerVec;
    constexpr uint32_t kVecMask = (1u << kTileMaskShift) - 1u;
    const unsigned char* rowp = p.logits + (long long)row * p.row_stride_bytes;
    const RowExtent ext = row_extent<T>(p.V);
    const uint32_t min_key = (uint32_t)bin << kHistShift;
    unsigned long long last = ~0ull;
    int found = 0;
    for (; found < p.k; ++found) {
        unsigned long long best = 0ull;
        // the vectors to look at: those listed in sm->pass (n_listed >= 0), else every marked vector
        // of every passing tile of the hand-over
        const int n_items = n_listed >= 0 ? n_listed : n_tiles * kVecsPerLane;
        for (int i = tid; i < n_items; i += NT) {
            int vi;
            if (n_listed >= 0) {
                vi = (int)sm->pass[i];
            } else {
                const uint2 e = __ldcg(&ent[i / kVecsPerLane]);
                const int j = i % kVecsPerLane;
                if (e.y < min_key || !((e.x >> (kTileMaskShift + j)) & 1u)) continue;
                vi = (int)(e.x & kVecMask) + 32 * j;
            }
            float z[kPer];
            load_row_vector<T>(rowp, vi, ext, p.V, z);
#pragma unroll
            for (int q = 0; q < kPer; ++q) {
                if (z[q] >= -3.4028234e38f && rel_key(z[q], z0) >= min_key) {
                    const unsigned long long comp = ((unsigned long long)float_to_key(z[q]) << 32) |
                                                    (unsigned long long)(0xffffffffu - (uint32_t)(vi * kPer + q));
                    if (comp < last && comp > best) best = comp;
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long t = __shfl_xor_sync(0xffffffffu, best, o);
            best = t > best ? t : best;
        }
        if ((tid & 31) == 0) sm->best[tid >> 5] = best;
        small_sync<NT>();
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) best = sm->best[w] > best ? sm->best[w] : best;
        small_sync<NT>();
        if (best == 0ull) break;
        if (tid == 0) sm->comp[found] = best;
        last = best;
    }
    small_sync<NT>();
    return found;
}

// NT threads: the row was handed over as n_tiles staged lane tiles and its final threshold bin.
// Puts the row's candidates (every logit whose bin is >= bin, at least its k largest) into
// sm->comp and returns their number (<= small_list_cap(NT)).  The marked vectors of the tiles that pass
// (largest logit in a bin >= bin) are listed, then one thread per listed vector reads it back and
// appends its candidates.  (Inlined into the kernel so that the compiler sees sm in the shared
// address space: atomics through a generic pointer to shared memory are several times slower.)
template <typename T, int NT>
__device__ __forceinline__ int candidates_from_tiles(const SparsifyParams& p, int row, const uint2* ent, int n_tiles, int bin,
                                                     float z0, SmallSharedFor<NT>* sm, int tid) {
    constexpr int kPer = Elt<T>::kPerVec;
    constexpr uint32_t kVecMask = (1u << kTileMaskShift) - 1u;
    const unsigned char* rowp = p.logits + (long long)row * p.row_stride_bytes;
    const RowExtent ext = row_extent<T>(p.V);
    const uint32_t min_key = (uint32_t)bin << kHistShift;
    const int lane = tid & 31;
    if (tid == 0) {
        sm->n_pass = 0;
        sm->n_cand = 0;
    }
    small_sync<NT>();
    // ---- the marked vectors of the passing tiles, as a list ------------------------------------------
    for (int base = 0; base < n_tiles; base += 8 * NT) {
        uint32_t m = 0;  // which of this thread's eight entries pass
        int cnt = 0;     // marked vectors in them
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = base + u * NT + tid;
            const uint2 e = i < n_tiles ? __ldcg(&ent[i]) : make_uint2(0u, 0u);  // key 0 never passes
            if (e.y >= min_key) {
                m |= 1u << u;
                cnt += __popc(e.x >> kTileMaskShift);
            }
        }
        int pos = warp_reserve(&sm->n_pass, cnt, lane);
        while (m) {  // few: read them again (cached) rather than keep eight entries in registers
            const int u = __ffs(m) - 1;
            m &= m - 1;
            const uint32_t w = __ldcg(&ent[base + u * NT + tid].x);
#pragma unroll
            for (int j = 0; j < kVecsPerLane; ++j) {
                if ((w >> (kTileMaskShift + j)) & 1u) {
                    if (pos < small_pass_cap(NT)) sm->pass[pos] = (w & kVecMask) + 32u * j;
                    ++pos;
                }
            }
        }
    }
    small_sync<NT>();
    const int nvec = sm->n_pass;
    if (nvec <= small_pass_cap(NT)) {
        // ---- one thread per listed vector: read it back, append its candidates ----------------------
        constexpr int kInFlight = 2;
        static_assert(kInFlight * kPer <= 32, "one mask bit per logit a thread holds");
        for (int base = 0; base < nvec; base += kInFlight * NT) {
            float z[kInFlight][kPer];
            int vi[kInFlight];
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const int i = base + u * NT + tid;
                vi[u] = i < nvec ? (int)sm->pass[i] : -1;
                if (vi[u] >= 0) {
                    load_row_vector<T>(rowp, vi[u], ext, p.V, z[u]);
                } else {
#pragma unroll
                    for (int e = 0; e < kPer; ++e) z[u][e] = -INFINITY;
                }
            }
            uint32_t m = 0;
#pragma unroll
            for (int u = 0; u < kInFlight; ++u)
#pragma unroll
                for (int e = 0; e < kPer; ++e)
                    if (z[u][e] >= -3.4028234e38f && rel_key(z[u][e], z0) >= min_key) m |= 1u << (u * kPer + e);
            int pos = warp_reserve(&sm->n_cand, __popc(m), lane);
#pragma unroll
            for (int u = 0; u < kInFlight; ++u)
#pragma unroll
                for (int e = 0; e < kPer; ++e) {
                    if ((m >> (u * kPer + e)) & 1u) {
                        if (pos < small_list_cap(NT))
                            sm->comp[pos] = ((unsigned long long)float_to_key(z[u][e]) << 32) |
                                            (unsigned long long)(0xffffffffu - (uint32_t)(vi[u] * kPer + e));
                        ++pos;
                    }
                }
        }
        small_sync<NT>();
        if (sm->n_cand <= small_list_cap(NT)) return sm->n_cand;
    }
    return winners_one_by_one<T, NT>(p, row, ent, n_tiles, bin, z0, nvec <= small_pass_cap(NT) ? nvec : -1, sm, tid);
}

constexpr int small_resident(int nt) { return nt == 64 ? 24 : nt == 96 ? 16 : nt == 128 ? 12 : 6; }

template <typename T, int NT>
__global__ void __launch_bounds__(NT, small_resident(NT)) sparsify_finish_small_kernel(const SparsifyParams p) {
    constexpr int kHeld = (small_cand_cap(NT) + NT - 1) / NT;  // candidates a thread holds in registers
    __shared__ SmallSharedFor<NT> sm;
    const int tid = threadIdx.x, row = blockIdx.x, k = p.k;
    float u_raw = 0.f;
    if (tid < p.num_samples) u_raw = p.uniforms[(size_t)row * p.num_samples + tid];  // an input: may be read early
    // Nothing the streaming kernel wrote is read before this point.  The row's own ready flag is
    // enough to go on (see poll_row_ready); if it does not come, the end of the streaming kernel is.
    if (tid == 0) sm.n_cut = poll_row_ready(&p.row_ready[row]) ? 1 : 0;
    small_sync<NT>();
    if (!sm.n_cut) wait_for_primary_kernel();
    small_sync<NT>();
    if (row == 0 && tid == 0) *p.status = 0;
    // ---- one trip to memory: the candidates, their count, the per-warp statistics, the uniforms' line
    const SegStat* st = &p.seg_stats[row];
    const uint2* ent = p.seg_entries + (size_t)row * p.seg_stride;
    unsigned long long held[kHeld];  // key << 32 | ~index
#pragma unroll
    for (int c = 0; c < kHeld; ++c) {
        const int i = tid + c * NT;
        const uint2 e = i < p.seg_cap ? __ldcg(&ent[i]) : make_uint2(0u, 0u);
        held[c] = ((unsigned long long)e.x << 32) | (unsigned long long)(0xffffffffu - e.y);
    }
    int nc = __ldcg(&st->n);
    const int raw_bin = __ldcg(&st->raw_bin);
    // the log-normaliser once, by one warp (fp64 is scarce): one per-warp pair per lane
    if (tid < 32) {
        const double Sw = tid < kWarps ? __ldcg(&st->S[tid]) : 0.0;
        const double Mw = tid < kWarps ? (double)__ldcg(&st->M[tid]) : -INFINITY;
        const double Mrow = warp_max(Sw > 0.0 ? Mw : -INFINITY);
        const double Srow = warp_sum(Sw > 0.0 ? Sw * exp2(Mw - Mrow) : 0.0);
        if (tid == 0) sm.lrow = Mrow + log2(Srow);
    }
    if (raw_bin >= 0) {  // the entries are staged lane tiles: make the candidates from them first
        nc = candidates_from_tiles<T, NT>(p, row, ent, nc, raw_bin, __ldcg(&st->z0), &sm, tid);
#pragma unroll
        for (int c = 0; c < kHeld; ++c) {
            const int i = tid + c * NT;
            held[c] = i < nc ? sm.comp[i] : 0ull;
        }
    } else {
        nc = nc < 0 ? 0 : (nc > small_cand_cap(NT) ? small_cand_cap(NT) : nc);
#pragma unroll
        for (int c = 0; c < kHeld; ++c) {
            const int i = tid + c * NT;
            if (i < nc) sm.comp[i] = held[c];
        }
    }
    small_sync<NT>();
    // ---- exact top-k by counting ranks under (key descending, index ascending) -------------------
    // (only the threads that hold a candidate count; the 64-bit composite makes it one compare per entry)
#pragma unroll
    for (int c = 0; c < kHeld; ++c) {
        if (tid + c * NT < nc) {
            const unsigned long long mine = held[c];
            int r = 0;
            for (int j = 0; j < nc; ++j) r += sm.comp[j] > mine ? 1 : 0;
            if (r < k) {
                sm.wkey[r] = (uint32_t)(mine >> 32);
                sm.widx[r] = (int)(0xffffffffu - (uint32_t)mine);
            }
        }
    }
    for (int i = kHeld * NT + tid; i < nc; i += NT) {  // a long list made from tiles: the rest of it
        const unsigned long long mine = sm.comp[i];
        int r = 0;
        for (int j = 0; j < nc; ++j) r += sm.comp[j] > mine ? 1 : 0;
        if (r < k) {
            sm.wkey[r] = (uint32_t)(mine >> 32);
            sm.widx[r] = (int)(0xffffffffu - (uint32_t)mine);
        }
    }
    small_sync<NT>();
    const int n0 = nc < k ? nc : k;
    const double L2 = sm.lrow;  // written before the barriers above
    const double cd = p.c.d;
    // ---- nucleus cut on the cumulative q in that order ---------------------------------------------
    int n = n0;
    double mass = 0.0;
    {
        double q = 0.0;
        if (tid < n0) q = exp2((double)key_to_float(sm.wkey[tid]) * cd - L2);
        double tot;
        const double c_incl = small_scan<NT>(q, tid, sm.red, &tot);
        if (p.top_p < 1.0f) {
            if (tid == 0) sm.n_cut = n0;
            if (tid < n0) sm.cum[tid] = c_incl;
            small_sync<NT>();
            const double tp = (double)p.top_p;
            // first crossing of the cumulative: exactly one thread, if any
            if (tid < n0 && c_incl >= tp && (tid == 0 || sm.cum[tid - 1] < tp)) sm.n_cut = tid + 1;
            small_sync<NT>();
            n = sm.n_cut;
            mass = n > 0 ? sm.cum[n - 1] : 0.0;
            small_sync<NT>();
        } else {
            mass = tot;
        }
    }
    // ---- ascending index order -----------------------------------------------------------------------
    if (tid < n) {
        const int mine = sm.widx[tid];
        int r = 0;
        for (int j = 0; j < n; ++j) r += sm.widx[j] < mine ? 1 : 0;
        sm.oidx[r] = mine;
        sm.okey[r] = sm.wkey[tid];
    }
    small_sync<NT>();
    // ---- renormalised truncated distribution and its CDF in fp64 -------------------------------------
    double y = -INFINITY;
    if (tid < n) y = (double)key_to_float(sm.okey[tid]) * cd;
    const double mS = small_max<NT>(y, tid, sm.red);
    const double w = tid < n ? exp2(y - mS) : 0.0;
    double W;
    const double cw = small_scan<NT>(w, tid, sm.red, &W);
    if (tid < n) { sm.cum[tid] = cw; sm.wv[tid] = w; }
    small_sync<NT>();
    // ---- outputs ----------------------------------------------------------------------------------------
    int* o_idx = p.idx + (size_t)row * k;
    float* o_logit = p.logit + (size_t)row * k;
    if (tid < k) {
        o_idx[tid] = tid < n ? sm.oidx[tid] : -1;
        o_logit[tid] = tid < n ? key_to_float(sm.okey[tid]) : -INFINITY;
    }
    if (tid == 0) {
        p.count[row] = n;
        if (p.lse) p.lse[row] = n0 > 0 ? (float)(L2 * 0.6931471805599453) : -INFINITY;
        if (p.mass) p.mass[row] = n0 > 0 ? (float)mass : 0.f;
    }
    for (int sidx = tid; sidx < p.num_samples; sidx += NT) {
        int tok = -1;
        if (n > 0) {
            const float u = clamp_uniform(sidx == tid ? u_raw : p.uniforms[(size_t)row * p.num_samples + sidx]);
            int pos = first_greater(sm.cum, n, (double)u * W);
            if (pos >= n) {
                pos = n - 1;
                while (pos > 0 && !(sm.wv[pos] > 0.0)) --pos;
            }
            tok = sm.oidx[pos];
        }
        p.token[(size_t)row * p.num_samples + sidx] = tok;
    }
    // This kernel's completion must imply the streaming kernel's (what follows on the stream relies
    // on it): one CTA sees to that; the others leave and make room.
    if (row == 0) wait_for_primary_kernel();
}

// The small finish kernel for this k: a warp's worth of threads per 32 of k, at least two warps.
template <typename T> static void (*small_finish_kernel(int k, int* threads))(const SparsifyParams) {
    if (k <= 64) { *threads = 64; return sparsify_finish_small_kernel<T, 64>; }
    if (k <= 96) { *threads = 96; return sparsify_finish_small_kernel<T, 96>; }
    if (k <= 128) { *threads = 128; return sparsify_finish_small_kernel<T, 128>; }
    *threads = 256;
    return sparsify_finish_small_kernel<T, 256>;
}

// ---- host side -------------------------------------------------------------------------------

struct SparsifyPlan {
    int nchunks, cap, high, fin_cap, vcap, vhigh, seg_cap, seg_stride, raw_cap;
    bool small_finish;
    RowSplit split;
    size_t smem;
    size_t ws_stats_off, ws_entries_off, ws_ready_off, ws_bytes;
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

constexpr int kSmemPerSm = 227 * 1024;

static SparsifyPlan make_sparsify_plan(int rows, int V, int k, int elt_bytes) {
    SparsifyPlan pl;
    const long long row_bytes = (long long)V * elt_bytes;
    pl.nchunks = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);
    pl.cap = 16 * k;
    if (pl.cap < 1024) pl.cap = 1024;
    if (pl.cap > 4096) pl.cap = 4096;
    // k <= 256: the staged tiles normally go to the finish kernel unexpanded, so the staging buffer
    // is sized never to fill on ordinary rows (about 8 k tiles are staged) and the candidate list,
    // used only when it does, is kept small: four CTAs still fit an SM
    if (k <= kSmallMaxThreads) pl.cap = 1024;
    pl.high = pl.cap - pl.cap / 4;
    // (large k stages thousands of tiles per row: a buffer that holds most of them saves the early
    // expansions, each a rendezvous of the warps and a round of reads back)
    pl.vcap = k <= 64 ? 1024 : k <= 256 ? 2048 : 4096;
    pl.vhigh = pl.vcap - pl.vcap / 4;
    pl.seg_cap = 2 * k;  // what one segment of a split row hands over (its k-th bin and above); see below
    pl.smem = sparsify_smem_bytes(pl.cap, pl.vcap, k);
    // CTAs the machine holds at once: launch bounds and the shared-memory footprint decide
    int per_sm = (int)(kSmemPerSm / (pl.smem + 1024));
    if (per_sm > kSparsifyCtasPerSm) per_sm = kSparsifyCtasPerSm;
    if (per_sm < 1) per_sm = 1;
    // a split row's segments must fit the candidate list of the CTA that merges them
    const int max_seg = pl.cap / pl.seg_cap < 16 ? pl.cap / pl.seg_cap : 16;
    // One CTA per row.  Only when there are fewer rows than half the SMs and the rows are long is a
    // row cut into segments (of at least 32 chunks): every segment pays the first threshold and the
    // hand-over, which on small batches (tens of rows) costs more than it gains.
    (void)per_sm;
    pl.split.rows = rows;
    int nseg = 1;
    if (rows > 0 && 2 * rows < sm_count_cached()) {
        nseg = sm_count_cached() / rows;
        if (nseg > pl.nchunks / 32) nseg = pl.nchunks / 32;
        if (nseg > max_seg) nseg = max_seg;
        if (nseg < 1) nseg = 1;
    }
    int cps = (pl.nchunks + nseg - 1) / nseg;
    cps = (cps + kWarps - 1) / kWarps * kWarps;
    if (cps < kWarps) cps = kWarps;
    pl.split.nseg = (pl.nchunks + cps - 1) / cps;
    if (pl.split.nseg < 1) pl.split.nseg = 1;
    pl.split.cps = cps;
    pl.split.grid = rows * pl.split.nseg;
    // the generic finish kernel holds what the row's segments hand over, no more: it fits more CTAs per SM
    pl.fin_cap = pl.split.nseg * pl.seg_cap;
    if (pl.fin_cap < 1024) pl.fin_cap = 1024;
    // rows of one segment with k <= 256 go to the small finish kernel, and hand their staged tiles over raw
    pl.small_finish = pl.split.nseg == 1 && k <= kSmallMaxThreads;  // (seg_cap = 2 k fits small_cand_cap)
    pl.raw_cap = pl.small_finish ? pl.vcap : 0;
    pl.seg_stride = pl.seg_cap > pl.raw_cap ? pl.seg_cap : pl.raw_cap;
    const size_t split_rows = (size_t)rows;
    size_t off = kWsHeaderBytes;
    pl.ws_stats_off = off;
    off = align_up(off + split_rows * pl.split.nseg * sizeof(SegStat), 256);
    pl.ws_entries_off = off;
    off = align_up(off + split_rows * pl.split.nseg * pl.seg_stride * sizeof(uint2), 256);
    pl.ws_ready_off = off;
    if (pl.split.nseg == 1) off = align_up(off + split_rows * sizeof(int), 256);
    pl.ws_bytes = off;
    return pl;
}

ScaleC make_scale(float temperature) {
    const double c = 1.4426950408889634 / (double)temperature;
    ScaleC s;
    s.f = (float)c;
    s.d = c;
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
    p.V = V; p.rows = rows; p.k = k;
    p.top_p = top_p;
    p.c = make_scale(temperature);
    p.num_samples = num_samples;
    p.uniforms = uniforms;
    p.idx = idx; p.logit = logit; p.count = count; p.token = token; p.lse = lse; p.mass = mass;
    p.nchunks = pl.nchunks; p.split = pl.split;
    p.cap = pl.cap; p.high = pl.high; p.fin_cap = pl.fin_cap; p.vcap = pl.vcap; p.vhigh = pl.vhigh; p.seg_cap = pl.seg_cap;
    p.seg_stride = pl.seg_stride; p.raw_cap = pl.raw_cap;
    p.idx_hi_byte = (V - 1) >= (1 << 24) ? 3 : (V - 1) >= (1 << 16) ? 2 : (V - 1) >= (1 << 8) ? 1 : 0;
    unsigned char* ws = (unsigned char*)workspace;
    p.status = (int*)ws;
    p.seg_stats = (SegStat*)(ws + pl.ws_stats_off);
    p.seg_entries = (uint2*)(ws + pl.ws_entries_off);
    p.row_ready = pl.split.nseg == 1 ? (int*)(ws + pl.ws_ready_off) : nullptr;  // rows of one segment only

    cudaStream_t st = (cudaStream_t)stream;
    auto kern = dtype == TSLT_F32 ? sparsify_kernel<float> : sparsify_kernel<bf16_t>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)sparsify_smem_bytes(4096, kMaxStagedTiles, TSLT_MAX_K)) != cudaSuccess)
        return TSLT_ERR_CUDA;
    kern<<<pl.split.grid, kBlockThreads, pl.smem, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return TSLT_ERR_CUDA;
    if (pl.small_finish) {
        int threads = 0;
        auto fin = dtype == TSLT_F32 ? small_finish_kernel<float>(k, &threads) : small_finish_kernel<bf16_t>(k, &threads);
        if (launch_dependent(fin, rows, threads, 0, st, p) != cudaSuccess) return TSLT_ERR_CUDA;
    } else {
        auto fin = dtype == TSLT_F32 ? sparsify_finish_kernel<float> : sparsify_finish_kernel<bf16_t>;
        if (cudaFuncSetAttribute(fin, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sparsify_smem_bytes(4096, 0, TSLT_MAX_K)) != cudaSuccess)
            return TSLT_ERR_CUDA;
        if (launch_dependent(fin, rows, kBlockThreads, sparsify_smem_bytes(pl.fin_cap, 0, k), st, p) != cudaSuccess)
            return TSLT_ERR_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return TSLT_ERR_CUDA;
    return TSLT_OK;
}
