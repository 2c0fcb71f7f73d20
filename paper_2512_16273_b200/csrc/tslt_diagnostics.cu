// tslt_diagnostics: the truncation diagnostics of the paper on pairs of (draft, target) rows: the
// retained mass rho(K) of the top-K set for a list of K (the top-K mass curve of Section 5), the
// acceptance rates beta^(j) of the j-th candidate (Section 4.3) without truncation and beta_hat^(j)(K)
// with it, the residual normalisers Z^(j) (recursive TV lemma), and the total acceptance theta.
// Theorem 1 (|beta_hat - beta| <= sigma, TV(Q^, Q) = sigma = 1 - rho) and Theorem 2 are then checks
// on these outputs.
//
// Four steps on the caller's stream:
//   1. tslt_sparsify with k = the largest K and no samples: the top-K_max set of every draft row;
//   2. diag_lse_kernel: the log-normalisers of the draft and the target row (one pass over both);
//   3. diag_chain_kernel, once per candidate j: beta^(j) = sum_v min(q, p^(j)) and Z^(j+1) =
//      sum_v max(0, p^(j) - q) over the whole vocabulary, p^(j) rebuilt per logit from p, q and the
//      earlier Z (p^(s+1) = max(0, p^(s) - q) / Z^(s+1));
//   4. diag_topk_kernel: the top-K_max pairs in the order (logit descending, index ascending), their q
//      and p, the cumulative q (rho for every K), and for every K the candidate chain against the
//      truncated, renormalised q^ on the K values plus one scalar for the mass outside them.
// Steps 2 and 3 stream both rows again: these are diagnostics, 2 + 2 c reads of the logits, not a hot path.
#include <math.h>

#include "tslt_common.cuh"
#include "tslt_rowmath.cuh"

namespace tslt {

constexpr int kMaxDiagK = 16;         // entries of the K list
constexpr int kMaxDiagCandidates = 8;
// A residual mass at or below this is rounding noise of two distributions that agree (exact
// arithmetic gives 0): like the verifier, the chain then leaves p^(j) as it is.
constexpr double kDiagMinResidualMass = 4.0e-7;

struct DiagParams {
    const unsigned char* zq;
    const unsigned char* zp;
    long long row_stride_bytes;
    int V, rows, kmax, nk, c, j;  // j: the candidate of this launch of diag_chain_kernel (1-based)
    int klist[kMaxDiagK];
    ScaleC cq, cp;
    const int* idx;      // [rows, kmax] from tslt_sparsify
    const float* logit;  // [rows, kmax]
    const int* count;    // [rows]
    double* lse2;        // [rows, 2]: base-2 log-normalisers of the draft and the target row
    double* chain;       // [rows, 2 c]: beta^(1..c) then Z^(2..c+1)
    float* beta_j;       // [rows, c]
    float* z_j;          // [rows, c]
    float* theta;        // [rows]
    float* rho;          // [rows, nk]
    float* beta_hat_j;   // [rows, nk, c]
    float* theta_hat;    // [rows, nk]
};

// base-2 log of sum 2^(z c) over one row, by the CTA's 8 warps (the streaming core of the library)
template <typename T>
__device__ __forceinline__ double row_log2_sum(const unsigned char* rowp, int V, float c, int nchunks, int tid, double* scratch) {
    const int lane = tid & 31, warp = tid >> 5;
    const RowExtent ext = row_extent<T>(V);
    LaneSum ls;
    ls.reset();
    for (int ch = warp; ch < nchunks; ch += kWarps) {
        LaneTile<T> lt;
        lt.load(rowp, ch * kVecsPerChunk, lane, ext);
        ls.raise_to(lt.reduce_max(), c);
        lt.accumulate(ls, c);
    }
    const double M = block_max((double)ls.M, tid, scratch);
    const double S = block_sum(ls.total_f64() * exp2((double)ls.M - M), tid, scratch);
    return S > 0.0 ? M + log2(S) : -INFINITY;
}

template <typename T>
__global__ void __launch_bounds__(kBlockThreads, 4) diag_lse_kernel(const DiagParams p) {
    __shared__ double scratch[16];
    const int row = blockIdx.x, tid = threadIdx.x;
    const int nchunks = (int)(((long long)p.V * Elt<T>::kBytes + kChunkBytes - 1) / kChunkBytes);
    const double lq = row_log2_sum<T>(p.zq + (long long)row * p.row_stride_bytes, p.V, p.cq.f, nchunks, tid, scratch);
    const double lp = row_log2_sum<T>(p.zp + (long long)row * p.row_stride_bytes, p.V, p.cp.f, nchunks, tid, scratch);
    if (tid == 0) {
        p.lse2[2 * row] = lq;
        p.lse2[2 * row + 1] = lp;
    }
}

// beta^(j) and Z^(j+1) over the whole vocabulary.  p^(j)(v) is rebuilt from p(v), q(v) and Z^(2..j).
template <typename T>
__global__ void __launch_bounds__(kBlockThreads, 4) diag_chain_kernel(const DiagParams p) {
    __shared__ double scratch[16];
    const int row = blockIdx.x, tid = threadIdx.x, j = p.j;
    const unsigned char* rq = p.zq + (long long)row * p.row_stride_bytes;
    const unsigned char* rp = p.zp + (long long)row * p.row_stride_bytes;
    const double lq = p.lse2[2 * row], lp = p.lse2[2 * row + 1];
    const double cq = (double)p.cq.f, cp = (double)p.cp.f;  // the scales the normalisers were summed with
    float inv_z[kMaxDiagCandidates];
#pragma unroll
    for (int s = 0; s < kMaxDiagCandidates; ++s) {
        const double z = s < j - 1 ? p.chain[(size_t)row * 2 * p.c + p.c + s] : 1.0;
        inv_z[s] = z > kDiagMinResidualMass ? (float)(1.0 / z) : -1.f;  // negative: no update at this step
    }
    double b = 0.0, zsum = 0.0;
    for (int v = tid; v < p.V; v += kBlockThreads) {
        const float fq = Elt<T>::load(rq, v), fp = Elt<T>::load(rp, v);
        const float q = fabsf(fq) <= 3.4028234e38f ? exp2f((float)((double)fq * cq - lq)) : 0.f;
        float r = fabsf(fp) <= 3.4028234e38f ? exp2f((float)((double)fp * cp - lp)) : 0.f;
#pragma unroll
        for (int s = 0; s < kMaxDiagCandidates; ++s)
            if (s < j - 1 && inv_z[s] > 0.f) r = fmaxf(0.f, r - q) * inv_z[s];
        b += (double)fminf(q, r);
        zsum += (double)fmaxf(0.f, r - q);
    }
    b = block_sum(b, tid, scratch);
    zsum = block_sum(zsum, tid, scratch);
    if (tid == 0) {
        p.chain[(size_t)row * 2 * p.c + (j - 1)] = b;
        p.chain[(size_t)row * 2 * p.c + p.c + (j - 1)] = zsum;
        p.beta_j[(size_t)row * p.c + (j - 1)] = (float)b;
        p.z_j[(size_t)row * p.c + (j - 1)] = (float)zsum;
    }
}

// Bitonic sort of a[0..P) (P a power of two, shared memory), descending, by the 256 threads.
__device__ __forceinline__ void diag_sort_desc(unsigned long long* a, int P, int tid) {
    for (int size = 2; size <= P; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = tid; i < (P >> 1); i += kBlockThreads) {
                const int lo = 2 * i - (i & (stride - 1));
                const int hi = lo + stride;
                const bool up = ((lo & size) == 0);
                const unsigned long long x = a[lo], y = a[hi];
                if (up ? x < y : x > y) {
                    a[lo] = y;
                    a[hi] = x;
                }
            }
            consumer_sync();
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kBlockThreads, 2) diag_topk_kernel(const DiagParams p) {
    __shared__ unsigned long long comp[TSLT_MAX_K];
    __shared__ double qv[TSLT_MAX_K], pv[TSLT_MAX_K], av[TSLT_MAX_K];
    __shared__ double scratch[16];
    const int row = blockIdx.x, tid = threadIdx.x;
    const unsigned char* rp = p.zp + (long long)row * p.row_stride_bytes;
    const double lq = p.lse2[2 * row], lp = p.lse2[2 * row + 1];
    int n = p.count[row];
    n = n < 0 ? 0 : (n > p.kmax ? p.kmax : n);
    int P = 1;
    while (P < n) P <<= 1;
    const int* idx = p.idx + (size_t)row * p.kmax;
    const float* lg = p.logit + (size_t)row * p.kmax;
    for (int i = tid; i < P; i += kBlockThreads)
        comp[i] = i < n ? (((unsigned long long)float_to_key(lg[i]) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)idx[i])) : 0ull;
    consumer_sync();
    diag_sort_desc(comp, P, tid);
    // q and p of the pairs in that order; cumulative q
    for (int i = tid; i < n; i += kBlockThreads) {
        const float z = key_to_float((uint32_t)(comp[i] >> 32));
        const int v = (int)(0xffffffffu - (uint32_t)comp[i]);
        qv[i] = exp2((double)z * (double)p.cq.f - lq);
        const float zt = Elt<T>::load(rp, v);
        pv[i] = fabsf(zt) <= 3.4028234e38f ? exp2((double)zt * (double)p.cp.f - lp) : 0.0;
    }
    consumer_sync();
    // theta of the untruncated chain, from the betas the chain kernel left
    if (tid == 0) {
        double theta = 0.0, stay = 1.0;
        for (int j = 0; j < p.c; ++j) {
            const double b = p.chain[(size_t)row * 2 * p.c + j];
            theta += stay * b;
            stay *= 1.0 - b;
        }
        p.theta[row] = (float)theta;
    }
    for (int ik = 0; ik < p.nk; ++ik) {
        const int K = min(p.klist[ik], n);
        double part = 0.0;
        for (int i = tid; i < K; i += kBlockThreads) part += qv[i];
        const double rho = block_sum(part, tid, scratch);
        part = 0.0;
        for (int i = tid; i < K; i += kBlockThreads) {
            av[i] = pv[i];
            part += pv[i];
        }
        const double PS = block_sum(part, tid, scratch);
        const double out_mass = 1.0 - PS > 0.0 ? 1.0 - PS : 0.0;  // mass of p outside the K tokens
        double c_out = 1.0, theta = 0.0, stay = 1.0;
        for (int j = 0; j < p.c; ++j) {
            double bpart = 0.0, zpart = 0.0;
            for (int i = tid; i < K; i += kBlockThreads) {
                const double qh = rho > 0.0 ? qv[i] / rho : 0.0;
                bpart += fmin(qh, av[i]);
                zpart += fmax(0.0, av[i] - qh);
            }
            const double b = block_sum(bpart, tid, scratch);
            const double Z = block_sum(zpart, tid, scratch) + c_out * out_mass;
            if (tid == 0) p.beta_hat_j[((size_t)row * p.nk + ik) * p.c + j] = (float)b;
            theta += stay * b;
            stay *= 1.0 - b;
            if (Z > kDiagMinResidualMass) {
                for (int i = tid; i < K; i += kBlockThreads) {
                    const double qh = rho > 0.0 ? qv[i] / rho : 0.0;
                    av[i] = fmax(0.0, av[i] - qh) / Z;
                }
                c_out /= Z;
            }
            consumer_sync();
        }
        if (tid == 0) {
            p.rho[(size_t)row * p.nk + ik] = (float)rho;
            p.theta_hat[(size_t)row * p.nk + ik] = (float)theta;
        }
    }
}

ScaleC make_scale(float temperature);  // defined with the sparsify launcher

struct DiagPlan {
    size_t sparsify_bytes, idx_off, logit_off, count_off, lse_off, chain_off, total;
};
static int make_diag_plan(int rows, int V, int kmax, int c, DiagPlan* pl) {
    size_t sb = 0;
    const int rc = tslt_sparsify_workspace_bytes(rows, V, kmax, 0, &sb);
    if (rc != TSLT_OK) return rc;
    size_t off = align_up256(sb);
    pl->sparsify_bytes = sb;
    pl->idx_off = off;
    off = align_up256(off + (size_t)rows * kmax * sizeof(int));
    pl->logit_off = off;
    off = align_up256(off + (size_t)rows * kmax * sizeof(float));
    pl->count_off = off;
    off = align_up256(off + (size_t)rows * sizeof(int));
    pl->lse_off = off;
    off = align_up256(off + (size_t)rows * 2 * sizeof(double));
    pl->chain_off = off;
    off = align_up256(off + (size_t)rows * 2 * (c > 0 ? c : 1) * sizeof(double));
    pl->total = off;
    return TSLT_OK;
}

}  // namespace tslt

using namespace tslt;

extern "C" int tslt_diagnostics_workspace_bytes(int rows, int V, int k_max, int num_candidates, size_t* bytes) {
    if (!bytes || rows < 0 || V <= 0 || k_max <= 0 || k_max > V || k_max > TSLT_MAX_K || num_candidates < 1 ||
        num_candidates > kMaxDiagCandidates)
        return TSLT_ERR_INVALID_ARG;
    DiagPlan pl;
    const int rc = make_diag_plan(rows, V, k_max, num_candidates, &pl);
    if (rc != TSLT_OK) return rc;
    *bytes = pl.total;
    return TSLT_OK;
}

extern "C" int tslt_diagnostics(const void* draft_logits, const void* target_logits, int dtype, int rows, int V,
                                long long row_stride_elems, const int* k_list, int n_k, int num_candidates,
                                float draft_temperature, float target_temperature, float* beta_j, float* z_j,
                                float* theta, float* rho, float* beta_hat_j, float* theta_hat, void* workspace,
                                size_t workspace_bytes, void* stream) {
    if (dtype != TSLT_F32 && dtype != TSLT_BF16) return TSLT_ERR_UNSUPPORTED;
    const int eb = dtype == TSLT_F32 ? 4 : 2;
    if (rows < 0 || V <= 0 || !k_list || n_k < 1 || n_k > kMaxDiagK || num_candidates < 1 ||
        num_candidates > kMaxDiagCandidates || !(draft_temperature > 0.f) || !(target_temperature > 0.f) ||
        !isfinite(draft_temperature) || !isfinite(target_temperature))
        return TSLT_ERR_INVALID_ARG;
    for (int i = 0; i < n_k; ++i)
        if (k_list[i] < 1 || k_list[i] > V || k_list[i] > TSLT_MAX_K || (i > 0 && k_list[i] <= k_list[i - 1]))
            return TSLT_ERR_INVALID_ARG;
    if (rows == 0) return TSLT_OK;
    if (!draft_logits || !target_logits || !beta_j || !z_j || !theta || !rho || !beta_hat_j || !theta_hat || !workspace)
        return TSLT_ERR_INVALID_ARG;
    if (row_stride_elems < V || ((uintptr_t)draft_logits & 15) || ((uintptr_t)target_logits & 15) ||
        ((row_stride_elems * eb) & 15) || ((uintptr_t)workspace & 255))
        return TSLT_ERR_INVALID_ARG;
    const int kmax = k_list[n_k - 1];
    DiagPlan pl;
    int rc = make_diag_plan(rows, V, kmax, num_candidates, &pl);
    if (rc != TSLT_OK) return rc;
    if (workspace_bytes < pl.total) return TSLT_ERR_WORKSPACE;
    unsigned char* ws = (unsigned char*)workspace;
    int* idx = (int*)(ws + pl.idx_off);
    float* logit = (float*)(ws + pl.logit_off);
    int* count = (int*)(ws + pl.count_off);
    rc = tslt_sparsify(draft_logits, dtype, rows, 1, V, row_stride_elems, kmax, 1.0f, draft_temperature, 0, nullptr, idx,
                       logit, count, nullptr, nullptr, nullptr, ws, pl.sparsify_bytes, stream);
    if (rc != TSLT_OK) return rc;
    DiagParams p = {};
    p.zq = (const unsigned char*)draft_logits;
    p.zp = (const unsigned char*)target_logits;
    p.row_stride_bytes = row_stride_elems * eb;
    p.V = V; p.rows = rows; p.kmax = kmax; p.nk = n_k; p.c = num_candidates;
    for (int i = 0; i < n_k; ++i) p.klist[i] = k_list[i];
    p.cq = make_scale(draft_temperature);
    p.cp = make_scale(target_temperature);
    p.idx = idx; p.logit = logit; p.count = count;
    p.lse2 = (double*)(ws + pl.lse_off);
    p.chain = (double*)(ws + pl.chain_off);
    p.beta_j = beta_j; p.z_j = z_j; p.theta = theta; p.rho = rho; p.beta_hat_j = beta_hat_j; p.theta_hat = theta_hat;
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == TSLT_F32) diag_lse_kernel<float><<<rows, kBlockThreads, 0, st>>>(p);
    else diag_lse_kernel<bf16_t><<<rows, kBlockThreads, 0, st>>>(p);
    for (int j = 1; j <= num_candidates; ++j) {
        p.j = j;
        if (dtype == TSLT_F32) diag_chain_kernel<float><<<rows, kBlockThreads, 0, st>>>(p);
        else diag_chain_kernel<bf16_t><<<rows, kBlockThreads, 0, st>>>(p);
    }
    if (dtype == TSLT_F32) diag_topk_kernel<float><<<rows, kBlockThreads, 0, st>>>(p);
    else diag_topk_kernel<bf16_t><<<rows, kBlockThreads, 0, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? TSLT_OK : TSLT_ERR_CUDA;
}
