// Per-row kernels of the CAT loss: merging the vocabulary-split softmax partials into lse,
// the confidence of Eq. 9, the segmented exclusive product scan of Eq. 10 (warp shuffles,
// strictly left to right so the binary32 result equals the sequential product), the weighted
// loss of Eq. 11 with a fixed-order reduction, and the small set-up kernel of the backward pass.
// These touch O(T) data and are bandwidth/latency-bound; no tensor cores are involved.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace cat {
namespace rows {

constexpr int ROW_THREADS = 256;

// Per-CTA partial sums, reduced in a fixed order by finalize_kernel.
struct CtaPartial {
    double loss;        // sum_r weight_r * (lse_r - z[r, y_r])
    double sum_w;       // sum_r weight_r
    double sum_wc;      // sum_r weight_r * conf_r   (Eq. 8 estimate, summed over blocks)
    long long n_valid;
    long long n_bad;
};

struct RowParams {
    const float* part_m;       // [S][part_stride]
    const float* part_l;       // [S][part_stride]
    const float* z_label;      // [T]
    const long long* labels;   // [T]
    const unsigned char* valid;  // [T] or nullptr
    const float* conf_ext;     // [T] or nullptr
    float* lse;                // [T]
    float* conf;               // [T]
    float* weight;             // [T]
    float* row_ce;             // [T] scratch: lse - z_label (0 for invalid rows); used by the general-K path
    CtaPartial* partials;      // [gridDim.x]
    long long part_stride;     // row pitch of the partial arrays (>= T)
    int T, V, K, S;
    int fixed_decay;           // 0: Eq. 10 (product of confidences); 1: gamma^k by position
    float gamma;
};

__device__ __forceinline__ void block_reduce_store(double loss, double sw, double swc, long long nv, long long nb,
                                                   CtaPartial* out) {
    // fixed-order tree: shuffles inside each warp, then warp 0 adds the per-warp sums in order
    __shared__ double s_loss[ROW_THREADS / 32], s_sw[ROW_THREADS / 32], s_swc[ROW_THREADS / 32];
    __shared__ long long s_nv[ROW_THREADS / 32], s_nb[ROW_THREADS / 32];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        loss += __shfl_down_sync(0xffffffffu, loss, off);
        sw += __shfl_down_sync(0xffffffffu, sw, off);
        swc += __shfl_down_sync(0xffffffffu, swc, off);
        nv += __shfl_down_sync(0xffffffffu, nv, off);
        nb += __shfl_down_sync(0xffffffffu, nb, off);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { s_loss[warp] = loss; s_sw[warp] = sw; s_swc[warp] = swc; s_nv[warp] = nv; s_nb[warp] = nb; }
    __syncthreads();
    if (threadIdx.x == 0) {
        CtaPartial p = {0.0, 0.0, 0.0, 0, 0};
        for (int w = 0; w < ROW_THREADS / 32; ++w) {
            p.loss += s_loss[w]; p.sum_w += s_sw[w]; p.sum_wc += s_swc[w]; p.n_valid += s_nv[w]; p.n_bad += s_nb[w];
        }
        *out = p;
    }
}

// One thread per row.  SCAN = true: K is a power of two <= 32, the K rows of a block sit in K
// adjacent lanes and the exclusive product is formed with K-1 shuffles, left to right.
// SCAN = false: only lse / conf / row_ce are written; block_scan_kernel finishes the job.
template <bool SCAN>
__global__ void __launch_bounds__(ROW_THREADS) row_kernel(const RowParams p) {
    const int r = blockIdx.x * ROW_THREADS + threadIdx.x;
    const bool in_range = r < p.T;
    bool ok = false, bad = false;
    float c = 1.f, ce = 0.f;
    if (in_range) {
        // merge the per-split (max, sum-exp) pairs in split order
        float m = -INFINITY;
        for (int s = 0; s < p.S; ++s) m = fmaxf(m, p.part_m[static_cast<size_t>(s) * p.part_stride + r]);
        float l = 0.f;
        for (int s = 0; s < p.S; ++s)
            l += p.part_l[static_cast<size_t>(s) * p.part_stride + r] * expf(p.part_m[static_cast<size_t>(s) * p.part_stride + r] - m);
        const float lse = m + logf(l);
        p.lse[r] = lse;
        const long long y = p.labels[r];
        const bool mask = (p.valid == nullptr) || (p.valid[r] != 0);
        const bool y_ok = (y >= 0 && y < p.V);
        ok = mask && y_ok;
        bad = mask && !y_ok;
        if (ok) {
            const float zy = p.z_label[r];
            ce = lse - zy;
            c = p.conf_ext ? p.conf_ext[r] : expf(zy - lse);   // Eq. 9
        }
        p.conf[r] = c;
    }
    if (SCAN) {
        // Eq. 10: weight_k = ((1 * c_0) * c_1) ... * c_{k-1}; invalid rows carry the factor 1.
        // Fixed decay: every position carries the factor gamma instead.
        const int lane = threadIdx.x & 31;
        const int k = lane & (p.K - 1);
        const int base = lane - k;
        const float factor = p.fixed_decay ? p.gamma : c;
        float run = 1.f;
        for (int j = 0; j + 1 < p.K; ++j) {
            const float cj = __shfl_sync(0xffffffffu, factor, base + j);
            if (k > j) run = run * cj;
        }
        const float w = ok ? run : 0.f;
        if (in_range) p.weight[r] = w;
        block_reduce_store(static_cast<double>(w) * static_cast<double>(ce), w, static_cast<double>(w) * c,
                           ok ? 1 : 0, bad ? 1 : 0, &p.partials[blockIdx.x]);
    } else {
        if (in_range) p.row_ce[r] = ce;
    }
}

// General K (not a power of two, or > 32): one thread per draft block, sequential product.
__global__ void __launch_bounds__(ROW_THREADS) block_scan_kernel(const RowParams p) {
    const int b = blockIdx.x * ROW_THREADS + threadIdx.x;
    const int B = p.T / p.K;
    double loss = 0.0, sw = 0.0, swc = 0.0;
    long long nv = 0, nb = 0;
    if (b < B) {
        float run = 1.f;
        for (int k = 0; k < p.K; ++k) {
            const int r = b * p.K + k;
            const long long y = p.labels[r];
            const bool mask = (p.valid == nullptr) || (p.valid[r] != 0);
            const bool y_ok = (y >= 0 && y < p.V);
            const bool ok = mask && y_ok;
            const float c = p.conf[r];
            const float w = ok ? run : 0.f;
            p.weight[r] = w;
            if (p.fixed_decay) run = run * p.gamma;
            else if (ok) run = run * c;
            loss += static_cast<double>(w) * static_cast<double>(p.row_ce[r]);
            sw += w;
            swc += static_cast<double>(w) * c;
            nv += ok ? 1 : 0;
            nb += (mask && !y_ok) ? 1 : 0;
        }
    }
    block_reduce_store(loss, sw, swc, nv, nb, &p.partials[blockIdx.x]);
}

struct StatsOut {   // mirrors cat_stats
    long long n_valid, n_bad_labels;
    float sum_weight, est_accept_len;
    int device_status, reserved;
};

// Single CTA: adds the per-CTA partials in index order and writes loss = sum / N (Eq. 11).
__global__ void __launch_bounds__(ROW_THREADS) finalize_kernel(const CtaPartial* partials, int n_partials, int n_blocks,
                                                               float* loss, StatsOut* stats, const int* status) {
    __shared__ CtaPartial sh[ROW_THREADS];
    CtaPartial acc = {0.0, 0.0, 0.0, 0, 0};
    for (int i = threadIdx.x; i < n_partials; i += ROW_THREADS) {
        const CtaPartial q = partials[i];
        acc.loss += q.loss; acc.sum_w += q.sum_w; acc.sum_wc += q.sum_wc; acc.n_valid += q.n_valid; acc.n_bad += q.n_bad;
    }
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int off = ROW_THREADS / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off) {
            CtaPartial a = sh[threadIdx.x];
            const CtaPartial b = sh[threadIdx.x + off];
            a.loss += b.loss; a.sum_w += b.sum_w; a.sum_wc += b.sum_wc; a.n_valid += b.n_valid; a.n_bad += b.n_bad;
            sh[threadIdx.x] = a;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const CtaPartial t = sh[0];
        *loss = t.n_valid > 0 ? static_cast<float>(t.loss / static_cast<double>(t.n_valid)) : 0.f;
        if (stats) {
            stats->n_valid = t.n_valid;
            stats->n_bad_labels = t.n_bad;
            stats->sum_weight = static_cast<float>(t.sum_w);
            stats->est_accept_len = n_blocks > 0 ? static_cast<float>(t.sum_wc / n_blocks) : 0.f;
            stats->device_status = *status;
            stats->reserved = 0;
        }
    }
}

// Eq. 8 estimate per draft block: accept_len[b] = sum_k weight * conf, added in position order.
__global__ void __launch_bounds__(ROW_THREADS) accept_len_kernel(const float* conf, const float* weight, float* out,
                                                                 int n_blocks, int K) {
    const int b = blockIdx.x * ROW_THREADS + threadIdx.x;
    if (b >= n_blocks) return;
    float acc = 0.f;
    for (int k = 0; k < K; ++k) {
        const size_t r = static_cast<size_t>(b) * K + k;
        acc = fmaf(weight[r], conf[r], acc);
    }
    out[b] = acc;
}

// Eq. 12 layout: draft row (block b, position k) takes the confidence of sequence position
// block_start[b] + k; positions outside the sequence read as 1.
__global__ void __launch_bounds__(ROW_THREADS) conf_window_kernel(const float* conf_seq, long long L,
                                                                  const long long* block_start, long long n_rows, int K,
                                                                  float* conf_ext) {
    const long long r = static_cast<long long>(blockIdx.x) * ROW_THREADS + threadIdx.x;
    if (r >= n_rows) return;
    const long long b = r / K;
    const long long i = block_start[b] + (r - b * K);
    conf_ext[r] = (i >= 0 && i < L) ? conf_seq[i] : 1.f;
}

// Backward set-up, single CTA: N = number of valid rows, scale = g / N (0 when N = 0).
__global__ void __launch_bounds__(1024) bwd_scale_kernel(const long long* labels, const unsigned char* valid, int T, int V,
                                                         const float* grad_loss, float* scale) {
    __shared__ int sh[32];
    int n = 0;
    for (int r = threadIdx.x; r < T; r += 1024) {
        const long long y = labels[r];
        n += ((valid == nullptr || valid[r] != 0) && y >= 0 && y < V) ? 1 : 0;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) n += __shfl_down_sync(0xffffffffu, n, off);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < 32; ++w) tot += sh[w];
        const float g = grad_loss ? *grad_loss : 1.f;
        *scale = tot > 0 ? g / static_cast<float>(tot) : 0.f;
    }
}

// Single CTA: N = number of rows that take part (mask bit set and label inside [0, V)).
__global__ void __launch_bounds__(1024) count_valid_kernel(const long long* labels, const unsigned char* valid, int T, int V,
                                                           long long* n_out) {
    __shared__ int sh[32];
    int n = 0;
    for (int r = threadIdx.x; r < T; r += 1024) {
        const long long y = labels[r];
        n += ((valid == nullptr || valid[r] != 0) && y >= 0 && y < V) ? 1 : 0;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) n += __shfl_down_sync(0xffffffffu, n, off);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long tot = 0;
        for (int w = 0; w < 32; ++w) tot += sh[w];
        *n_out = tot;
    }
}

// One-call path, before the logits GEMM of a row slab: the per-row reference of the stored
// softmax numerators, ref[r] = z[r, y_r] = H[r, :] . W[y_r, :] as an fp32 dot product (one warp per
// row).  Any finite per-row constant would do; the label logit keeps exp(z - ref) near the
// probabilities' ratio to the label's.  Rows that take no part get 0.
__global__ void __launch_bounds__(ROW_THREADS) label_ref_kernel(const __nv_bfloat16* H, long long ldH, const __nv_bfloat16* W,
                                                                long long ldW, int d, const long long* labels,
                                                                const unsigned char* valid, int n_rows, int V, float* ref) {
    const int warp = (blockIdx.x * ROW_THREADS + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= n_rows) return;
    const long long y = labels[warp];
    float acc = 0.f;
    if ((valid == nullptr || valid[warp] != 0) && y >= 0 && y < V) {
        const uint4* h = reinterpret_cast<const uint4*>(H + static_cast<size_t>(warp) * ldH);
        const uint4* w = reinterpret_cast<const uint4*>(W + static_cast<size_t>(y) * ldW);
        for (int i = lane; i < d / 8; i += 32) {
            const uint4 a = h[i], b = w[i];
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[j]));
                const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[j]));
                acc = fmaf(fa.x, fb.x, acc);
                acc = fmaf(fa.y, fb.y, acc);
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    }
    if (lane == 0) ref[warp] = acc;
}

// One-call path, after the row kernel of a slab (lse and weights known).  With the slab holding
// e[r, v] = exp(z[r, v] - ref[r]), the backward's dz[r, v] = weight[r] * (exp(z - lse) - [v == y_r])
// equals a[r] * e'[r, v], where a[r] = weight[r] * exp(ref[r] - lse[r]) and e' is e with the label
// entry lowered by exp(lse[r] - ref[r]).  One CTA per row:
//   * a[r] (0 for rows that take no part) for the dH GEMM's epilogue;
//   * the label entry of the slab row patched in place (from the fp32 label logit);
//   * Hs[r, :] = a[r] * H[r, :] in bf16, the dW GEMM's second operand (the factor rides on the
//     contraction index there, so it has to sit in an operand).
__global__ void __launch_bounds__(ROW_THREADS) slab_prep_kernel(void* zs, long long ldz, const __nv_bfloat16* H, long long ldH,
                                                                int d, const long long* labels, const unsigned char* valid,
                                                                const float* lse, const float* weight, const float* z_label,
                                                                const float* ref, int V, float* a_out, __nv_bfloat16* Hs) {
    const int r = blockIdx.x;
    const long long y = labels[r];
    const bool ok = (valid == nullptr || valid[r] != 0) && y >= 0 && y < V;
    const float a = ok ? weight[r] * expf(ref[r] - lse[r]) : 0.f;
    if (threadIdx.x == 0) {
        a_out[r] = a;
        if (ok) {
            // exp(lse - ref) = 1 / (probability of the label) when ref is the label logit; capped like the slab
            const float e_label = expf(fminf(z_label[r] - ref[r], 79.f)) - expf(fminf(lse[r] - ref[r], 79.f));
            reinterpret_cast<__nv_bfloat16*>(zs)[static_cast<size_t>(r) * ldz + y] = __float2bfloat16_rn(e_label);
        }
    }
    const uint4* src = reinterpret_cast<const uint4*>(H + static_cast<size_t>(r) * ldH);
    uint4* dst = reinterpret_cast<uint4*>(Hs + static_cast<size_t>(r) * d);
    for (int i = threadIdx.x; i < d / 8; i += ROW_THREADS) {
        const uint4 in = src[i];
        const uint32_t wds[4] = {in.x, in.y, in.z, in.w};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wds[j]));
            __nv_bfloat162 b = __floats2bfloat162_rn(a * f.x, a * f.y);
            o[j] = *reinterpret_cast<uint32_t*>(&b);
        }
        dst[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

}  // namespace rows
}  // namespace cat
