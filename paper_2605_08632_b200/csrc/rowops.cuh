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

// Fused path: turn one row of stored fp16 logits into bf16 dz in place,
//   dz[r, v] = weight_r * (exp(z[r, v] - lse_r) - [v == y_r]),
// the label entry formed from the fp32 label logit.  One CTA per row, 16-byte vectors; columns
// at or beyond V are written as zero.  Pure streaming: 2 bytes read + 2 bytes written per logit.
__global__ void __launch_bounds__(ROW_THREADS) z_to_dz_kernel(void* zs, long long ldz, const long long* labels,
                                                              const unsigned char* valid, const float* lse,
                                                              const float* weight, const float* z_label, int V) {
    const int r = blockIdx.x;
    const long long y = labels[r];
    const bool ok = (valid == nullptr || valid[r] != 0) && y >= 0 && y < V;
    const float w = ok ? weight[r] : 0.f;
    const float l2 = ok ? lse[r] * 1.4426950408889634f : INFINITY;
    const int yi = ok ? static_cast<int>(y) : -1;
    const float dz_label = ok ? w * (expf(z_label[r] - lse[r]) - 1.f) : 0.f;
    uint4* row = reinterpret_cast<uint4*>(static_cast<unsigned short*>(zs) + static_cast<size_t>(r) * ldz);
    const int groups = static_cast<int>(ldz / 8);
    for (int gi = threadIdx.x; gi < groups; gi += ROW_THREADS) {
        const uint4 in = __ldcs(row + gi);
        const uint32_t wds[4] = {in.x, in.y, in.z, in.w};
        float f[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&wds[i]));
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
        const int col = gi * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float pz;
            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(pz) : "f"(fmaf(f[i], 1.4426950408889634f, -l2)));
            f[i] = (col + i < V) ? w * pz : 0.f;
            if (col + i == yi) f[i] = dz_label;
        }
        uint4 out;
        __nv_bfloat162 b0 = __floats2bfloat162_rn(f[0], f[1]);
        __nv_bfloat162 b1 = __floats2bfloat162_rn(f[2], f[3]);
        __nv_bfloat162 b2 = __floats2bfloat162_rn(f[4], f[5]);
        __nv_bfloat162 b3 = __floats2bfloat162_rn(f[6], f[7]);
        out.x = *reinterpret_cast<uint32_t*>(&b0);
        out.y = *reinterpret_cast<uint32_t*>(&b1);
        out.z = *reinterpret_cast<uint32_t*>(&b2);
        out.w = *reinterpret_cast<uint32_t*>(&b3);
        row[gi] = out;
    }
}

}  // namespace rows
}  // namespace cat
