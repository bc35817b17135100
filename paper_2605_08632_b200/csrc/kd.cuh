// Row kernels of the distillation term of Eq. 12 (Section 3.3): per draft row the loss is
// s * (beta * CE + KD) with KD = KL(p_target || q_draft) over the vocabulary.  The target's
// distribution of draft row (block b, position k) is the one of sequence position
// t = block_start[b] + k, so one stored row of target logits serves every draft row that
// predicts that position.  These kernels stream the stored fp16 logits of the draft slab and
// of the target slab (HBM-bound, no tensor cores); the three contractions stay in tc_gemm.cuh.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "rowops.cuh"

namespace cat {
namespace kd {

using rows::ROW_THREADS;
constexpr float LOG2E = 1.4426950408889634f;

// A draft row takes part iff its mask bit is set, its label is a token id and its target
// position exists.  One thread per row.
__global__ void __launch_bounds__(ROW_THREADS) prepare_kernel(const long long* labels, const unsigned char* valid,
                                                              const long long* block_start, int T, int K, int V, long long L,
                                                              unsigned char* valid_eff) {
    const int r = blockIdx.x * ROW_THREADS + threadIdx.x;
    if (r >= T) return;
    const long long y = labels[r];
    const int b = r / K;
    const long long t = block_start[b] + (r - b * K);
    valid_eff[r] = ((valid == nullptr || valid[r] != 0) && y >= 0 && y < V && t >= 0 && t < L) ? 1 : 0;
}

// Target confidence of Eq. 9 for the draft rows of one slab: the target's logit of the row's own
// label, z_t[t, y_r] = Ht[t, :] . Wt[y_r, :], as an fp32 dot product (one warp per row), and
// conf = exp(z_t[t, y_r] - lse_t[t]).  Rows that take no part get logit 0 and confidence 1.
__global__ void __launch_bounds__(ROW_THREADS) target_conf_kernel(const __nv_bfloat16* Ht, long long ldHt, const __nv_bfloat16* Wt,
                                                                  long long ldWt, int d_t, const long long* labels,
                                                                  const unsigned char* valid_eff, const long long* block_start,
                                                                  int K, long long row0, int n_rows, long long lo,
                                                                  const float* lse_t_slab, float* zt_label_row, float* conf_out) {
    const int warp = (blockIdx.x * ROW_THREADS + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= n_rows) return;
    const long long r = row0 + warp;
    float zt = 0.f, c = 1.f;
    if (valid_eff[r]) {
        const long long b = r / K;
        const long long t = block_start[b] + (r - b * K);
        const uint4* h = reinterpret_cast<const uint4*>(Ht + t * ldHt);
        const uint4* w = reinterpret_cast<const uint4*>(Wt + labels[r] * ldWt);
        float acc = 0.f;
        for (int i = lane; i < d_t / 8; i += 32) {
            const uint4 a = h[i], bq = w[i];
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {bq.x, bq.y, bq.z, bq.w};
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
        zt = acc;
        c = expf(zt - lse_t_slab[t - lo]);
    }
    if (lane == 0) {
        zt_label_row[r] = zt;
        conf_out[r] = c;
    }
}

// One CTA per draft row of the slab.  Reads the row's stored draft logits z and its target
// position's stored logits z_t (fp16), forms q = exp(z - lse), p = exp(z_t - lse_t), and
//   * writes dz[v] = weight * ((1 + beta) q_v - p_v - beta [v == y]) as bf16 over z, in place
//     (the label entry from the fp32 label logits of both sides);
//   * reduces KD = sum_v p_v (z_t[v] - z[v]) - lse_t + lse in a fixed order and stores
//     weight * KD in kd_row[r].
// Rows that take no part get a zero dz row and kd_row = 0.  Traffic: 4 bytes read + 2 written per logit.
__global__ void __launch_bounds__(ROW_THREADS) z_to_dz_kernel(void* zs, const void* zts, long long ldz, const long long* labels,
                                                              const unsigned char* valid_eff, const long long* block_start, int K,
                                                              long long row0, long long lo, const float* lse,
                                                              const float* lse_t_slab, const float* weight, const float* z_label,
                                                              const float* zt_label_row, float beta, float* kd_row, int V) {
    __shared__ float s_part[ROW_THREADS / 32];
    const long long r = row0 + blockIdx.x;
    const bool ok = valid_eff[r] != 0;
    const long long b = r / K;
    const long long t = ok ? block_start[b] + (r - b * K) - lo : 0;
    const float w = ok ? weight[r] : 0.f;
    const float lse_r = ok ? lse[r] : 0.f;
    const float lse_t = ok ? lse_t_slab[t] : 0.f;
    const float l2 = ok ? lse_r * LOG2E : INFINITY;
    const float l2t = ok ? lse_t * LOG2E : INFINITY;
    const int yi = ok ? static_cast<int>(labels[r]) : -1;
    const float dz_label = ok ? w * ((1.f + beta) * expf(z_label[r] - lse_r) - beta - expf(zt_label_row[r] - lse_t)) : 0.f;
    uint4* row = reinterpret_cast<uint4*>(static_cast<unsigned short*>(zs) + static_cast<size_t>(blockIdx.x) * ldz);
    const uint4* trow = reinterpret_cast<const uint4*>(static_cast<const unsigned short*>(zts) + static_cast<size_t>(t) * ldz);
    const int groups = static_cast<int>(ldz / 8);
    const float opb = 1.f + beta;
    float cross = 0.f;
    for (int gi = threadIdx.x; gi < groups; gi += ROW_THREADS) {
        const uint4 in = __ldcs(row + gi);
        uint4 tin = make_uint4(0u, 0u, 0u, 0u);
        if (ok) tin = __ldg(trow + gi);
        const uint32_t zw[4] = {in.x, in.y, in.z, in.w}, tw[4] = {tin.x, tin.y, tin.z, tin.w};
        float f[8];
        const int col = gi * 8;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 z2 = __half22float2(*reinterpret_cast<const __half2*>(&zw[i]));
            const float2 t2 = __half22float2(*reinterpret_cast<const __half2*>(&tw[i]));
            const float zz[2] = {z2.x, z2.y}, tt[2] = {t2.x, t2.y};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = col + 2 * i + h;
                float q, p;
                asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(q) : "f"(fmaf(zz[h], LOG2E, -l2)));
                asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p) : "f"(fmaf(tt[h], LOG2E, -l2t)));
                const bool live = c < V;
                if (live) cross = fmaf(p, tt[h] - zz[h], cross);
                float v = live ? w * fmaf(opb, q, -p) : 0.f;
                if (c == yi) v = dz_label;
                f[2 * i + h] = v;
            }
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
    // fixed-order reduction of the cross term: shuffles inside each warp, then the warps in order
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cross += __shfl_down_sync(0xffffffffu, cross, off);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = cross;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
        for (int i = 0; i < ROW_THREADS / 32; ++i) tot += s_part[i];
        kd_row[r] = ok ? w * (tot - lse_t + lse_r) : 0.f;
    }
}

// Single CTA: loss_kd = (1/N) sum_r weight_r KD_r in a fixed order (fp64), and the total of
// Eq. 12, beta * loss_ce + loss_kd.  loss[0] holds loss_ce on entry (written by the forward's
// finalize kernel); on exit loss = {total, loss_ce, loss_kd}.
__global__ void __launch_bounds__(ROW_THREADS) finalize_kernel(const float* kd_row, const unsigned char* valid_eff, int T, float beta,
                                                               float* loss) {
    __shared__ double s_sum[ROW_THREADS];
    __shared__ long long s_n[ROW_THREADS];
    double acc = 0.0;
    long long n = 0;
    for (int r = threadIdx.x; r < T; r += ROW_THREADS) {
        acc += static_cast<double>(kd_row[r]);
        n += valid_eff[r] ? 1 : 0;
    }
    s_sum[threadIdx.x] = acc;
    s_n[threadIdx.x] = n;
    __syncthreads();
    for (int off = ROW_THREADS / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off) {
            s_sum[threadIdx.x] += s_sum[threadIdx.x + off];
            s_n[threadIdx.x] += s_n[threadIdx.x + off];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const float ce = loss[0];
        const float kdl = s_n[0] > 0 ? static_cast<float>(s_sum[0] / static_cast<double>(s_n[0])) : 0.f;
        loss[1] = ce;
        loss[2] = kdl;
        loss[0] = beta * ce + kdl;
    }
}

}  // namespace kd
}  // namespace cat
