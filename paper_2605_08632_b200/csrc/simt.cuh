// fp32 path ("fp32 throughout"): the same three contractions and epilogues as the tensor-core
// path, on plain FFMA with precise expf/logf.  It serves fp32 inputs, which the bf16 tensor
// cores cannot take without changing the arithmetic.  64x64 output tile per CTA, 16-deep
// k-slices staged in shared memory, 4x4 outputs per thread.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace cat {
namespace simt {

constexpr int TM = 64, TN = 64, TK = 16, THREADS = 256;

struct Operands {
    const float* A;   // element (m, k) at A[m * sAm + k * sAk]
    const float* B;   // element (k, n) at B[k * sBk + n * sBn]
    long long sAm, sAk, sBk, sBn;
    int M, N, Kd;     // output rows, output columns, contraction length
    int n_groups;     // gridDim.y; group g covers n-tiles [g*nt/n_groups, (g+1)*nt/n_groups)
};

enum { MODE_FWD = 0, MODE_DZ = 1, MODE_OUT = 2 };

struct EpiParams {
    // MODE_FWD
    const long long* labels;
    float* part_m;
    float* part_l;
    float* z_label;
    // MODE_DZ
    const unsigned char* valid;
    const float* lse;
    const float* weight;
    float* dz;
    long long ld_dz;
    int V;      // full vocabulary size (label range check)
    int v0;     // vocabulary index of column 0 of this launch
    // MODE_OUT
    const float* alpha;
    const float* add;
    float* out;
    long long ld_add, ld_out;
};

template <int MODE>
__global__ void __launch_bounds__(THREADS) gemm_kernel(const Operands op, const EpiParams ep) {
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.x * TM;
    const int n_tiles = (op.N + TN - 1) / TN;
    const int g = blockIdx.y;
    const int nt_begin = static_cast<int>((static_cast<long long>(g) * n_tiles) / op.n_groups);
    const int nt_end = static_cast<int>((static_cast<long long>(g + 1) * n_tiles) / op.n_groups);

    // per-row state (rows ty*4 + i), replicated over the 16 threads that share a row
    float m_run[4], l_run[4], w_row[4], lse_row[4];
    int y_row[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = m0 + ty * 4 + i;
        m_run[i] = -INFINITY; l_run[i] = 0.f; w_row[i] = 0.f; lse_row[i] = INFINITY; y_row[i] = -1;
        if (MODE != MODE_OUT && row < op.M) {
            const long long y = ep.labels[row];
            const bool y_ok = y >= 0 && y < ep.V;
            if (MODE == MODE_FWD) {
                if (y_ok) y_row[i] = static_cast<int>(y);
            } else {
                const bool ok = y_ok && (ep.valid == nullptr || ep.valid[row] != 0);
                if (ok) { y_row[i] = static_cast<int>(y) - ep.v0; w_row[i] = ep.weight[row]; lse_row[i] = ep.lse[row]; }
            }
        }
    }
    const float alpha = (MODE == MODE_OUT && ep.alpha) ? *ep.alpha : 1.f;

    for (int nt = nt_begin; nt < nt_end; ++nt) {
        const int n0 = nt * TN;
        float acc[4][4] = {};
        for (int k0 = 0; k0 < op.Kd; k0 += TK) {
            // stage a TK x TM slice of A and a TK x TN slice of B
            for (int e = tid; e < TK * TM; e += THREADS) {
                const int kk = e & (TK - 1), mm = e >> 4;
                const int m = m0 + mm, k = k0 + kk;
                As[kk][mm] = (m < op.M && k < op.Kd) ? op.A[m * op.sAm + k * op.sAk] : 0.f;
            }
            for (int e = tid; e < TK * TN; e += THREADS) {
                const int kk = e & (TK - 1), nn = e >> 4;
                const int n = n0 + nn, k = k0 + kk;
                Bs[kk][nn] = (n < op.N && k < op.Kd) ? op.B[k * op.sBk + n * op.sBn] : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < TK; ++kk) {
                float a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
                for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
            __syncthreads();
        }

        if (MODE == MODE_FWD) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = m0 + ty * 4 + i;
                float cmax = -INFINITY;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int col = n0 + tx * 4 + j;
                    if (col < op.N) cmax = fmaxf(cmax, acc[i][j]);
                    if (col == y_row[i]) ep.z_label[row] = acc[i][j];
                }
#pragma unroll
                for (int off = 1; off < 16; off <<= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, off));
                const float m_new = fmaxf(m_run[i], cmax);
                float sum = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int col = n0 + tx * 4 + j;
                    if (col < op.N) sum += expf(acc[i][j] - m_new);
                }
#pragma unroll
                for (int off = 1; off < 16; off <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                l_run[i] = l_run[i] * expf(m_run[i] - m_new) + sum;
                m_run[i] = m_new;
            }
        } else if (MODE == MODE_DZ) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = m0 + ty * 4 + i;
                if (row >= op.M) continue;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int col = n0 + tx * 4 + j;
                    if (col >= op.N) continue;
                    float pz = expf(acc[i][j] - lse_row[i]);
                    if (col == y_row[i]) pz -= 1.f;
                    ep.dz[row * ep.ld_dz + col] = w_row[i] * pz;
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = m0 + ty * 4 + i;
                if (row >= op.M) continue;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int col = n0 + tx * 4 + j;
                    if (col >= op.N) continue;
                    float v = alpha * acc[i][j];
                    if (ep.add) v += ep.add[row * ep.ld_add + col];
                    ep.out[row * ep.ld_out + col] = v;
                }
            }
        }
    }
    if (MODE == MODE_FWD && tx == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = m0 + ty * 4 + i;
            if (row < op.M) {
                ep.part_m[static_cast<size_t>(g) * op.M + row] = m_run[i];
                ep.part_l[static_cast<size_t>(g) * op.M + row] = l_run[i];
            }
        }
    }
}

}  // namespace simt
}  // namespace cat
