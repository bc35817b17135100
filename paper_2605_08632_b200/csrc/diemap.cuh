// Which SMs share an L2 partition, found by measurement, and a numbering of the GEMM kernels' workers
// that follows it.
//
// B200 is two dies, each with its own L2 partition.  A persistent GEMM whose CTA pairs share operand
// tiles reads less from HBM, and runs faster, when the pairs that share a tile sit on the same die:
// numbered by blockIdx, the same kernels read 4.9 to 12.6 GB from DRAM per launch depending on the
// part (which SMs are fused off decides where consecutive clusters land); numbered die by die they
// read 4.7 to 6.6 GB.  CUDA does not say which SM is on which die, so it is measured once per
// device: an atomic on global memory is carried out in the L2 partition that the line's address
// belongs to, so from one die it takes about 350 cycles and from the other about 700.  Every SM times
// atomics on the same few dozen lines; two SMs are on the same die when they see the same lines
// near.  The result is a table worker_of_tpc[smid >> 1] (a CTA pair occupies the two SMs of one TPC):
// TPCs of one die first, then the other's.  Neighbouring worker indices share operand tiles in the
// kernels' schedules, so that is all the schedules need.
//
// The table is advice only.  Each pair claims its worker index with an atomic and moves on to the
// next free one when the index is taken (see claim_worker), so a wrong or missing table, or two
// pairs that run on the same TPC one after the other, costs locality, never correctness.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace cat {
namespace die {

constexpr int MAX_SM = 256;
constexpr int N_LINES = 32;            // lines timed per SM
constexpr int N_TRIES = 3;             // best of
constexpr int CHAIN = 4;               // dependent atomics per timing
constexpr int MIN_GAP = 120;           // cycles between the near and the far cluster of a usable line

struct Map {
    int valid;                          // 1 once worker_of_tpc is final (written last)
    int n_tpc;                          // TPCs = CTA pairs the table covers
    int n_die0;                         // TPCs in the class of the first SM
    int worker_of_tpc[MAX_SM / 2];
};

__device__ Map g_map;
__device__ int g_claimed[MAX_SM];
__device__ unsigned short g_lat[MAX_SM * N_LINES];

__device__ __forceinline__ unsigned smid() {
    unsigned r;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(r));
    return r;
}

// One thread per SM (the first CTA to arrive on it) times CHAIN dependent atomic adds of zero on each line;
// `lines` is any device buffer of at least N_LINES * stride_words words whose contents must survive (adding
// zero leaves them as they are).
__global__ void probe_kernel(unsigned* lines, size_t stride_words, int n_sm) {
    if (threadIdx.x != 0) return;
    const unsigned s = smid();
    if (s >= static_cast<unsigned>(n_sm) || s >= MAX_SM || atomicCAS(&g_claimed[s], 0, 1) != 0) return;
    for (int i = 0; i < N_LINES; ++i) {
        unsigned best = 65535u;
        unsigned* p = lines + static_cast<size_t>(i) * stride_words;
        for (int t = 0; t < N_TRIES; ++t) {
            unsigned v = 0;
            const long long t0 = clock64();
#pragma unroll 1
            for (int c = 0; c < CHAIN; ++c)
                asm volatile("atom.global.add.u32 %0, [%1], 0;" : "=r"(v) : "l"(p + (v & 7u)) : "memory");   // the next address waits for the result
            __threadfence();
            const long long dt = (clock64() - t0) / CHAIN;
            const unsigned d = dt > 65535 ? 65535u : static_cast<unsigned>(dt);
            best = d < best ? d : best;
        }
        g_lat[s * N_LINES + i] = static_cast<unsigned short>(best);
    }
}

// One thread: classes from the latencies, table from the classes.  Leaves valid = 0 when the picture is not
// clean (an SM that did not report, lines without two clusters, a TPC whose SMs disagree, one class only).
__global__ void classify_kernel(int n_sm) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const int n_tpc = n_sm / 2;
    bool ok = n_sm >= 2 && n_sm <= MAX_SM && (n_sm % 2) == 0;
    for (int s = 0; ok && s < n_sm; ++s) ok = g_claimed[s] == 1;
    int thr[N_LINES];
    int usable = 0;
    for (int i = 0; ok && i < N_LINES; ++i) {
        int mn = 65535, mx = 0;
        for (int s = 0; s < n_sm; ++s) {
            const int v = g_lat[s * N_LINES + i];
            mn = v < mn ? v : mn;
            mx = v > mx ? v : mx;
        }
        thr[i] = mx - mn >= MIN_GAP ? (mn + mx) / 2 : -1;
        usable += thr[i] >= 0;
    }
    ok = ok && usable >= N_LINES / 2;
    int cls[MAX_SM];
    int n1 = 0;
    for (int s = 0; ok && s < n_sm; ++s) {
        int same = 0;
        for (int i = 0; i < N_LINES; ++i)
            if (thr[i] >= 0) same += (g_lat[s * N_LINES + i] > thr[i]) == (g_lat[i] > thr[i]);     // against SM 0
        if (same * 8 >= usable * 7) cls[s] = 0;
        else if (same * 8 <= usable) cls[s] = 1;
        else ok = false;                                                                           // neither clearly alike nor clearly opposite
        n1 += ok && cls[s] == 1;
    }
    for (int t = 0; ok && t < n_tpc; ++t) ok = cls[2 * t] == cls[2 * t + 1];
    ok = ok && n1 > 0 && n1 < n_sm;
    if (ok) {
        int rank = 0;
        for (int c = 0; c < 2; ++c)
            for (int t = 0; t < n_tpc; ++t)
                if (cls[2 * t] == c) g_map.worker_of_tpc[t] = rank++;
        g_map.n_tpc = n_tpc;
        g_map.n_die0 = (n_sm - n1) / 2;
        __threadfence();
        g_map.valid = 1;
    } else {
        g_map.n_tpc = 0;
        g_map.valid = -1;               // measured, not usable
    }
}

// Worker index of a CTA pair: the table's suggestion for this pair's TPC when there is one for exactly this
// many pairs, else blockIdx order; then the first index from there on that nobody has claimed in this launch.
// claims[i] == serial means index i is taken (serial is unique per launch, never 0).
__device__ __forceinline__ int claim_worker(int* claims, int serial, int by_block, int n_workers) {
    int pref = by_block;
    if (g_map.valid == 1 && g_map.n_tpc == n_workers) {
        const unsigned t = smid() >> 1;
        if (t < MAX_SM / 2) {
            const int w = g_map.worker_of_tpc[t];
            if (w >= 0 && w < n_workers) pref = w;
        }
    }
    int id = pref;
    for (int tries = 0; tries < n_workers; ++tries) {
        if (atomicExch(&claims[id], serial) != serial) return id;
        id = id + 1 == n_workers ? 0 : id + 1;
    }
    return by_block;                    // not reached: there are as many indices as pairs
}

}  // namespace die
}  // namespace cat
