// Persistent, warp-specialised bf16 GEMM for sm_100a: TMA-fed shared-memory ring,
// tcgen05.mma with fp32 accumulators in tensor memory (two 128x256 accumulators, so the
// epilogue of one tile overlaps the main loop of the next), and pluggable epilogues that
// read the accumulators straight from TMEM, one output row per thread.
//
// The three dense contractions of the CAT loss all run through this kernel:
//   logits        z  = H W^T          A = H  (K-major),  B = W   (K-major)   forward + recompute
//   dW slice      dW = dz^T H         A = dz (MN-major), B = H   (MN-major)
//   dH            dH += dz W          A = dz (K-major),  B = W   (MN-major)
// Operands are never transposed in memory: MN-major operands are described to the tensor
// core through the shared-memory descriptor's leading/stride offsets and the instruction
// descriptor's major bits.
//
// Warp roles (192 threads): warp 0 = TMA producer (one lane), warp 1 = TMEM owner and MMA
// issuer (one lane), warps 2-5 = epilogue (TMEM lane quarter = warp index mod 4).
// Every mbarrier wait is bounded; when one expires the CTA raises an abort flag, records
// CAT_ERR_TIMEOUT in the status word, drains what it issued, frees its TMEM and returns.
#pragma once
#include "ptx.cuh"
#include "diemap.cuh"
#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace cat {
namespace tc {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int MAX_STAGES = 8;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr int MN_ATOM_BYTES = 64 * BK * 2;                // one 64(MN) x BK box of an MN-major operand
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // default limit of a wait (Sched::wait_ns)
constexpr unsigned long long DRAIN_LIMIT_NS = 20000000ull;    // after an abort: how long issued copies / MMAs get to land
constexpr int STATUS_TIMEOUT = -8;                        // CAT_ERR_TIMEOUT
constexpr float LOG2E = 1.4426950408889634f;

// Static tile schedule shared by the three roles of a CTA.
struct Sched {
    int num_m_tiles;   // tiles of BM rows of the output
    int num_n_tiles;   // tiles of BN columns of the output
    int num_kb;        // ring stages (BK * k-slices per stage) along the contraction
    int n_groups;      // column groups per m-tile: one item = (m-tile, group); a group is a run of n-tiles
    int band_m;        // m-tiles per band when m runs fastest (keeps a band of A rows L2-resident)
    int n_fastest;     // 1: items ordered group-fastest within an m-tile; 0: m-fastest within (band, group)
    int n_items;       // num_m_tiles * n_groups
    unsigned long long wait_ns;   // limit of every mbarrier wait in the kernel
    int* claims;       // CTA pairs: worker indices taken in this launch (>= gridDim.x / 2 ints), or nullptr = blockIdx order
    int serial;        // this launch's mark in `claims`, unique per launch and not 0
};

__device__ __forceinline__ void decode_item(const Sched& s, int item, int& m_tile, int& group, int& n_begin, int& n_end) {
    if (s.n_fastest) {
        m_tile = item / s.n_groups;
        group = item - m_tile * s.n_groups;
    } else {
        const int per_band = s.band_m * s.n_groups;
        const int band = item / per_band;
        const int rem = item - band * per_band;
        const int mb = min(s.band_m, s.num_m_tiles - band * s.band_m);
        group = rem / mb;
        m_tile = band * s.band_m + (rem - group * mb);
    }
    n_begin = static_cast<int>((static_cast<long long>(group) * s.num_n_tiles) / s.n_groups);
    n_end = static_cast<int>((static_cast<long long>(group + 1) * s.num_n_tiles) / s.n_groups);
}

struct Ctl {
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    unsigned long long drain;
    uint32_t tmem_base;
    uint32_t worker;
    volatile int abort;
};

// Waits for phase `parity` of an mbarrier, at most `limit_ns`.  A wait that runs out raises the CTA's abort
// flag and records CAT_ERR_TIMEOUT; a wait that sees the flag raised by another role gives up at once.
// DRAIN = true is for the clean-up after an abort: the flag is already up, so it is neither heeded nor
// set, and the wait simply ends when the barrier completes or the limit passes.
template <bool DRAIN = false>
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort, int* status,
                                             unsigned long long limit_ns) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    while (true) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (!DRAIN && *abort) return false;
            const unsigned long long now = ptx::globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
                if (!DRAIN) {
                    *abort = 1;
                    atomicExch(status, STATUS_TIMEOUT);
                }
                return false;
            }
        }
    }
}

// Per-warp staging of 16-bit output tiles.  An epilogue thread owns one row, so a direct global
// store makes every lane of a warp write a different row: 32 scattered 16-byte pieces per
// instruction, which at a short contraction (d = 1024) held the logits GEMM at 70 % tensor
// activity.  Instead the lanes write their pieces into a shared-memory tile of 32 rows x 64 columns
// (128-byte rows, 128-byte swizzle, so the 8 lanes of a store phase hit different banks) and lane 0
// sends the tile to global memory with one TMA store, which writes whole 128-byte lines and clips
// rows / columns outside the tensor.  Two tiles per warp alternate; a tile is reused once the
// store issued from it has read it (cp.async.bulk.wait_group.read).
constexpr int OUT_TILE_BYTES = 32 * 128;
constexpr int OUT_STAGE_BYTES = 4 * 2 * OUT_TILE_BYTES;      // four epilogue warps, two tiles each
struct OutStage {
    const CUtensorMap* tm;
    uint32_t buf;      // shared-memory address of this warp's two tiles
    int row0;          // tensor row of this warp's lane 0
    int n_rows;        // rows of the tensor: a tile that starts at or past it is not sent
    int lane;
    int sel;
    __device__ __forceinline__ void begin() {
        if (lane == 0) ptx::tma_store_wait_read<1>();     // the store before last (same tile) has read it
        __syncwarp();
    }
    // 16-byte piece `j` (0..7) of this lane's 128-byte row
    __device__ __forceinline__ void put(int j, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
        ptx::st_shared_v4(buf + sel * OUT_TILE_BYTES + lane * 128 + ((j ^ (lane & 7)) << 4), a, b, c, d);
    }
    __device__ __forceinline__ void flush(int x, bool add = false) {
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < n_rows) {
            if (add) ptx::tma_reduce_add_2d(tm, buf + sel * OUT_TILE_BYTES, x, row0);
            else ptx::tma_store_2d(tm, buf + sel * OUT_TILE_BYTES, x, row0);
            ptx::tma_store_commit();
        }
        sel ^= 1;
    }
    __device__ __forceinline__ void finish() {
        if (lane == 0) ptx::tma_store_wait_all();
        __syncwarp();
    }
};

// ------------------------------------------------------------------------------------------
// Epilogues.  Each epilogue thread owns output row (m_tile*BM + row_in_tile) and walks the
// 256 accumulator columns of a tile in chunks of 32 (one tcgen05.ld each).  taddr is the TMEM
// address of column 0 of the tile for this warp's lane quarter.
// ------------------------------------------------------------------------------------------

// Forward: online max / sum-exp over the vocabulary (softmax partition function of Eq. 11's
// log P), and the label logit z[r, y_r] picked from the accumulator chunk that holds it.
// STORE = 1 additionally writes the logits of the tile as fp16 (saturating) into a row slab
// (the distillation path, which needs the logits of both models side by side).
// STORE = 2 writes e[r, v] = exp(z[r, v] - ref[r]) as bf16 instead: softmax numerators relative to
// a per-row reference fixed before the GEMM (the row's label logit), so that later
// softmax[r, v] = exp(ref[r] - lse[r]) * e[r, v] needs only a per-row factor, which the dH / dW
// GEMMs absorb, and no second pass over the slab.  e is formed as exp(z - m) * exp(m - ref) with m the
// running maximum, the second factor's exponent capped at EXP_CAP_LOG2, so e stays finite whatever
// the inputs.
constexpr float EXP_CAP_LOG2 = 115.0f;   // 2^115 = e^79.7

template <int STORE>
struct EpiFwdT {
    struct Params {
        const long long* labels;   // [T]
        float* part_m;             // [n_groups][part_stride] running max of each (row, vocabulary split)
        float* part_l;             // [n_groups][part_stride] sum exp(z - max)
        float* z_label;            // [T]
        __half* zs;                // [T][ldz] 16-bit slab: fp16 logits (STORE 1) or bf16 exp(z - ref) (STORE 2)
        const float* ref;          // [T] per-row reference (STORE 2 only)
        long long ldz;
        long long part_stride;
        int T;
        int V;
    };
    struct State {
        float m_run, l_run;
        float ref2;                // ref[row] * log2(e)
        int y;
        int row;
    };
    __device__ static __forceinline__ void begin_item(const Params& p, State& s, int m_tile, int row_in_tile) {
        s.row = m_tile * BM + row_in_tile;
        s.m_run = -INFINITY;
        s.l_run = 0.f;
        s.ref2 = 0.f;
        s.y = -1;
        if (s.row < p.T) {
            const long long y = p.labels[s.row];
            if (y >= 0 && y < p.V) s.y = static_cast<int>(y);
            if (STORE == 2) s.ref2 = p.ref[s.row] * LOG2E;
        }
    }
    __device__ static __forceinline__ void tile(const Params& p, State& s, int n_tile, uint32_t taddr, OutStage& o) {
        const int col0 = n_tile * BN;
        const int ncols = min(BN, p.V - col0);
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            if (c * 32 >= ncols) break;
            const bool closes_pair = (c & 1) != 0 || (c + 1) * 32 >= ncols;   // last chunk of its 64-column staging tile
            if (STORE != 0 && (c & 1) == 0) o.begin();
            uint32_t v[32];
            ptx::tmem_ld_32x32(taddr + c * 32, v);
            ptx::tmem_ld_wait();
            float f[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(v[i]);
            const int live = ncols - c * 32;
            if (live < 32) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i >= live) f[i] = -INFINITY;
            }
            if (STORE == 1) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    o.put((c & 1) * 4 + q, ptx::pack_f16x2_sat(f[q * 8 + 0], f[q * 8 + 1]), ptx::pack_f16x2_sat(f[q * 8 + 2], f[q * 8 + 3]),
                          ptx::pack_f16x2_sat(f[q * 8 + 4], f[q * 8 + 5]), ptx::pack_f16x2_sat(f[q * 8 + 6], f[q * 8 + 7]));
                if (closes_pair) o.flush(col0 + (c >> 1) * 64);
            }
            const int rel = s.y - (col0 + c * 32);
            if (rel >= 0 && rel < 32) {
                float zy = 0.f;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i == rel) zy = f[i];
                p.z_label[s.row] = zy;
            }
            float cmax = ptx::max3_f32(f[0], f[1], f[2]);
#pragma unroll
            for (int i = 3; i + 1 < 32; i += 2) cmax = ptx::max3_f32(cmax, f[i], f[i + 1]);
            cmax = fmaxf(cmax, f[31]);
            const float m_new = fmaxf(s.m_run, cmax);
            const float mb = m_new * LOG2E;
            float sum = 0.f;
            if (STORE == 2) {
                // One exponential per logit serves both uses: exp(z - m) for the running sum, and
                // exp(z - ref) = exp(z - m) * exp(m - ref) for the slab (the factor capped so that the product
                // stays finite).  The scale, sum and product run on packed fp32 pairs.
                const uint64_t l2e2 = ptx::pack_f32x2(LOG2E, LOG2E), nmb2 = ptx::pack_f32x2(-mb, -mb);
                const float fac = ptx::ex2_approx(fminf(mb - s.ref2, EXP_CAP_LOG2));
                const uint64_t fac2 = ptx::pack_f32x2(fac, fac);
                uint64_t sum2 = ptx::pack_f32x2(0.f, 0.f);
                uint32_t packed[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float x0, x1;
                    ptx::unpack_f32x2(ptx::fma_f32x2(ptx::pack_f32x2(f[2 * i], f[2 * i + 1]), l2e2, nmb2), x0, x1);
                    const uint64_t e2 = ptx::pack_f32x2(ptx::ex2_approx(x0), ptx::ex2_approx(x1));
                    sum2 = ptx::add_f32x2(sum2, e2);
                    float y0, y1;
                    ptx::unpack_f32x2(ptx::mul_f32x2(e2, fac2), y0, y1);
                    packed[i] = ptx::pack_bf16x2(y0, y1);
                }
                float s0, s1;
                ptx::unpack_f32x2(sum2, s0, s1);
                sum = s0 + s1;
#pragma unroll
                for (int q = 0; q < 4; ++q) o.put((c & 1) * 4 + q, packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                if (closes_pair) o.flush(col0 + (c >> 1) * 64);
            } else {
                const uint64_t l2e2 = ptx::pack_f32x2(LOG2E, LOG2E), nmb2 = ptx::pack_f32x2(-mb, -mb);
                uint64_t sum2 = ptx::pack_f32x2(0.f, 0.f);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float x0, x1;
                    ptx::unpack_f32x2(ptx::fma_f32x2(ptx::pack_f32x2(f[2 * i], f[2 * i + 1]), l2e2, nmb2), x0, x1);
                    sum2 = ptx::add_f32x2(sum2, ptx::pack_f32x2(ptx::ex2_approx(x0), ptx::ex2_approx(x1)));
                }
                float s0, s1;
                ptx::unpack_f32x2(sum2, s0, s1);
                sum = s0 + s1;
            }
            s.l_run = fmaf(s.l_run, ptx::ex2_approx((s.m_run - m_new) * LOG2E), sum);
            s.m_run = m_new;
        }
    }
    __device__ static __forceinline__ int out_rows(const Params& p) { return STORE != 0 ? p.T : 0; }
    __device__ static __forceinline__ void end_item(const Params& p, const State& s, int group) {
        if (s.row < p.T) {
            p.part_m[static_cast<size_t>(group) * p.part_stride + s.row] = s.m_run;
            p.part_l[static_cast<size_t>(group) * p.part_stride + s.row] = s.l_run;
        }
    }
};
using EpiFwd = EpiFwdT<0>;
using EpiFwdStore = EpiFwdT<1>;
using EpiFwdExp = EpiFwdT<2>;

// Backward recompute: dz[r, v] = weight_r * (exp(z - lse_r) - [v == y_r]) as a bf16 tile of the
// current vocabulary slab (the scalar g/N is applied later, in fp32, by the dH / dW epilogues).
struct EpiDz {
    struct Params {
        const long long* labels;   // [T]
        const unsigned char* valid;  // [T] or nullptr
        const float* lse;          // [T]
        const float* weight;       // [T]
        __nv_bfloat16* dz;         // [T][ld] slab, column 0 = vocabulary index v0
        long long ld;
        int T;
        int V;
        int v0;
    };
    struct State {
        float w, l2;
        int y_rel;
        int row;
    };
    __device__ static __forceinline__ void begin_item(const Params& p, State& s, int m_tile, int row_in_tile) {
        s.row = m_tile * BM + row_in_tile;
        s.w = 0.f;
        s.l2 = INFINITY;
        s.y_rel = -1;
        if (s.row < p.T) {
            const long long y = p.labels[s.row];
            const bool ok = (p.valid == nullptr || p.valid[s.row] != 0) && y >= 0 && y < p.V;
            if (ok) {
                s.w = p.weight[s.row];
                s.l2 = p.lse[s.row] * LOG2E;
                s.y_rel = static_cast<int>(y) - p.v0;
            }
        }
    }
    __device__ static __forceinline__ void tile(const Params& p, State& s, int n_tile, uint32_t taddr, OutStage& o) {
        const int col0 = n_tile * BN;
        const int ncols = min(BN, p.V - p.v0 - col0);
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            if (c * 32 >= ncols) break;                     // columns past the vocabulary are never read back
            if ((c & 1) == 0) o.begin();
            uint32_t v[32];
            ptx::tmem_ld_32x32(taddr + c * 32, v);
            ptx::tmem_ld_wait();
            float f[32];
            const int live = ncols - c * 32;
            {   // w * exp2(z * log2e - lse * log2e) on packed fp32 pairs
                const uint64_t l2e2 = ptx::pack_f32x2(LOG2E, LOG2E), nl2 = ptx::pack_f32x2(-s.l2, -s.l2), w2 = ptx::pack_f32x2(s.w, s.w);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float x0, x1;
                    ptx::unpack_f32x2(ptx::fma_f32x2(ptx::pack_f32x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])), l2e2, nl2), x0, x1);
                    ptx::unpack_f32x2(ptx::mul_f32x2(ptx::pack_f32x2(ptx::ex2_approx(x0), ptx::ex2_approx(x1)), w2), f[2 * i], f[2 * i + 1]);
                }
            }
            if (live < 32) {   // ragged last tile of the vocabulary
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i >= live) f[i] = 0.f;
            }
            const int rel = s.y_rel - (col0 + c * 32);
            if (rel >= 0 && rel < 32) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i == rel) f[i] -= s.w;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                o.put((c & 1) * 4 + q, ptx::pack_bf16x2(f[q * 8 + 0], f[q * 8 + 1]), ptx::pack_bf16x2(f[q * 8 + 2], f[q * 8 + 3]),
                      ptx::pack_bf16x2(f[q * 8 + 4], f[q * 8 + 5]), ptx::pack_bf16x2(f[q * 8 + 6], f[q * 8 + 7]));
            if ((c & 1) != 0 || (c + 1) * 32 >= ncols) o.flush(col0 + (c >> 1) * 64);
        }
    }
    __device__ static __forceinline__ int out_rows(const Params& p) { return p.T; }
    __device__ static __forceinline__ void end_item(const Params&, const State&, int) {}
};

// Plain output: out = add + alpha * acc, fp32 or bf16, with optional fp32/bf16 addend
// (dH accumulation across vocabulary slabs, accumulate_dW).
struct EpiOut {
    struct Params {
        const float* alpha;            // device scalar or nullptr (= 1)
        const float* row_scale;        // [M] per-output-row factor or nullptr (= 1)
        const float* add_f32;          // [M][ld_add] or nullptr
        const __nv_bfloat16* add_bf16; // [M][ld_add] or nullptr
        float* out_f32;                // [M][ld_out] or nullptr
        __nv_bfloat16* out_bf16;       // [M][ld_out] or nullptr
        long long ld_add, ld_out;
        int M, N;
        int staged;                    // 1: fp32 output, no addend or the output itself as addend: tiles of
                                       //    32 x 32 go through shared memory and a TMA store / reduce-add
    };
    struct State {
        float alpha;
        int row;
    };
    __device__ static __forceinline__ void begin_item(const Params& p, State& s, int m_tile, int row_in_tile) {
        s.row = m_tile * BM + row_in_tile;
        s.alpha = p.alpha ? *p.alpha : 1.f;
        if (p.row_scale && s.row < p.M) s.alpha *= p.row_scale[s.row];
    }
    __device__ static __forceinline__ void tile(const Params& p, State& s, int n_tile, uint32_t taddr, OutStage& o) {
        const int col0 = n_tile * BN;
        const bool row_ok = s.row < p.M;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            if (col0 + c * 32 >= p.N) break;
            if (p.staged) o.begin();
            uint32_t v[32];
            ptx::tmem_ld_32x32(taddr + c * 32, v);
            ptx::tmem_ld_wait();
            if (p.staged) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    o.put(j, __float_as_uint(s.alpha * __uint_as_float(v[4 * j])), __float_as_uint(s.alpha * __uint_as_float(v[4 * j + 1])),
                          __float_as_uint(s.alpha * __uint_as_float(v[4 * j + 2])), __float_as_uint(s.alpha * __uint_as_float(v[4 * j + 3])));
                o.flush(col0 + c * 32, p.add_f32 != nullptr);
                continue;
            }
            if (!row_ok) continue;
            const int cbase = col0 + c * 32;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int col = cbase + q * 8;
                if (col + 8 > p.N) continue;   // N is a multiple of 8: groups are all-in or all-out
                float f[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = s.alpha * __uint_as_float(v[q * 8 + i]);
                if (p.add_f32) {
                    const float4* a = reinterpret_cast<const float4*>(p.add_f32 + static_cast<size_t>(s.row) * p.ld_add + col);
                    const float4 a0 = a[0], a1 = a[1];
                    f[0] += a0.x; f[1] += a0.y; f[2] += a0.z; f[3] += a0.w;
                    f[4] += a1.x; f[5] += a1.y; f[6] += a1.z; f[7] += a1.w;
                } else if (p.add_bf16) {
                    const uint4 a = *reinterpret_cast<const uint4*>(p.add_bf16 + static_cast<size_t>(s.row) * p.ld_add + col);
                    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
                        f[2 * i] += t.x;
                        f[2 * i + 1] += t.y;
                    }
                }
                if (p.out_f32) {
                    float4* o = reinterpret_cast<float4*>(p.out_f32 + static_cast<size_t>(s.row) * p.ld_out + col);
                    o[0] = make_float4(f[0], f[1], f[2], f[3]);
                    o[1] = make_float4(f[4], f[5], f[6], f[7]);
                } else {
                    uint4 pk;
                    __nv_bfloat162 b0 = __floats2bfloat162_rn(f[0], f[1]);
                    __nv_bfloat162 b1 = __floats2bfloat162_rn(f[2], f[3]);
                    __nv_bfloat162 b2 = __floats2bfloat162_rn(f[4], f[5]);
                    __nv_bfloat162 b3 = __floats2bfloat162_rn(f[6], f[7]);
                    pk.x = *reinterpret_cast<uint32_t*>(&b0);
                    pk.y = *reinterpret_cast<uint32_t*>(&b1);
                    pk.z = *reinterpret_cast<uint32_t*>(&b2);
                    pk.w = *reinterpret_cast<uint32_t*>(&b3);
                    *reinterpret_cast<uint4*>(p.out_bf16 + static_cast<size_t>(s.row) * p.ld_out + col) = pk;
                }
            }
        }
    }
    __device__ static __forceinline__ int out_rows(const Params& p) { return p.staged ? p.M : 0; }
    __device__ static __forceinline__ void end_item(const Params&, const State&, int) {}
};

// ------------------------------------------------------------------------------------------
// The kernel.  tmA / tmB are 2-D tiled tensor maps with 128-byte swizzle:
//   K-major operand  [rows = M or N][cols = K]: box {BK, rows of the tile this CTA loads};
//   MN-major operand [rows = K][cols = M or N]: box {64, BK}, one box per 64 rows of the tile.
// Rows/columns past the tensor's extent are zero-filled by TMA, which makes ragged M, N and K
// contribute exact zeros.
//
// CG = 1: one CTA per 128 x 256 output tile.
// CG = 2: a cluster of two CTAs shares a 256 x 256 output tile (tcgen05 cta_group::2).  CTA
//   `rank` of the pair loads the A rows of its own 128-row half and half of the B tile (128 of
//   the 256 columns): 32 KB per 64-wide k-slice instead of 48 KB per CTA.  A ring stage holds
//   two k-slices (64 KB, three stages): the MMA-issuing thread then pays the per-stage
//   bookkeeping (commit, barrier wait, fence), which sits on the tensor pipe's critical path,
//   once per eight MMAs instead of four.  The leader (rank 0) issues every MMA; each CTA's accumulator half (its 128 rows x
//   256 columns) lives in its own TMEM and is drained by its own epilogue warps.  Barrier
//   wiring: `full` lives in the leader and counts the bytes of both CTAs' loads; `empty` and
//   `tfull` are signalled in both CTAs at once by the leader's tcgen05.commit; `tempty` lives in
//   the leader and collects one arrival per epilogue warp of both CTAs.
// ------------------------------------------------------------------------------------------
// one TMA box; in pair mode the byte count may be signalled on the peer's barrier
template <int CG>
__device__ __forceinline__ void load_box(uint32_t dst, const CUtensorMap* m, int x, int y, uint32_t bar) {
    if (CG == 1) ptx::tma_load_2d(dst, m, x, y, bar);
    else ptx::tma_load_2d_pair(dst, m, x, y, bar);
}

constexpr int PAIR_KSLICES = 2;   // BK-wide k-slices per ring stage in pair mode (1: six 32 KB stages, 2: three 64 KB stages)

template <int CG>
struct Geo {
    static constexpr int KS = CG == 1 ? 1 : PAIR_KSLICES;        // k-slices of BK per stage
    static constexpr int STAGES = CG == 1 ? 4 : 6 / KS;
    static constexpr int BN_CTA = BN / CG;                        // B-tile rows this CTA loads
    static constexpr int B_SLICE_BYTES = BN_CTA * BK * 2;
    static constexpr int A_BYTES = A_STAGE_BYTES * KS;
    static constexpr int B_BYTES = B_SLICE_BYTES * KS;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
    static constexpr int SMEM_BYTES = RING_BYTES + OUT_STAGE_BYTES + 1024;   // + slack to align the ring to 1024 B
    static constexpr int TILE_M = BM * CG;                        // output rows per scheduled m-tile
};

// Set-up shared by every CTA of the kernels below: barriers, the abort flag, TMEM (warp 1 owns it).
// On return the barriers exist in both CTAs of a pair and ctl.tmem_base is valid.
template <int CG>
__device__ __forceinline__ void cta_begin(Ctl& ctl, int n_stages, int warp) {
    if (threadIdx.x == 0) {
        for (int i = 0; i < n_stages; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctl.full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctl.empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctl.tfull[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctl.tempty[i]), CG == 1 ? NUM_THREADS - 64 : 2 * (NUM_THREADS - 64) / 32);
        }
        ptx::mbar_init(ptx::smem_u32(&ctl.drain), 1);
        ctl.abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        if (CG == 1) {
            ptx::tmem_alloc<TMEM_COLS>(ptx::smem_u32(&ctl.tmem_base));
            ptx::tmem_relinquish();
        } else {
            ptx::tmem_alloc_pair<TMEM_COLS>(ptx::smem_u32(&ctl.tmem_base));
            ptx::tmem_relinquish_pair();
        }
    }
    ptx::tc_fence_before();
    if (CG == 1) __syncthreads();
    else ptx::cluster_sync_all();     // the peer's barriers must exist before anything signals them
    ptx::tc_fence_after();
}

// Teardown, also after an abort.  Nothing of a pair may leave while its peer can still signal its
// barriers or read its shared memory, so the pair meets here before TMEM is returned.
template <int CG>
__device__ __forceinline__ void cta_end(int warp, uint32_t tmem) {
    ptx::tc_fence_before();
    if (CG == 1) __syncthreads();
    else ptx::cluster_sync_all();
    if (warp == 1) {
        ptx::tc_fence_after();
        if (CG == 1) ptx::tmem_dealloc<TMEM_COLS>(tmem);
        else ptx::tmem_dealloc_pair<TMEM_COLS>(tmem);
    }
}

template <int A_MN, int B_MN, class Epi, int CG>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmOut, const Sched sched, const typename Epi::Params ep, int* status) {
    using G = Geo<CG>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ Ctl ctl;
    const uint32_t ring = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = CG == 2 ? ptx::cluster_ctarank() : 0u;
    const bool leader = rank == 0;
    const int n_workers = gridDim.x / CG;        // a worker is a CTA (CG = 1) or a CTA pair (CG = 2)
    int worker = blockIdx.x / CG;
    const bool claimed = CG == 2 && sched.claims != nullptr;

    if (threadIdx.x == 0) {
        ptx::prefetch_tmap(&tmA);
        ptx::prefetch_tmap(&tmB);
        ptx::prefetch_tmap(&tmOut);
        // pairs are numbered die by die where the device's map is known (neighbouring workers share operand tiles)
        if (claimed && leader) ctl.worker = static_cast<uint32_t>(die::claim_worker(sched.claims, sched.serial, worker, n_workers));
    }
    cta_begin<CG>(ctl, G::STAGES, warp);
    if (claimed) worker = static_cast<int>(leader ? ctl.worker : ptx::ld_shared_cluster_u32(ptx::mapa_shared(ptx::smem_u32(&ctl.worker), 0)));
    const uint32_t tmem = ctl.tmem_base;
    volatile int* abort = &ctl.abort;
    const unsigned long long wait_ns = sched.wait_ns;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            // Consecutive tiles walk the contraction in opposite directions: an operand that every tile re-reads
            // from start to end (the scaled H rows in dW, 39 MB at config 2, next to the streaming slab) is then
            // met again most-recent-lines first, which an LRU cache can serve, instead of oldest first, which it
            // cannot once the footprint exceeds it.  dW read 4.6 GB per launch one way only, 3.7 GB this way.
            // (The sum over k is taken in another order in every other tile: still fixed, run to run.)
            uint32_t rev = 0;
            for (int item = worker; item < sched.n_items && ok; item += n_workers) {
                int m_tile, group, n_begin, n_end;
                decode_item(sched, item, m_tile, group, n_begin, n_end);
                const int m0 = (m_tile * CG + static_cast<int>(rank)) * BM;
                for (int n = n_begin; n < n_end && ok; ++n, rev ^= 1u) {
                    const int n0 = n * BN + static_cast<int>(rank) * G::BN_CTA;
                    for (int kbi = 0; kbi < sched.num_kb; ++kbi) {
                        const int kb = rev ? sched.num_kb - 1 - kbi : kbi;
                        if (!wait_bounded(ptx::smem_u32(&ctl.empty[stage]), phase ^ 1u, abort, status, wait_ns)) { ok = false; break; }
                        const uint32_t full_local = ptx::smem_u32(&ctl.full[stage]);
                        if (leader) ptx::mbar_arrive_expect_tx(full_local, G::STAGE_BYTES * CG);
                        const uint32_t full_sig = CG == 1 ? full_local : ptx::mapa_shared(full_local, 0);   // pair: the leader's barrier
#pragma unroll
                        for (int h = 0; h < G::KS; ++h) {
                            const uint32_t a_dst = ring + stage * G::STAGE_BYTES + h * A_STAGE_BYTES;
                            const uint32_t b_dst = ring + stage * G::STAGE_BYTES + G::A_BYTES + h * G::B_SLICE_BYTES;
                            const int k0 = (kb * G::KS + h) * BK;
                            if (A_MN) {
#pragma unroll
                                for (int j = 0; j < BM / 64; ++j) load_box<CG>(a_dst + j * MN_ATOM_BYTES, &tmA, m0 + j * 64, k0, full_sig);
                            } else {
                                load_box<CG>(a_dst, &tmA, k0, m0, full_sig);
                            }
                            if (B_MN) {
#pragma unroll
                                for (int j = 0; j < G::BN_CTA / 64; ++j) load_box<CG>(b_dst + j * MN_ATOM_BYTES, &tmB, n0 + j * 64, k0, full_sig);
                            } else {
                                load_box<CG>(b_dst, &tmB, k0, n0, full_sig);
                            }
                        }
                        ++issued;
                        if (++stage == G::STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (!ok) {
                // aborted: let the copies already issued land before the CTA exits.  The leader can
                // watch its own `full` barriers; the peer, whose copies signal the leader, just waits.
                if (leader) {
                    const uint32_t back = issued < G::STAGES ? issued : G::STAGES;
                    for (uint32_t i = 0; i < back; ++i) {
                        const uint32_t q = issued - 1 - i;
                        wait_bounded<true>(ptx::smem_u32(&ctl.full[q % G::STAGES]), (q / G::STAGES) & 1u, abort, status, DRAIN_LIMIT_NS);
                    }
                } else {
                    const unsigned long long t0 = ptx::globaltimer_ns();
                    while (ptx::globaltimer_ns() - t0 < DRAIN_LIMIT_NS) __nanosleep(1000);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(BM * CG, BN, A_MN, B_MN);
            // The tensor pipe takes only a few MMAs ahead of the one it executes, so the instructions between
            // two issues are on its critical path: the shared-memory descriptors of stage 0 are built once and
            // those of the other stages and k-slices follow by adding to the (address >> 4) field.
            //   K-major: 16 elements = 32 bytes further inside the 128-byte swizzle row;
            //   MN-major: 16 k-rows = two 8-row swizzle atoms (2048 bytes) further.
            const uint64_t adesc0 = A_MN ? ptx::smem_desc_sw128(ring, MN_ATOM_BYTES, 1024) : ptx::smem_desc_sw128(ring, 16, 1024);
            const uint64_t bdesc0 = B_MN ? ptx::smem_desc_sw128(ring + G::A_BYTES, MN_ATOM_BYTES, 1024)
                                         : ptx::smem_desc_sw128(ring + G::A_BYTES, 16, 1024);
            constexpr uint64_t A_SLICE_STEP = A_STAGE_BYTES >> 4, B_SLICE_STEP = G::B_SLICE_BYTES >> 4;
            constexpr uint64_t STAGE_STEP = G::STAGE_BYTES >> 4;
            constexpr uint64_t A_KSTEP = (A_MN ? 2048 : 32) >> 4;
            constexpr uint64_t B_KSTEP = (B_MN ? 2048 : 32) >> 4;
            const uint32_t full0 = ptx::smem_u32(&ctl.full[0]), empty0 = ptx::smem_u32(&ctl.empty[0]);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            uint64_t adesc = adesc0, bdesc = bdesc0;
            bool ok = true;
            for (int item = worker; item < sched.n_items && ok; item += n_workers) {
                int m_tile, group, n_begin, n_end;
                decode_item(sched, item, m_tile, group, n_begin, n_end);
                for (int n = n_begin; n < n_end && ok; ++n) {
                    if (!wait_bounded(ptx::smem_u32(&ctl.tempty[acc]), acc_phase ^ 1u, abort, status, wait_ns)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem + acc * BN;
                    for (int kb = 0; kb < sched.num_kb; ++kb) {
                        if (!wait_bounded(full0 + stage * 8u, phase, abort, status, wait_ns)) { ok = false; break; }
                        ptx::tc_fence_after();
#pragma unroll
                        for (int h = 0; h < G::KS; ++h) {
#pragma unroll
                            for (int j = 0; j < BK / 16; ++j) {
                                const uint32_t accumulate = (h != 0 || j != 0 || kb != 0) ? 1u : 0u;
                                const uint64_t ad = adesc + h * A_SLICE_STEP + j * A_KSTEP, bd = bdesc + h * B_SLICE_STEP + j * B_KSTEP;
                                if (CG == 1) ptx::umma_bf16(d_tmem, ad, bd, idesc, accumulate);
                                else ptx::umma_bf16_pair(d_tmem, ad, bd, idesc, accumulate);
                            }
                        }
                        // frees the stage (in both CTAs of a pair) once these MMAs have read it
                        if (CG == 1) ptx::umma_commit(empty0 + stage * 8u);
                        else ptx::umma_commit_pair(empty0 + stage * 8u, 3);
                        if (++stage == G::STAGES) {
                            stage = 0; phase ^= 1u; adesc = adesc0; bdesc = bdesc0;
                        } else {
                            adesc += STAGE_STEP; bdesc += STAGE_STEP;
                        }
                    }
                    if (!ok) break;
                    // accumulator complete (in both CTAs of a pair)
                    if (CG == 1) ptx::umma_commit(ptx::smem_u32(&ctl.tfull[acc]));
                    else ptx::umma_commit_pair(ptx::smem_u32(&ctl.tfull[acc]), 3);
                    acc ^= 1u;
                    if (acc == 0) acc_phase ^= 1u;
                }
            }
            if (!ok) {
                // aborted: make sure no MMA is still in flight before TMEM is freed
                if (CG == 1) ptx::umma_commit(ptx::smem_u32(&ctl.drain));
                else ptx::umma_commit_pair(ptx::smem_u32(&ctl.drain), 1);
                wait_bounded<true>(ptx::smem_u32(&ctl.drain), 0, abort, status, DRAIN_LIMIT_NS);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        typename Epi::State st;
        OutStage out;
        out.tm = &tmOut;
        out.buf = ring + G::RING_BYTES + static_cast<uint32_t>(quarter) * 2 * OUT_TILE_BYTES;
        out.lane = lane;
        out.sel = 0;
        out.row0 = 0;
        out.n_rows = Epi::out_rows(ep);
        for (int item = worker; item < sched.n_items && ok; item += n_workers) {
            int m_tile, group, n_begin, n_end;
            decode_item(sched, item, m_tile, group, n_begin, n_end);
            Epi::begin_item(ep, st, m_tile * CG + static_cast<int>(rank), row_in_tile);
            out.row0 = (m_tile * CG + static_cast<int>(rank)) * BM + quarter * 32;
            for (int n = n_begin; n < n_end; ++n) {
                ok = wait_bounded(ptx::smem_u32(&ctl.tfull[acc]), acc_phase, abort, status, wait_ns);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after();
                Epi::tile(ep, st, n, lane_base + acc * BN, out);
                ptx::tc_fence_before();
                if (CG == 1) {
                    ptx::mbar_arrive(ptx::smem_u32(&ctl.tempty[acc]));
                } else {
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&ctl.tempty[acc]), 0));
                }
                acc ^= 1u;
                if (acc == 0) acc_phase ^= 1u;
            }
            if (ok) Epi::end_item(ep, st, group);
        }
        out.finish();      // the staged tiles have left shared memory before the CTA may exit
    }

    cta_end<CG>(warp, tmem);
}

// ------------------------------------------------------------------------------------------
// Test hook for the time-out path: the set-up, the role split, the abort flag and the teardown of
// gemm_kernel (same functions), with no copy and no MMA in flight.  Every role waits on a barrier
// that nothing ever signals: role `which` (0 = producer lane, 1 = MMA lane, 2 = epilogue warps) with
// the limit `short_ns`, the others with `long_ns`.  The short wait runs out, raises the CTA's abort
// flag and writes CAT_ERR_TIMEOUT to *status; the other roles must then leave through the flag long
// before their own limit.  elapsed_ns[cta * 6 + warp] reports how long each warp waited.  The kernel
// returns by itself; nothing traps and nothing is left waiting.
// ------------------------------------------------------------------------------------------
template <int CG>
__global__ void __launch_bounds__(NUM_THREADS, 1)
wait_probe_kernel(int which, unsigned long long short_ns, unsigned long long long_ns, int* status, unsigned long long* elapsed_ns) {
    __shared__ Ctl ctl;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    cta_begin<CG>(ctl, 1, warp);
    const uint32_t tmem = ctl.tmem_base;
    volatile int* abort = &ctl.abort;
    const unsigned long long t0 = ptx::globaltimer_ns();
    const int role = warp < 2 ? warp : 2;
    const unsigned long long limit = role == which ? short_ns : long_ns;
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) ok = wait_bounded(ptx::smem_u32(&ctl.empty[0]), 0, abort, status, limit);
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) ok = wait_bounded(ptx::smem_u32(&ctl.full[0]), 0, abort, status, limit);
        __syncwarp();
    } else {
        ok = wait_bounded(ptx::smem_u32(&ctl.tfull[0]), 0, abort, status, limit);
        ok = __all_sync(0xffffffffu, ok);
    }
    if (lane == 0) elapsed_ns[blockIdx.x * (NUM_THREADS / 32) + warp] = (ptx::globaltimer_ns() - t0) | (ok ? (1ull << 63) : 0ull);
    cta_end<CG>(warp, tmem);
}

}  // namespace tc
}  // namespace cat
