// C ABI of the CAT loss library: host-side validation, workspace planning, tensor-map
// construction and kernel launches.  Nothing here allocates device memory.
#include "../../include/cat_loss.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string.h>

#include <stdlib.h>

#include <math.h>

#include <atomic>
#include <mutex>

#include "kd.cuh"
#include "rowops.cuh"
#include "simt.cuh"
#include "tc_gemm.cuh"

// ------------------------------------------------------------------------------------------
// Forward pass with built-in scratch, for callers that may not allocate device memory.
// The array below is part of the module image: each GPU that loads the library carries it
// until the process ends.  Host code must not use the symbol's name as a pointer (on the host
// it is only a stand-in); the device address is fetched once per device with
// cudaGetSymbolAddress and that address is what the kernels receive.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[CAT_STATIC_SCRATCH_BYTES];

namespace {

using namespace cat;

constexpr int kPlanSMs = 148;            // B200: the static schedules are planned for 148 SMs
constexpr size_t kHeaderBytes = 1024;    // workspace header: int32 status at byte 0, fp32 g/N at byte 64, worker claims from byte 256
constexpr size_t kClaimsOffset = 256;    // up to 192 ints: one per CTA pair of a GEMM launch
constexpr size_t kScaleOffset = 64;
constexpr int kMaxSplits = 128;
constexpr long long kDefaultSlabMiB = 2048;
constexpr long long kDefaultFusedSlabMiB = 3072;

inline size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }
inline long long cdiv(long long a, long long b) { return (a + b - 1) / b; }

// CTAs per tensor-core output tile: 2 (a CTA pair shares a 256 x 256 tile, tcgen05 cta_group::2)
// unless the environment variable CAT_LOSS_CTA_PAIR=0 selects the one-CTA 128 x 256 kernel.
// Read once per process: plans and workspace sizes depend on it.
int cta_group() {
    static const int cg = [] {
        const char* e = getenv("CAT_LOSS_CTA_PAIR");
        return (e && e[0] == '0') ? 1 : 2;
    }();
    return cg;
}
inline long long tile_m() { return static_cast<long long>(tc::BM) * cta_group(); }   // rows per scheduled m-tile
inline long long plan_workers() { return kPlanSMs / cta_group(); }                    // CTAs or CTA pairs

// ------------------------------------------------------------------------------ validation
int check_shape(const cat_shape* s) {
    if (!s) return CAT_ERR_NULL;
    if (s->T <= 0 || s->d <= 0 || s->V <= 0 || s->K < 1) return CAT_ERR_SHAPE;
    if (s->T >= (1ll << 31) || s->V >= (1ll << 31) || s->d > 65536) return CAT_ERR_SHAPE;
    if (s->T % s->K != 0) return CAT_ERR_SHAPE;
    if (s->ldH < s->d || s->ldW < s->d) return CAT_ERR_SHAPE;
    if (s->slab_mib < 0) return CAT_ERR_SHAPE;
    if (s->in_dtype != CAT_BF16 && s->in_dtype != CAT_F32) return CAT_ERR_DTYPE;
    if (s->dW_dtype != CAT_BF16 && s->dW_dtype != CAT_F32) return CAT_ERR_DTYPE;
    if (s->in_dtype == CAT_F32 && s->dW_dtype != CAT_F32) return CAT_ERR_DTYPE;
    if (s->weight_mode != CAT_WEIGHT_CONFIDENCE && s->weight_mode != CAT_WEIGHT_FIXED_DECAY) return CAT_ERR_SHAPE;
    if (s->weight_mode == CAT_WEIGHT_FIXED_DECAY && !(s->decay_gamma >= 0.f && s->decay_gamma <= 3.0e38f)) return CAT_ERR_SHAPE;
    if (s->in_dtype == CAT_BF16 && (s->d % 8 != 0 || s->ldH % 8 != 0 || s->ldW % 8 != 0)) return CAT_ERR_ALIGN;
    return CAT_OK;
}

inline bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

// ------------------------------------------------------------------------------ planning
struct FwdPlan {
    int S;                 // vocabulary splits
    int n_row_ctas;        // CTAs of the per-row kernel (or of the per-block kernel for general K)
    bool warp_scan;        // K is a power of two <= 32
    size_t off_part_m, off_part_l, off_z_label, off_row_ce, off_partials, total;
};

// Vocabulary splits of the forward GEMM: persistent workers (CTAs or CTA pairs) take items
// (m-tile, split) round-robin, so the cost is waves * longest item, plus a small charge per split.
int fwd_splits(long long rows, long long V) {
    const long long num_m = cdiv(rows, tile_m()), num_n = cdiv(V, tc::BN);
    const long long smax = num_n < kMaxSplits ? num_n : kMaxSplits;
    double best = 1e300;
    int S_best = 1;
    for (long long S = 1; S <= smax; ++S) {
        const double cost = static_cast<double>(cdiv(num_m * S, plan_workers())) * static_cast<double>(cdiv(num_n, S)) + 1e-3 * S;
        if (cost < best) { best = cost; S_best = static_cast<int>(S); }
    }
    return S_best;
}

FwdPlan plan_fwd(const cat_shape* s) {
    FwdPlan p;
    if (s->in_dtype == CAT_BF16) {
        p.S = fwd_splits(s->T, s->V);
    } else {
        const long long num_m = cdiv(s->T, simt::TM), num_n = cdiv(s->V, simt::TN);
        long long S = (2 * kPlanSMs) / num_m;
        if (S < 1) S = 1;
        if (S > num_n) S = num_n;
        if (S > 64) S = 64;
        p.S = static_cast<int>(S);
    }
    p.warp_scan = s->K <= 32 && (s->K & (s->K - 1)) == 0;
    const long long units = p.warp_scan ? s->T : s->T / s->K;
    p.n_row_ctas = static_cast<int>(cdiv(units, rows::ROW_THREADS));
    size_t off = kHeaderBytes;
    p.off_part_m = off;  off = align256(off + sizeof(float) * p.S * s->T);
    p.off_part_l = off;  off = align256(off + sizeof(float) * p.S * s->T);
    p.off_z_label = off; off = align256(off + sizeof(float) * s->T);
    p.off_row_ce = off;  off = align256(off + sizeof(float) * s->T);
    p.off_partials = off; off = align256(off + sizeof(rows::CtaPartial) * p.n_row_ctas);
    p.total = off;
    return p;
}

struct BwdPlan {
    long long Vs;          // slab width in vocabulary entries (multiple of 256)
    int n_slabs;
    size_t off_dz, off_dh_acc, total;
};

BwdPlan plan_bwd(const cat_shape* s) {
    BwdPlan p;
    const size_t elt = s->in_dtype == CAT_BF16 ? 2 : 4;
    const long long mib = s->slab_mib > 0 ? s->slab_mib : kDefaultSlabMiB;
    const long long v_pad = cdiv(s->V, 256) * 256;
    long long Vs = (mib << 20) / static_cast<long long>(elt * s->T);
    Vs = (Vs / 256) * 256;
    if (Vs < 256) Vs = 256;
    if (Vs > v_pad) Vs = v_pad;
    p.n_slabs = static_cast<int>(cdiv(s->V, Vs));
    p.Vs = cdiv(cdiv(s->V, p.n_slabs), 256) * 256;      // rebalance the slabs
    if (s->in_dtype == CAT_BF16) {
        // Among slab widths within the cap take the one whose dW GEMMs (tiles of a slab = vocabulary tiles x
        // d/256, one per worker at a time) need the fewest waves in total, charging one wave per slab for its
        // fixed costs (launches, one more pass over the fp32 dH accumulator).  A slab of 32 vocabulary tiles at
        // d = 3072 is 384 tiles = 5.2 waves of 74 and pays for 6; 30 tiles is 4.9 and pays for 5.
        const long long n_tiles_n = cdiv(s->d, tc::BN);
        long long best_vs = p.Vs, best_cost = -1;
        for (long long vs = Vs, tries = 0; vs >= 256 && tries < 128; vs -= 256, ++tries) {
            long long cost = 0;
            for (long long v0 = 0; v0 < s->V; v0 += vs) {
                const long long w = (s->V - v0) < vs ? (s->V - v0) : vs;
                cost += cdiv(cdiv(w, tile_m()) * n_tiles_n, plan_workers()) + 1;
            }
            if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_vs = vs; }
        }
        {   // the even split above, if it is at least as good
            long long cost = 0;
            for (long long v0 = 0; v0 < s->V; v0 += p.Vs) {
                const long long w = (s->V - v0) < p.Vs ? (s->V - v0) : p.Vs;
                cost += cdiv(cdiv(w, tile_m()) * n_tiles_n, plan_workers()) + 1;
            }
            if (cost > best_cost) p.Vs = best_vs;
        }
    }
    p.n_slabs = static_cast<int>(cdiv(s->V, p.Vs));
    size_t off = kHeaderBytes;
    p.off_dz = off; off = align256(off + elt * static_cast<size_t>(s->T) * p.Vs);
    p.off_dh_acc = off;
    if (s->in_dtype == CAT_BF16 && p.n_slabs > 1) off = align256(off + sizeof(float) * static_cast<size_t>(s->T) * s->d);
    p.total = off;
    return p;
}

// Fused forward+backward: rows are processed in slabs of whole m-tiles and whole draft
// blocks; one slab of fp16 logits (turned into bf16 dz in place) is the only large scratch.
struct FusedPlan {
    long long Ts;          // rows per slab (multiple of lcm(K, rows per m-tile)), last slab may be shorter
    long long ldz;         // row pitch of the logits slab (V rounded up to 256)
    int n_slabs;
    int S_max;             // largest vocabulary split count over the slabs
    int n_row_ctas;        // per-row / per-block kernel CTAs summed over the slabs
    bool warp_scan;
    bool dw_acc;           // bf16 dW with several slabs: accumulate in an fp32 scratch copy
    size_t off_part_m, off_part_l, off_z_label, off_row_ce, off_partials, off_ref, off_a, off_hs, off_z, off_dw_acc, total;
};

long long gcd_ll(long long a, long long b) { return b == 0 ? a : gcd_ll(b, a % b); }

FusedPlan plan_fused(const cat_shape* s) {
    FusedPlan p;
    p.ldz = cdiv(s->V, 256) * 256;
    const long long L = (static_cast<long long>(s->K) * tile_m()) / gcd_ll(s->K, tile_m());   // lcm(K, rows per m-tile)
    const long long mib = s->slab_mib > 0 ? s->slab_mib : kDefaultFusedSlabMiB;
    long long cap = ((mib << 20) / (p.ldz * 2) / L) * L;       // rows that fit the slab cap
    const long long most = ((s->T - 1) / L) * L;                // at least two slabs: the T x V logits never coexist
    if (most >= L && cap > most) cap = most;
    if (cap < L) cap = L;
    // Among slab heights within the cap take the one that costs the three GEMMs the fewest tile-steps
    // (waves of the 74 tile-workers x k-slices per tile, summed over the slabs): the logits GEMM (items are
    // runs of vocabulary tiles, see fwd_splits), dH (row tiles x d/256 tiles, the whole vocabulary contracted)
    // and dW (vocabulary tiles x d/256 tiles, the slab's rows contracted).  Ties go to the taller slab.
    const long long n_tiles_n = cdiv(s->d, tc::BN), n_tiles_v = cdiv(s->V, tc::BN);
    long long best_ts = cap;
    double best_cost = -1.0;
    for (long long ts = cap, tries = 0; ts >= L && tries < 96; ts -= L, ++tries) {
        double cost = 0.0;
        for (long long r0 = 0; r0 < s->T; r0 += ts) {
            const long long rws = (s->T - r0) < ts ? (s->T - r0) : ts;
            const long long num_m = cdiv(rws, tile_m());
            const long long S = fwd_splits(rws, s->V);
            cost += static_cast<double>(cdiv(num_m * S, plan_workers()) * cdiv(n_tiles_v, S)) * static_cast<double>(s->d);   // logits
            cost += static_cast<double>(cdiv(num_m * n_tiles_n, plan_workers())) * static_cast<double>(s->V);               // dH
            cost += static_cast<double>(cdiv(n_tiles_v * n_tiles_n, plan_workers())) * static_cast<double>(rws);             // dW
        }
        if (best_cost < 0.0 || cost < best_cost * (1.0 - 1e-9)) { best_cost = cost; best_ts = ts; }
    }
    p.Ts = best_ts;
    p.n_slabs = static_cast<int>(cdiv(s->T, p.Ts));
    p.warp_scan = s->K <= 32 && (s->K & (s->K - 1)) == 0;
    p.S_max = 1;
    p.n_row_ctas = 0;
    for (long long r0 = 0; r0 < s->T; r0 += p.Ts) {
        const long long rws = (s->T - r0) < p.Ts ? (s->T - r0) : p.Ts;
        const int S = fwd_splits(rws, s->V);
        if (S > p.S_max) p.S_max = S;
        p.n_row_ctas += static_cast<int>(cdiv(p.warp_scan ? rws : rws / s->K, rows::ROW_THREADS));
    }
    p.dw_acc = s->dW_dtype == CAT_BF16 && p.n_slabs > 1;
    size_t off = kHeaderBytes;
    p.off_part_m = off;  off = align256(off + sizeof(float) * p.S_max * s->T);
    p.off_part_l = off;  off = align256(off + sizeof(float) * p.S_max * s->T);
    p.off_z_label = off; off = align256(off + sizeof(float) * s->T);
    p.off_row_ce = off;  off = align256(off + sizeof(float) * s->T);
    p.off_partials = off; off = align256(off + sizeof(rows::CtaPartial) * p.n_row_ctas);
    p.off_ref = off;     off = align256(off + sizeof(float) * s->T);                                  // reference of the stored exp(z - ref)
    p.off_a = off;       off = align256(off + sizeof(float) * s->T);                                  // per-row factor of the backward
    p.off_hs = off;      off = align256(off + 2 * static_cast<size_t>(p.Ts) * static_cast<size_t>(s->d));   // a[r] * H[r, :] of one slab
    p.off_z = off;       off = align256(off + 2 * static_cast<size_t>(p.Ts) * p.ldz);
    p.off_dw_acc = off;
    if (p.dw_acc) off = align256(off + sizeof(float) * static_cast<size_t>(s->V) * s->d);
    p.total = off;
    return p;
}

// Distillation side of cat_kd_loss_fwd_bwd: what one call needs beyond the fused plan.
struct KdArgs {
    const cat_kd_desc* desc;
    const void* Ht;
    const void* Wt;
    const int64_t* block_start_host;
    const float* user_conf_ext;
};

inline long long clampll(long long x, long long lo, long long hi) { return x < lo ? lo : (x > hi ? hi : x); }

// Target positions [lo, lo + span) that the draft rows [r0, r0 + rws) refer to (block starts are sorted).
void slab_target_range(const int64_t* start, long long r0, long long rws, int K, long long L, long long* lo, long long* span) {
    const long long b0 = r0 / K, b1 = (r0 + rws) / K;       // slabs hold whole blocks
    const long long a = clampll(start[b0], 0, L), b = clampll(start[b1 - 1] + K, 0, L);
    *lo = a;
    *span = b > a ? b - a : 0;
}

struct KdPlan {
    long long Ls_max;       // most target positions any draft slab refers to
    int S_t_max;            // most vocabulary splits of a target slab GEMM
    size_t off_start, off_valid_eff, off_neg_labels, off_zt_label_row, off_conf_dev, off_kd_row, off_part_m_t, off_part_l_t,
        off_zt_label_t, off_lse_t, off_conf_t, off_weight_t, off_partials_t, off_zt, total;
};

int check_kd(const cat_shape* s, const cat_kd_desc* k, const int64_t* start) {
    if (!k || !start) return CAT_ERR_NULL;
    if (s->in_dtype != CAT_BF16) return CAT_ERR_DTYPE;
    if (k->L <= 0 || k->L >= (1ll << 31) || k->d_t <= 0 || k->d_t > 65536 || k->ldHt < k->d_t || k->ldWt < k->d_t) return CAT_ERR_SHAPE;
    if (k->d_t % 8 != 0 || k->ldHt % 8 != 0 || k->ldWt % 8 != 0) return CAT_ERR_ALIGN;
    if (!(k->beta >= 0.f && k->beta <= 3.0e38f)) return CAT_ERR_SHAPE;
    if (k->conf_source != CAT_CONF_TARGET && k->conf_source != CAT_CONF_DRAFT) return CAT_ERR_SHAPE;
    const long long nb = s->T / s->K;
    for (long long b = 0; b + 1 < nb; ++b)
        if (start[b] > start[b + 1]) return CAT_ERR_SHAPE;          // block starts must be sorted
    if (start[0] < -(1ll << 40) || start[nb - 1] > (1ll << 40)) return CAT_ERR_SHAPE;
    return CAT_OK;
}

KdPlan plan_kd(const cat_shape* s, const FusedPlan& fp, const cat_kd_desc* k, const int64_t* start, size_t base) {
    KdPlan p;
    p.Ls_max = 1;
    p.S_t_max = 1;
    for (long long r0 = 0; r0 < s->T; r0 += fp.Ts) {
        const long long rws = (s->T - r0) < fp.Ts ? (s->T - r0) : fp.Ts;
        long long lo, span;
        slab_target_range(start, r0, rws, s->K, k->L, &lo, &span);
        if (span > p.Ls_max) p.Ls_max = span;
        if (span > 0) {
            const int S = fwd_splits(span, s->V);
            if (S > p.S_t_max) p.S_t_max = S;
        }
    }
    const size_t Ls = static_cast<size_t>(p.Ls_max), T = static_cast<size_t>(s->T);
    size_t off = align256(base);
    p.off_start = off;        off = align256(off + sizeof(long long) * (T / s->K));
    p.off_valid_eff = off;    off = align256(off + T);
    p.off_neg_labels = off;   off = align256(off + sizeof(long long) * Ls);
    p.off_zt_label_row = off; off = align256(off + sizeof(float) * T);
    p.off_conf_dev = off;     off = align256(off + sizeof(float) * T);
    p.off_kd_row = off;       off = align256(off + sizeof(float) * T);
    p.off_part_m_t = off;     off = align256(off + sizeof(float) * p.S_t_max * Ls);
    p.off_part_l_t = off;     off = align256(off + sizeof(float) * p.S_t_max * Ls);
    p.off_zt_label_t = off;   off = align256(off + sizeof(float) * Ls);
    p.off_lse_t = off;        off = align256(off + sizeof(float) * Ls);
    p.off_conf_t = off;       off = align256(off + sizeof(float) * Ls);
    p.off_weight_t = off;     off = align256(off + sizeof(float) * Ls);
    p.off_partials_t = off;   off = align256(off + sizeof(rows::CtaPartial) * static_cast<size_t>(cdiv(p.Ls_max, rows::ROW_THREADS)));
    p.off_zt = off;           off = align256(off + 2 * Ls * static_cast<size_t>(fp.ldz));
    p.total = off;
    return p;
}

// ------------------------------------------------------------------------------ device / driver
int check_device(int* sm_count) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_ARCH; }
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_ARCH; }
    if (major != 10) return CAT_ERR_ARCH;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
    *sm_count = sms;
    return CAT_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// 2-D bf16 row-major tensor [rows][cols] with row pitch `ld` elements, 128-byte swizzle.
// box = {box_cols (inner, 64 elements = 128 bytes), box_rows}.  Out-of-range elements read as zero.
int make_tmap(CUtensorMap* m, const void* base, long long rows, long long cols, long long ld, int box_cols, int box_rows,
              bool f32 = false) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return CAT_ERR_CUDA;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * (f32 ? 4 : 2)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CAT_OK : CAT_ERR_CUDA;
}
inline int tmap_k_major(CUtensorMap* m, const void* base, long long mn, long long k, long long ld, int box_mn) {
    return make_tmap(m, base, mn, k, ld, tc::BK, box_mn);          // [MN rows][K cols]
}
inline int tmap_mn_major(CUtensorMap* m, const void* base, long long k, long long mn, long long ld) {
    return make_tmap(m, base, k, mn, ld, 64, tc::BK);              // [K rows][MN cols]
}

// K-major A operand: this CTA's 128 rows.  K-major B operand: the 256 columns of the tile, or the
// 128 of them that one CTA of a pair loads.
inline int tmap_a(CUtensorMap* m, const void* base, long long mn, long long k, long long ld) {
    return tmap_k_major(m, base, mn, k, ld, tc::BM);
}
inline int tmap_b(CUtensorMap* m, const void* base, long long mn, long long k, long long ld) {
    return tmap_k_major(m, base, mn, k, ld, tc::BN / cta_group());
}

// Output slab [rows][cols] of 16-bit values, written by the epilogue warps as boxes of 32 rows x 64 columns.
inline int tmap_out(CUtensorMap* m, const void* base, long long rows, long long cols, long long ld) {
    return make_tmap(m, base, rows, cols, ld, 64, 32);
}

// fp32 output [rows][cols], written as boxes of 32 rows x 32 columns (128-byte rows).
inline int tmap_out_f32(CUtensorMap* m, const void* base, long long rows, long long cols, long long ld) {
    return make_tmap(m, base, rows, cols, ld, 32, 32, true);
}

int band_tiles(long long d) {
    long long b = (64ll << 20) / (tile_m() * d * 2);
    return static_cast<int>(b < 1 ? 1 : b);
}


constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// Set-up, once per device, with that device current: resolve the array's device address.
int static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_ARCH; }
    if (dev < 0 || dev >= kMaxDevices) return CAT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return CAT_ERR_CUDA; }
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return CAT_OK;
}
void* static_scratch_base() {
    void* p = nullptr;
    return static_scratch_address(&p) == CAT_OK ? p : nullptr;
}

// The device's die map (diemap.cuh) is measured by the first GEMM launch on each device, on that launch's
// stream, ahead of the GEMM: two small kernels, about 0.2 ms, nothing allocated (the lines they time lie in
// the library's built-in scratch array, whose contents they leave as they are), no synchronisation.  Kernels
// that run before the table is final number their workers by blockIdx.  Skipped while the stream is being
// captured (it would be replayed with every graph launch) and tried again on the next call.
std::mutex g_die_mu;
bool g_die_launched[64] = {};

void ensure_die_map(int sm_count, cudaStream_t st) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return; }
    std::lock_guard<std::mutex> lock(g_die_mu);
    if (g_die_launched[dev]) return;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) { cudaGetLastError(); return; }
    static const bool off = [] { const char* e = getenv("CAT_LOSS_DIE_MAP"); return e && e[0] == '0'; }();     // CAT_LOSS_DIE_MAP=0: number the pairs by blockIdx
    void* base = off ? nullptr : static_scratch_base();
    if (!base || sm_count > die::MAX_SM) { g_die_launched[dev] = true; return; }      // no table: blockIdx order stays
    // N_LINES lines about 1 MiB apart (a whole number of 128-byte lines), all inside the array
    const size_t stride_words = static_cast<size_t>(CAT_STATIC_SCRATCH_BYTES) / 4 / die::N_LINES - 64;
    die::probe_kernel<<<sm_count * 8, 32, 0, st>>>(static_cast<unsigned*>(base), stride_words, sm_count);
    die::classify_kernel<<<1, 32, 0, st>>>(sm_count);
    cudaGetLastError();
    g_die_launched[dev] = true;
}

unsigned next_launch_serial() {
    static std::atomic<unsigned> n{0};
    unsigned v = ++n;
    v &= 0x7fffffffu;
    return v == 0 ? ++n & 0x7fffffffu : v;
}

template <int A_MN, int B_MN, class Epi, int CG>
int launch_tc_cg(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmOut, const tc::Sched& sched_in,
                 const typename Epi::Params& ep, int* status, int sm_count, cudaStream_t st) {
    tc::Sched sched = sched_in;
    if (CG == 2) {
        ensure_die_map(sm_count, st);
        sched.claims = status + kClaimsOffset / sizeof(int);        // `status` is the first word of a workspace header
        sched.serial = static_cast<int>(next_launch_serial());
    }
    auto kern = tc::gemm_kernel<A_MN, B_MN, Epi, CG>;
    constexpr int smem = tc::Geo<CG>::SMEM_BYTES;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
        cudaGetLastError();
        return CAT_ERR_CUDA;
    }
    const int workers = sm_count / CG;
    const int grid = CG * (sched.n_items < workers ? sched.n_items : workers);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(tc::NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmOut, sched, ep, status) != cudaSuccess) {
        cudaGetLastError();
        return CAT_ERR_CUDA;
    }
    return CAT_OK;
}

// `tmOut`: tensor map of the 16-bit slab an epilogue stores through shared memory (tmap_out), or
// NULL for epilogues that write their output directly.
template <int A_MN, int B_MN, class Epi>
int launch_tc(const CUtensorMap& tmA, const CUtensorMap& tmB, const tc::Sched& sched, const typename Epi::Params& ep,
              int* status, int sm_count, cudaStream_t st, const CUtensorMap* tmOut = nullptr) {
    const CUtensorMap& o = tmOut ? *tmOut : tmA;
    return cta_group() == 2 ? launch_tc_cg<A_MN, B_MN, Epi, 2>(tmA, tmB, o, sched, ep, status, sm_count, st)
                            : launch_tc_cg<A_MN, B_MN, Epi, 1>(tmA, tmB, o, sched, ep, status, sm_count, st);
}

// Launch of a GEMM with the plain-output epilogue: fp32 outputs that either overwrite or accumulate in
// place (pitch a multiple of 4 elements) take the staged TMA store / reduce-add route.
template <int A_MN, int B_MN>
int launch_out(const CUtensorMap& tmA, const CUtensorMap& tmB, const tc::Sched& sched, tc::EpiOut::Params ep, int* status,
               int sm_count, cudaStream_t st) {
    CUtensorMap tmO;
    ep.staged = 0;
    if (ep.out_f32 && !ep.add_bf16 && (ep.add_f32 == nullptr || ep.add_f32 == ep.out_f32) && ep.ld_out % 4 == 0 &&
        !misaligned(ep.out_f32, 16)) {
        if (tmap_out_f32(&tmO, ep.out_f32, ep.M, ep.N, ep.ld_out) != CAT_OK) return CAT_ERR_CUDA;
        ep.staged = 1;
    }
    return launch_tc<A_MN, B_MN, tc::EpiOut>(tmA, tmB, sched, ep, status, sm_count, st, ep.staged ? &tmO : nullptr);
}

tc::Sched make_sched(long long M, long long N, long long Kd, int n_groups, int band_m, int n_fastest) {
    tc::Sched s;
    s.num_m_tiles = static_cast<int>(cdiv(M, tile_m()));
    s.num_n_tiles = static_cast<int>(cdiv(N, tc::BN));
    s.num_kb = static_cast<int>(cdiv(Kd, tc::BK * (cta_group() == 2 ? tc::Geo<2>::KS : tc::Geo<1>::KS)));   // ring stages along the contraction
    s.n_groups = n_groups > 0 ? n_groups : s.num_n_tiles;
    s.band_m = band_m < 1 ? 1 : band_m;
    s.n_fastest = n_fastest;
    s.n_items = s.num_m_tiles * s.n_groups;
    s.wait_ns = tc::WAIT_LIMIT_NS;
    s.claims = nullptr;
    s.serial = 0;
    return s;
}

// Forward + backward over row slabs with the slab's logits kept (cat_loss_fwd_bwd); with `kd` also the
// distillation term of Eq. 12 (cat_kd_loss_fwd_bwd): per slab a second logits GEMM on the target
// side, the target confidences of Eq. 9, and a dz that carries both terms.
int fused_core(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid_in,
               const float* conf_ext_in, const float* grad_loss, float* loss, float* lse, float* conf, float* weight,
               cat_stats* stats, void* dH, void* dW, int accumulate_dW, void* workspace, size_t workspace_bytes,
               void* cuda_stream, const KdArgs* kd, void* const* marks = nullptr) {
    if (!shape || !H || !W || !labels || !loss || !lse || !conf || !weight || !dH || !dW) return CAT_ERR_NULL;
    // optional timing marks (cat_loss_fwd_bwd_events): the next caller-owned event is recorded after each stage
    int n_marked = 0;
    auto mark = [&](cudaStream_t s) { if (marks) cudaEventRecord(static_cast<cudaEvent_t>(marks[n_marked++]), s); };
    const int sc = check_shape(shape);
    if (sc != CAT_OK) return sc;
    const uint8_t* valid = valid_in;
    const float* conf_ext = conf_ext_in;
    if (kd) {
        const int kc = check_kd(shape, kd->desc, kd->block_start_host);
        if (kc != CAT_OK) return kc;
        if (!kd->Ht || !kd->Wt) return CAT_ERR_NULL;
        if (misaligned(kd->Ht, 16) || misaligned(kd->Wt, 16)) return CAT_ERR_ALIGN;
    }
    if (shape->in_dtype != CAT_BF16) {
        // fp32 path: forward then backward, sharing one workspace (the passes run back to back)
        const size_t need = cat_loss_workspace_bytes(shape, 2);
        if (!workspace || misaligned(workspace, 256) || workspace_bytes < need) return CAT_ERR_WORKSPACE;
        const int rc = cat_loss_fwd(shape, H, W, labels, valid, conf_ext, loss, lse, conf, weight, stats, workspace,
                                    workspace_bytes, cuda_stream);
        if (rc != CAT_OK) return rc;
        return cat_loss_bwd(shape, H, W, labels, valid, lse, weight, grad_loss, dH, dW, accumulate_dW, workspace,
                            workspace_bytes, cuda_stream);
    }
    if (misaligned(H, 16) || misaligned(W, 16) || misaligned(dH, 16) || misaligned(dW, 16) || misaligned(labels, 8) ||
        misaligned(loss, 4) || misaligned(lse, 4) || misaligned(conf, 4) || misaligned(weight, 4) ||
        (conf_ext && misaligned(conf_ext, 4)) || (grad_loss && misaligned(grad_loss, 4)) || (stats && misaligned(stats, 8)))
        return CAT_ERR_ALIGN;
    const FusedPlan plan = plan_fused(shape);
    KdPlan kp;
    memset(&kp, 0, sizeof(kp));
    if (kd) kp = plan_kd(shape, plan, kd->desc, kd->block_start_host, plan.total);
    if (!workspace || misaligned(workspace, 256) || workspace_bytes < (kd ? kp.total : plan.total)) return CAT_ERR_WORKSPACE;
    int sm_count = 0;
    const int dc = check_device(&sm_count);
    if (dc != CAT_OK) return dc;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* status = reinterpret_cast<int*>(ws);
    float* scale = reinterpret_cast<float*>(ws + kScaleOffset);
    float* part_m = reinterpret_cast<float*>(ws + plan.off_part_m);
    float* part_l = reinterpret_cast<float*>(ws + plan.off_part_l);
    float* z_label = reinterpret_cast<float*>(ws + plan.off_z_label);
    float* row_ce = reinterpret_cast<float*>(ws + plan.off_row_ce);
    rows::CtaPartial* partials = reinterpret_cast<rows::CtaPartial*>(ws + plan.off_partials);
    void* zs = ws + plan.off_z;
    float* dw_acc = reinterpret_cast<float*>(ws + plan.off_dw_acc);
    float* ref = reinterpret_cast<float*>(ws + plan.off_ref);
    float* a_row = reinterpret_cast<float*>(ws + plan.off_a);
    __nv_bfloat16* h_scaled = reinterpret_cast<__nv_bfloat16*>(ws + plan.off_hs);
    const int T = static_cast<int>(shape->T), V = static_cast<int>(shape->V), d = static_cast<int>(shape->d);
    const long long* y = reinterpret_cast<const long long*>(labels);
    const __nv_bfloat16* Hb = static_cast<const __nv_bfloat16*>(H);

    CUtensorMap tmW_k, tmW_mn;
    if (tmap_b(&tmW_k, W, shape->V, shape->d, shape->ldW) != CAT_OK) return CAT_ERR_CUDA;
    if (tmap_mn_major(&tmW_mn, W, shape->V, shape->d, shape->ldW) != CAT_OK) return CAT_ERR_CUDA;
    if (cudaMemsetAsync(ws, 0, kHeaderBytes, st) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
    // distillation: device copies / scratch of this call
    long long* start_dev = nullptr;
    unsigned char* valid_eff = nullptr;
    float *zt_label_row = nullptr, *conf_dev = nullptr, *kd_row = nullptr;
    CUtensorMap tmWt_k;
    if (kd) {
        start_dev = reinterpret_cast<long long*>(ws + kp.off_start);
        valid_eff = ws + kp.off_valid_eff;
        zt_label_row = reinterpret_cast<float*>(ws + kp.off_zt_label_row);
        conf_dev = reinterpret_cast<float*>(ws + kp.off_conf_dev);
        kd_row = reinterpret_cast<float*>(ws + kp.off_kd_row);
        if (cudaMemcpyAsync(start_dev, kd->block_start_host, sizeof(long long) * (shape->T / shape->K), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemsetAsync(ws + kp.off_neg_labels, 0xFF, sizeof(long long) * kp.Ls_max, st) != cudaSuccess) {   // labels of -1: no label gather on the target side
            cudaGetLastError();
            return CAT_ERR_CUDA;
        }
        kd::prepare_kernel<<<static_cast<unsigned>(cdiv(T, rows::ROW_THREADS)), rows::ROW_THREADS, 0, st>>>(
            y, valid_in, start_dev, T, shape->K, V, kd->desc->L, valid_eff);
        valid = valid_eff;      // from here on a row without a target position is an invalid row
        if (tmap_b(&tmWt_k, kd->Wt, shape->V, kd->desc->d_t, kd->desc->ldWt) != CAT_OK) return CAT_ERR_CUDA;
    }
    mark(st);
    rows::bwd_scale_kernel<<<1, 1024, 0, st>>>(y, valid, T, V, grad_loss, scale);
    if (cudaGetLastError() != cudaSuccess) return CAT_ERR_CUDA;
    mark(st);

    int cta0 = 0;
    for (int sl = 0; sl < plan.n_slabs; ++sl) {
        const long long r0 = static_cast<long long>(sl) * plan.Ts;
        const long long rws = (shape->T - r0) < plan.Ts ? (shape->T - r0) : plan.Ts;
        const bool first = sl == 0, last = sl == plan.n_slabs - 1;
        const int S = fwd_splits(rws, shape->V);
        const __nv_bfloat16* Hs = Hb + r0 * shape->ldH;
        CUtensorMap tmH_k, tmH_mn, tmZ_k, tmZ_mn;
        if (tmap_a(&tmH_k, Hs, rws, shape->d, shape->ldH) != CAT_OK) return CAT_ERR_CUDA;
        if (tmap_mn_major(&tmH_mn, Hs, rws, shape->d, shape->ldH) != CAT_OK) return CAT_ERR_CUDA;
        if (tmap_a(&tmZ_k, zs, rws, shape->V, plan.ldz) != CAT_OK) return CAT_ERR_CUDA;
        if (tmap_mn_major(&tmZ_mn, zs, rws, shape->V, plan.ldz) != CAT_OK) return CAT_ERR_CUDA;
        CUtensorMap tmZ_out;
        if (tmap_out(&tmZ_out, zs, rws, shape->V, plan.ldz) != CAT_OK) return CAT_ERR_CUDA;
        if (kd) {   // logits of this row slab: softmax partials + label logit, logits kept as fp16
            const tc::Sched sched = make_sched(rws, shape->V, shape->d, S, band_tiles(shape->d), 0);
            tc::EpiFwdStore::Params ep;
            ep.labels = y + r0; ep.part_m = part_m + r0; ep.part_l = part_l + r0; ep.z_label = z_label + r0;
            ep.zs = static_cast<__half*>(zs); ep.ldz = plan.ldz; ep.part_stride = T; ep.ref = nullptr;
            ep.T = static_cast<int>(rws); ep.V = V;
            const int rc = launch_tc<0, 0, tc::EpiFwdStore>(tmH_k, tmW_k, sched, ep, status, sm_count, st, &tmZ_out);
            if (rc != CAT_OK) return rc;
        } else {
            // per-row reference (the label logit), then the logits GEMM: softmax partials + label logit,
            // and exp(z - ref) kept as bf16 so that the backward needs no second pass over the slab
            rows::label_ref_kernel<<<static_cast<unsigned>(cdiv(rws * 32, rows::ROW_THREADS)), rows::ROW_THREADS, 0, st>>>(
                Hs, shape->ldH, static_cast<const __nv_bfloat16*>(W), shape->ldW, d, y + r0, valid ? valid + r0 : nullptr,
                static_cast<int>(rws), V, ref + r0);
            if (cudaGetLastError() != cudaSuccess) return CAT_ERR_CUDA;
            mark(st);
            const tc::Sched sched = make_sched(rws, shape->V, shape->d, S, band_tiles(shape->d), 0);
            tc::EpiFwdExp::Params ep;
            ep.labels = y + r0; ep.part_m = part_m + r0; ep.part_l = part_l + r0; ep.z_label = z_label + r0;
            ep.zs = static_cast<__half*>(zs); ep.ldz = plan.ldz; ep.part_stride = T; ep.ref = ref + r0;
            ep.T = static_cast<int>(rws); ep.V = V;
            const int rc = launch_tc<0, 0, tc::EpiFwdExp>(tmH_k, tmW_k, sched, ep, status, sm_count, st, &tmZ_out);
            if (rc != CAT_OK) return rc;
            mark(st);
        }
        long long t_lo = 0, t_span = 0;
        float* lse_t_slab = nullptr;
        if (kd) {
            // target side of this slab: logits of the positions its rows refer to (kept as fp16), their lse,
            // and the target's confidence in each draft row's label (Eq. 9)
            slab_target_range(kd->block_start_host, r0, rws, shape->K, kd->desc->L, &t_lo, &t_span);
            lse_t_slab = reinterpret_cast<float*>(ws + kp.off_lse_t);
            if (t_span > 0) {
                const __nv_bfloat16* Hts = static_cast<const __nv_bfloat16*>(kd->Ht) + t_lo * kd->desc->ldHt;
                CUtensorMap tmHt_k;
                if (tmap_a(&tmHt_k, Hts, t_span, kd->desc->d_t, kd->desc->ldHt) != CAT_OK) return CAT_ERR_CUDA;
                const int St = fwd_splits(t_span, shape->V);
                const tc::Sched sched = make_sched(t_span, shape->V, kd->desc->d_t, St, band_tiles(kd->desc->d_t), 0);
                tc::EpiFwdStore::Params ep;
                ep.labels = reinterpret_cast<const long long*>(ws + kp.off_neg_labels);
                ep.part_m = reinterpret_cast<float*>(ws + kp.off_part_m_t);
                ep.part_l = reinterpret_cast<float*>(ws + kp.off_part_l_t);
                ep.z_label = reinterpret_cast<float*>(ws + kp.off_zt_label_t);
                ep.zs = reinterpret_cast<__half*>(ws + kp.off_zt); ep.ldz = plan.ldz; ep.part_stride = kp.Ls_max; ep.ref = nullptr;
                ep.T = static_cast<int>(t_span); ep.V = V;
                CUtensorMap tmZt_out;
                if (tmap_out(&tmZt_out, ws + kp.off_zt, t_span, shape->V, plan.ldz) != CAT_OK) return CAT_ERR_CUDA;
                const int rc = launch_tc<0, 0, tc::EpiFwdStore>(tmHt_k, tmWt_k, sched, ep, status, sm_count, st, &tmZt_out);
                if (rc != CAT_OK) return rc;
                rows::RowParams rp;
                rp.part_m = ep.part_m; rp.part_l = ep.part_l; rp.z_label = ep.z_label; rp.labels = ep.labels;
                rp.valid = nullptr; rp.conf_ext = nullptr;
                rp.lse = lse_t_slab; rp.conf = reinterpret_cast<float*>(ws + kp.off_conf_t);
                rp.weight = reinterpret_cast<float*>(ws + kp.off_weight_t); rp.row_ce = nullptr;
                rp.partials = reinterpret_cast<rows::CtaPartial*>(ws + kp.off_partials_t); rp.part_stride = kp.Ls_max;
                rp.T = static_cast<int>(t_span); rp.V = V; rp.K = 1; rp.S = St; rp.fixed_decay = 0; rp.gamma = 0.f;
                rows::row_kernel<true><<<static_cast<unsigned>(cdiv(t_span, rows::ROW_THREADS)), rows::ROW_THREADS, 0, st>>>(rp);
            }
            kd::target_conf_kernel<<<static_cast<unsigned>(cdiv(rws * 32, rows::ROW_THREADS)), rows::ROW_THREADS, 0, st>>>(
                static_cast<const __nv_bfloat16*>(kd->Ht), kd->desc->ldHt, static_cast<const __nv_bfloat16*>(kd->Wt), kd->desc->ldWt,
                static_cast<int>(kd->desc->d_t), y, valid_eff, start_dev, shape->K, r0, static_cast<int>(rws), t_lo, lse_t_slab,
                zt_label_row, conf_dev);
            if (cudaGetLastError() != cudaSuccess) return CAT_ERR_CUDA;
            conf_ext = kd->user_conf_ext ? kd->user_conf_ext : (kd->desc->conf_source == CAT_CONF_TARGET ? conf_dev : nullptr);
        }
        int n_ctas;
        {   // lse, confidence (Eq. 9), CAT weights (Eq. 10), loss partials of the slab's blocks
            rows::RowParams rp;
            rp.part_m = part_m + r0; rp.part_l = part_l + r0; rp.z_label = z_label + r0; rp.labels = y + r0;
            rp.valid = valid ? valid + r0 : nullptr; rp.conf_ext = conf_ext ? conf_ext + r0 : nullptr;
            rp.lse = lse + r0; rp.conf = conf + r0; rp.weight = weight + r0; rp.row_ce = row_ce + r0;
            rp.partials = partials + cta0; rp.part_stride = T;
            rp.T = static_cast<int>(rws); rp.V = V; rp.K = shape->K; rp.S = S;
            rp.fixed_decay = shape->weight_mode == CAT_WEIGHT_FIXED_DECAY; rp.gamma = shape->decay_gamma;
            if (plan.warp_scan) {
                n_ctas = static_cast<int>(cdiv(rws, rows::ROW_THREADS));
                rows::row_kernel<true><<<n_ctas, rows::ROW_THREADS, 0, st>>>(rp);
            } else {
                n_ctas = static_cast<int>(cdiv(rws / shape->K, rows::ROW_THREADS));
                rows::row_kernel<false><<<static_cast<unsigned>(cdiv(rws, rows::ROW_THREADS)), rows::ROW_THREADS, 0, st>>>(rp);
                rows::block_scan_kernel<<<n_ctas, rows::ROW_THREADS, 0, st>>>(rp);
            }
            cta0 += n_ctas;
            mark(st);
        }
        if (kd) {
            // both slabs of logits -> dz in place
            kd::z_to_dz_kernel<<<static_cast<unsigned>(rws), rows::ROW_THREADS, 0, st>>>(
                zs, ws + kp.off_zt, plan.ldz, y, valid_eff, start_dev, shape->K, r0, t_lo, lse, lse_t_slab, weight, z_label,
                zt_label_row, kd->desc->beta, kd_row, V);
        } else {
            // dz = a[r] * e' : per-row factor, patched label entry, and the scaled copy of the slab's H rows
            rows::slab_prep_kernel<<<static_cast<unsigned>(rws), rows::ROW_THREADS, 0, st>>>(
                zs, plan.ldz, Hs, shape->ldH, d, y + r0, valid ? valid + r0 : nullptr, lse + r0, weight + r0, z_label + r0,
                ref + r0, V, a_row + r0, h_scaled);
            if (tmap_mn_major(&tmH_mn, h_scaled, rws, shape->d, shape->d) != CAT_OK) return CAT_ERR_CUDA;
        }
        if (cudaGetLastError() != cudaSuccess) return CAT_ERR_CUDA;
        mark(st);
        {   // dH[r0 : r0 + rws, :] = (g/N) dz W : the whole vocabulary is contracted, written once
            const tc::Sched sched = make_sched(rws, shape->d, shape->V, 0, 1, 1);
            tc::EpiOut::Params ep;
            memset(&ep, 0, sizeof(ep));
            ep.alpha = scale; ep.M = static_cast<int>(rws); ep.N = d;
            if (!kd) ep.row_scale = a_row + r0;
            ep.out_bf16 = static_cast<__nv_bfloat16*>(dH) + r0 * shape->ldH; ep.ld_out = shape->ldH;
            const int rc = launch_out<0, 1>(tmZ_k, tmW_mn, sched, ep, status, sm_count, st);
            if (rc != CAT_OK) return rc;
            mark(st);
        }
        {   // dW += (g/N) dz^T H[r0 : r0 + rws, :]
            const tc::Sched sched = make_sched(shape->V, shape->d, rws, 0, 1, 1);
            tc::EpiOut::Params ep;
            memset(&ep, 0, sizeof(ep));
            ep.alpha = scale; ep.M = V; ep.N = d;
            if (shape->dW_dtype == CAT_F32) {
                ep.out_f32 = static_cast<float*>(dW); ep.ld_out = shape->ldW;
                if (!first || accumulate_dW) { ep.add_f32 = ep.out_f32; ep.ld_add = shape->ldW; }
            } else if (!plan.dw_acc) {
                ep.out_bf16 = static_cast<__nv_bfloat16*>(dW); ep.ld_out = shape->ldW;
                if (accumulate_dW) { ep.add_bf16 = ep.out_bf16; ep.ld_add = shape->ldW; }
            } else {
                // bf16 dW over several slabs: sum in fp32 scratch, round once at the end
                if (first) {
                    if (accumulate_dW) { ep.add_bf16 = static_cast<const __nv_bfloat16*>(dW); ep.ld_add = shape->ldW; }
                } else {
                    ep.add_f32 = dw_acc; ep.ld_add = shape->d;
                }
                if (last) { ep.out_bf16 = static_cast<__nv_bfloat16*>(dW); ep.ld_out = shape->ldW; }
                else { ep.out_f32 = dw_acc; ep.ld_out = shape->d; }
            }
            const int rc = launch_out<1, 1>(tmZ_mn, tmH_mn, sched, ep, status, sm_count, st);
            if (rc != CAT_OK) return rc;
            mark(st);
        }
    }
    rows::finalize_kernel<<<1, rows::ROW_THREADS, 0, st>>>(partials, cta0, T / shape->K, loss,
                                                         reinterpret_cast<rows::StatsOut*>(stats), status);
    mark(st);
    if (kd) kd::finalize_kernel<<<1, rows::ROW_THREADS, 0, st>>>(kd_row, valid_eff, T, kd->desc->beta, loss);
    return cudaGetLastError() == cudaSuccess ? CAT_OK : CAT_ERR_CUDA;
}


// cat_conf_fwd treats every sequence position as a draft block of its own (K = 1, Eq. 10 weights).
cat_shape per_position_shape(const cat_shape* s) {
    cat_shape one = *s;
    one.K = 1;
    one.dW_dtype = CAT_F32;
    one.weight_mode = CAT_WEIGHT_CONFIDENCE;
    one.decay_gamma = 0.f;
    return one;
}

}  // namespace

// =================================================================================== exports
extern "C" {

const char* cat_status_string(int status) {
    switch (status) {
        case CAT_OK: return "ok";
        case CAT_ERR_NULL: return "a required pointer is NULL";
        case CAT_ERR_SHAPE: return "invalid shape (T, d, V, K, pitches, T % K)";
        case CAT_ERR_DTYPE: return "unsupported dtype combination";
        case CAT_ERR_ALIGN: return "pointer or pitch alignment rule broken";
        case CAT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CAT_ERR_ARCH: return "current device is not compute capability 10.x";
        case CAT_ERR_CUDA: return "a CUDA call failed";
        case CAT_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
        case CAT_ERR_LIMIT: return "problem needs more scratch than the built-in static array holds";
        default: return "unknown status";
    }
}

size_t cat_loss_workspace_bytes(const cat_shape* shape, int pass) {
    if (check_shape(shape) != CAT_OK) return 0;
    if (pass == 0) return plan_fwd(shape).total;
    if (pass == 1) return plan_bwd(shape).total;
    if (pass == 2) {
        if (shape->in_dtype == CAT_BF16) return plan_fused(shape).total;
        const size_t a = plan_fwd(shape).total, b = plan_bwd(shape).total;
        return a > b ? a : b;
    }
    if (pass == 3) {
        const cat_shape one = per_position_shape(shape);
        return align256(plan_fwd(&one).total) + align256(sizeof(float) * (static_cast<size_t>(one.T) + 64));
    }
    return 0;
}

int cat_loss_launch_count(const cat_shape* shape, int pass) {
    if (check_shape(shape) != CAT_OK) return 0;
    if (pass == 0) return 1 + (plan_fwd(shape).warp_scan ? 1 : 2) + 1;
    if (pass == 1) return 1 + 3 * plan_bwd(shape).n_slabs;
    if (pass == 3) return 3;
    if (pass == 2) {
        if (shape->in_dtype != CAT_BF16)
            return cat_loss_launch_count(shape, 0) + cat_loss_launch_count(shape, 1);
        const FusedPlan p = plan_fused(shape);
        return 1 + p.n_slabs * (2 + (p.warp_scan ? 1 : 2) + 1 + 2) + 1;
    }
    return 0;
}

int cat_loss_fwd(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid,
                 const float* conf_ext, float* loss, float* lse, float* conf, float* weight, cat_stats* stats,
                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!shape || !H || !W || !labels || !loss || !lse || !conf || !weight) return CAT_ERR_NULL;
    const int sc = check_shape(shape);
    if (sc != CAT_OK) return sc;
    const bool bf16 = shape->in_dtype == CAT_BF16;
    if (misaligned(H, bf16 ? 16 : 4) || misaligned(W, bf16 ? 16 : 4) || misaligned(labels, 8) || misaligned(loss, 4) ||
        misaligned(lse, 4) || misaligned(conf, 4) || misaligned(weight, 4) || (conf_ext && misaligned(conf_ext, 4)) ||
        (stats && misaligned(stats, 8)))
        return CAT_ERR_ALIGN;
    const FwdPlan plan = plan_fwd(shape);
    if (!workspace || misaligned(workspace, 256) || workspace_bytes < plan.total) return CAT_ERR_WORKSPACE;
    int sm_count = 0;
    const int dc = check_device(&sm_count);
    if (dc != CAT_OK) return dc;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* status = reinterpret_cast<int*>(ws);
    float* part_m = reinterpret_cast<float*>(ws + plan.off_part_m);
    float* part_l = reinterpret_cast<float*>(ws + plan.off_part_l);
    float* z_label = reinterpret_cast<float*>(ws + plan.off_z_label);
    float* row_ce = reinterpret_cast<float*>(ws + plan.off_row_ce);
    rows::CtaPartial* partials = reinterpret_cast<rows::CtaPartial*>(ws + plan.off_partials);
    const int T = static_cast<int>(shape->T), V = static_cast<int>(shape->V);

    CUtensorMap tmH, tmW;
    if (bf16) {
        if (tmap_a(&tmH, H, shape->T, shape->d, shape->ldH) != CAT_OK) return CAT_ERR_CUDA;
        if (tmap_b(&tmW, W, shape->V, shape->d, shape->ldW) != CAT_OK) return CAT_ERR_CUDA;
    }
    if (cudaMemsetAsync(ws, 0, kHeaderBytes, st) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }

    if (bf16) {
        const tc::Sched sched = make_sched(shape->T, shape->V, shape->d, plan.S, band_tiles(shape->d), 0);
        tc::EpiFwd::Params ep;
        ep.labels = reinterpret_cast<const long long*>(labels);
        ep.part_m = part_m; ep.part_l = part_l; ep.z_label = z_label; ep.T = T; ep.V = V;
        ep.zs = nullptr; ep.ldz = 0; ep.part_stride = T; ep.ref = nullptr;
        const int rc = launch_tc<0, 0, tc::EpiFwd>(tmH, tmW, sched, ep, status, sm_count, st);
        if (rc != CAT_OK) return rc;
    } else {
        simt::Operands op;
        op.A = static_cast<const float*>(H); op.sAm = shape->ldH; op.sAk = 1;
        op.B = static_cast<const float*>(W); op.sBk = 1; op.sBn = shape->ldW;
        op.M = T; op.N = V; op.Kd = static_cast<int>(shape->d); op.n_groups = plan.S;
        simt::EpiParams ep;
        memset(&ep, 0, sizeof(ep));
        ep.labels = reinterpret_cast<const long long*>(labels);
        ep.part_m = part_m; ep.part_l = part_l; ep.z_label = z_label; ep.V = V; ep.v0 = 0;
        const dim3 grid(static_cast<unsigned>(cdiv(T, simt::TM)), static_cast<unsigned>(plan.S));
        simt::gemm_kernel<simt::MODE_FWD><<<grid, simt::THREADS, 0, st>>>(op, ep);
        if (cudaGetLastError() != cudaSuccess) return CAT_ERR_CUDA;
    }

    rows::RowParams rp;
    rp.part_m = part_m; rp.part_l = part_l; rp.z_label = z_label;
    rp.labels = reinterpret_cast<const long long*>(labels); rp.valid = valid; rp.conf_ext = conf_ext;
    rp.lse = lse; rp.conf = conf; rp.weight = weight; rp.row_ce = row_ce; rp.partials = partials;
    rp.T = T; rp.V = V; rp.K = shape->K; rp.S = plan.S; rp.part_stride = T;
    rp.fixed_decay = shape->weight_mode == CAT_WEIGHT_FIXED_DECAY; rp.gamma = shape->decay_gamma;
    if (plan.warp_scan) {
        rows::row_kernel<true><<<plan.n_row_ctas, rows::ROW_THREADS, 0, st>>>(rp);
    } else {
        rows::row_kernel<false><<<static_cast<unsigned>(cdiv(T, rows::ROW_THREADS)), rows::ROW_THREADS, 0, st>>>(rp);
        rows::block_scan_kernel<<<plan.n_row_ctas, rows::ROW_THREADS, 0, st>>>(rp);
    }
    rows::finalize_kernel<<<1, rows::ROW_THREADS, 0, st>>>(partials, plan.n_row_ctas, T / shape->K, loss,
                                                         reinterpret_cast<rows::StatsOut*>(stats), status);
    return cudaGetLastError() == cudaSuccess ? CAT_OK : CAT_ERR_CUDA;
}

// cat_loss_bwd / cat_loss_bwd_events: `slab_events` (host array of cudaEvent_t, one per vocabulary
// slab, or NULL) are recorded on the stream as soon as a slab's rows of dW are final.
static int bwd_core(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid,
                    const float* lse, const float* weight, const float* grad_loss, void* dH, void* dW, int accumulate_dW,
                    void* workspace, size_t workspace_bytes, void* cuda_stream, void* const* slab_events) {
    if (!shape || !H || !W || !labels || !lse || !weight || !dH || !dW) return CAT_ERR_NULL;
    const int sc = check_shape(shape);
    if (sc != CAT_OK) return sc;
    const bool bf16 = shape->in_dtype == CAT_BF16;
    const size_t in_al = bf16 ? 16 : 4;
    if (misaligned(H, in_al) || misaligned(W, in_al) || misaligned(dH, in_al) || misaligned(dW, 16) || misaligned(labels, 8) ||
        misaligned(lse, 4) || misaligned(weight, 4) || (grad_loss && misaligned(grad_loss, 4)))
        return CAT_ERR_ALIGN;
    const BwdPlan plan = plan_bwd(shape);
    if (!workspace || misaligned(workspace, 256) || workspace_bytes < plan.total) return CAT_ERR_WORKSPACE;
    int sm_count = 0;
    const int dc = check_device(&sm_count);
    if (dc != CAT_OK) return dc;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* status = reinterpret_cast<int*>(ws);
    float* scale = reinterpret_cast<float*>(ws + kScaleOffset);
    const int T = static_cast<int>(shape->T), V = static_cast<int>(shape->V), d = static_cast<int>(shape->d);
    const long long* y = reinterpret_cast<const long long*>(labels);

    // tensor maps that do not depend on the slab
    CUtensorMap tmH_k, tmH_mn;
    if (bf16) {
        if (tmap_a(&tmH_k, H, shape->T, shape->d, shape->ldH) != CAT_OK) return CAT_ERR_CUDA;
        if (tmap_mn_major(&tmH_mn, H, shape->T, shape->d, shape->ldH) != CAT_OK) return CAT_ERR_CUDA;
    }
    if (cudaMemsetAsync(ws, 0, kHeaderBytes, st) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
    rows::bwd_scale_kernel<<<1, 1024, 0, st>>>(y, valid, T, V, grad_loss, scale);
    if (cudaGetLastError() != cudaSuccess) return CAT_ERR_CUDA;

    for (int sl = 0; sl < plan.n_slabs; ++sl) {
        const long long v0 = static_cast<long long>(sl) * plan.Vs;
        const long long width = (shape->V - v0) < plan.Vs ? (shape->V - v0) : plan.Vs;
        const bool first = sl == 0, last = sl == plan.n_slabs - 1;
        if (bf16) {
            const __nv_bfloat16* Wb = static_cast<const __nv_bfloat16*>(W) + v0 * shape->ldW;
            __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(ws + plan.off_dz);
            float* dh_acc = reinterpret_cast<float*>(ws + plan.off_dh_acc);
            CUtensorMap tmW_k, tmW_mn, tmDz_k, tmDz_mn;
            if (tmap_b(&tmW_k, Wb, width, shape->d, shape->ldW) != CAT_OK) return CAT_ERR_CUDA;
            if (tmap_mn_major(&tmW_mn, Wb, width, shape->d, shape->ldW) != CAT_OK) return CAT_ERR_CUDA;
            if (tmap_a(&tmDz_k, dz, shape->T, width, plan.Vs) != CAT_OK) return CAT_ERR_CUDA;
            if (tmap_mn_major(&tmDz_mn, dz, shape->T, width, plan.Vs) != CAT_OK) return CAT_ERR_CUDA;
            {   // recompute the logits of this slab and turn them into dz
                // same item shape as the forward pass: (m-tile, run of vocabulary tiles), so the per-row state
                // (label, lse, weight) is loaded once per run
                const tc::Sched sched = make_sched(shape->T, width, shape->d, fwd_splits(shape->T, width), band_tiles(shape->d), 0);
                tc::EpiDz::Params ep;
                ep.labels = y; ep.valid = valid; ep.lse = lse; ep.weight = weight; ep.dz = dz; ep.ld = plan.Vs;
                ep.T = T; ep.V = V; ep.v0 = static_cast<int>(v0);
                CUtensorMap tmDz_out;
                if (tmap_out(&tmDz_out, dz, shape->T, width, plan.Vs) != CAT_OK) return CAT_ERR_CUDA;
                const int rc = launch_tc<0, 0, tc::EpiDz>(tmH_k, tmW_k, sched, ep, status, sm_count, st, &tmDz_out);
                if (rc != CAT_OK) return rc;
            }
            {   // dW[v0 : v0 + width, :] = (g/N) dz^T H
                const tc::Sched sched = make_sched(width, shape->d, shape->T, 0, 1, 1);
                tc::EpiOut::Params ep;
                memset(&ep, 0, sizeof(ep));
                ep.alpha = scale; ep.M = static_cast<int>(width); ep.N = d; ep.ld_add = shape->ldW; ep.ld_out = shape->ldW;
                if (shape->dW_dtype == CAT_F32) {
                    ep.out_f32 = static_cast<float*>(dW) + v0 * shape->ldW;
                    if (accumulate_dW) ep.add_f32 = ep.out_f32;
                } else {
                    ep.out_bf16 = static_cast<__nv_bfloat16*>(dW) + v0 * shape->ldW;
                    if (accumulate_dW) ep.add_bf16 = ep.out_bf16;
                }
                const int rc = launch_out<1, 1>(tmDz_mn, tmH_mn, sched, ep, status, sm_count, st);
                if (rc != CAT_OK) return rc;
                if (slab_events && cudaEventRecord(static_cast<cudaEvent_t>(slab_events[sl]), st) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
            }
            {   // dH (+)= (g/N) dz W[v0 : v0 + width, :]
                const tc::Sched sched = make_sched(shape->T, shape->d, width, 0, 1, 1);
                tc::EpiOut::Params ep;
                memset(&ep, 0, sizeof(ep));
                ep.alpha = scale; ep.M = T; ep.N = d;
                if (!first) { ep.add_f32 = dh_acc; ep.ld_add = shape->d; }
                if (last) { ep.out_bf16 = static_cast<__nv_bfloat16*>(dH); ep.ld_out = shape->ldH; }
                else { ep.out_f32 = dh_acc; ep.ld_out = shape->d; }
                const int rc = launch_out<0, 1>(tmDz_k, tmW_mn, sched, ep, status, sm_count, st);
                if (rc != CAT_OK) return rc;
            }
        } else {
            const float* Hf = static_cast<const float*>(H);
            const float* Wf = static_cast<const float*>(W) + v0 * shape->ldW;
            float* dz = reinterpret_cast<float*>(ws + plan.off_dz);
            const int w = static_cast<int>(width);
            {
                simt::Operands op;
                op.A = Hf; op.sAm = shape->ldH; op.sAk = 1; op.B = Wf; op.sBk = 1; op.sBn = shape->ldW;
                op.M = T; op.N = w; op.Kd = d; op.n_groups = static_cast<int>(cdiv(w, simt::TN));
                simt::EpiParams ep;
                memset(&ep, 0, sizeof(ep));
                ep.labels = y; ep.valid = valid; ep.lse = lse; ep.weight = weight; ep.dz = dz; ep.ld_dz = plan.Vs;
                ep.V = V; ep.v0 = static_cast<int>(v0);
                const dim3 grid(static_cast<unsigned>(cdiv(T, simt::TM)), static_cast<unsigned>(op.n_groups));
                simt::gemm_kernel<simt::MODE_DZ><<<grid, simt::THREADS, 0, st>>>(op, ep);
            }
            {   // dW slice = (g/N) dz^T H : A(m = v, k = r) = dz[r][v], B(k = r, n = i) = H[r][i]
                simt::Operands op;
                op.A = dz; op.sAm = 1; op.sAk = plan.Vs; op.B = Hf; op.sBk = shape->ldH; op.sBn = 1;
                op.M = w; op.N = d; op.Kd = T; op.n_groups = static_cast<int>(cdiv(d, simt::TN));
                simt::EpiParams ep;
                memset(&ep, 0, sizeof(ep));
                ep.alpha = scale; ep.out = static_cast<float*>(dW) + v0 * shape->ldW; ep.ld_out = shape->ldW;
                if (accumulate_dW) { ep.add = ep.out; ep.ld_add = shape->ldW; }
                const dim3 grid(static_cast<unsigned>(cdiv(w, simt::TM)), static_cast<unsigned>(op.n_groups));
                simt::gemm_kernel<simt::MODE_OUT><<<grid, simt::THREADS, 0, st>>>(op, ep);
                if (slab_events && cudaEventRecord(static_cast<cudaEvent_t>(slab_events[sl]), st) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
            }
            {   // dH (+)= (g/N) dz W slice : A(m = r, k = v) = dz[r][v], B(k = v, n = i) = W[v][i]
                simt::Operands op;
                op.A = dz; op.sAm = plan.Vs; op.sAk = 1; op.B = Wf; op.sBk = shape->ldW; op.sBn = 1;
                op.M = T; op.N = d; op.Kd = w; op.n_groups = static_cast<int>(cdiv(d, simt::TN));
                simt::EpiParams ep;
                memset(&ep, 0, sizeof(ep));
                ep.alpha = scale; ep.out = static_cast<float*>(dH); ep.ld_out = shape->ldH;
                if (!first) { ep.add = ep.out; ep.ld_add = shape->ldH; }
                const dim3 grid(static_cast<unsigned>(cdiv(T, simt::TM)), static_cast<unsigned>(op.n_groups));
                simt::gemm_kernel<simt::MODE_OUT><<<grid, simt::THREADS, 0, st>>>(op, ep);
            }
            if (cudaGetLastError() != cudaSuccess) return CAT_ERR_CUDA;
        }
    }
    return CAT_OK;
}

int cat_loss_bwd(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid,
                 const float* lse, const float* weight, const float* grad_loss, void* dH, void* dW, int accumulate_dW,
                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return bwd_core(shape, H, W, labels, valid, lse, weight, grad_loss, dH, dW, accumulate_dW, workspace, workspace_bytes,
                    cuda_stream, nullptr);
}

int cat_loss_fused_slabs(const cat_shape* shape, int64_t* row_begin, int capacity) {
    if (check_shape(shape) != CAT_OK || shape->in_dtype != CAT_BF16) return 0;
    const FusedPlan plan = plan_fused(shape);
    for (int sl = 0; row_begin && sl < plan.n_slabs && sl < capacity; ++sl) row_begin[sl] = static_cast<int64_t>(sl) * plan.Ts;
    return plan.n_slabs;
}

int cat_loss_fwd_bwd_events(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid,
                            const float* conf_ext, const float* grad_loss, float* loss, float* lse, float* conf, float* weight,
                            cat_stats* stats, void* dH, void* dW, int accumulate_dW, void* workspace, size_t workspace_bytes,
                            void* cuda_stream, void* const* stage_events, int n_events) {
    if (!stage_events) return CAT_ERR_NULL;
    if (check_shape(shape) != CAT_OK) return CAT_ERR_SHAPE;
    if (shape->in_dtype != CAT_BF16) return CAT_ERR_DTYPE;
    if (n_events != 6 * plan_fused(shape).n_slabs + 3) return CAT_ERR_SHAPE;
    for (int i = 0; i < n_events; ++i)
        if (!stage_events[i]) return CAT_ERR_NULL;
    return fused_core(shape, H, W, labels, valid, conf_ext, grad_loss, loss, lse, conf, weight, stats, dH, dW, accumulate_dW,
                      workspace, workspace_bytes, cuda_stream, nullptr, stage_events);
}

int cat_loss_bwd_slabs(const cat_shape* shape, int64_t* v_begin, int capacity) {
    if (check_shape(shape) != CAT_OK) return 0;
    const BwdPlan plan = plan_bwd(shape);
    for (int sl = 0; v_begin && sl < plan.n_slabs && sl < capacity; ++sl) v_begin[sl] = static_cast<int64_t>(sl) * plan.Vs;
    return plan.n_slabs;
}

int cat_loss_bwd_events(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid,
                        const float* lse, const float* weight, const float* grad_loss, void* dH, void* dW, int accumulate_dW,
                        void* workspace, size_t workspace_bytes, void* cuda_stream, void* const* slab_events, int n_events) {
    if (!slab_events) return CAT_ERR_NULL;
    if (check_shape(shape) != CAT_OK) return CAT_ERR_SHAPE;
    if (n_events != plan_bwd(shape).n_slabs) return CAT_ERR_SHAPE;
    for (int i = 0; i < n_events; ++i)
        if (!slab_events[i]) return CAT_ERR_NULL;
    return bwd_core(shape, H, W, labels, valid, lse, weight, grad_loss, dH, dW, accumulate_dW, workspace, workspace_bytes,
                    cuda_stream, slab_events);
}

int cat_count_valid(const cat_shape* shape, const int64_t* labels, const uint8_t* valid, int64_t* n_valid, void* cuda_stream) {
    if (!shape || !labels || !n_valid) return CAT_ERR_NULL;
    if (shape->T <= 0 || shape->T >= (1ll << 31) || shape->V <= 0 || shape->V >= (1ll << 31)) return CAT_ERR_SHAPE;
    if (misaligned(labels, 8) || misaligned(n_valid, 8)) return CAT_ERR_ALIGN;
    rows::count_valid_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        reinterpret_cast<const long long*>(labels), valid, static_cast<int>(shape->T), static_cast<int>(shape->V),
        reinterpret_cast<long long*>(n_valid));
    return cudaGetLastError() == cudaSuccess ? CAT_OK : CAT_ERR_CUDA;
}

int cat_loss_fwd_bwd(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid,
                     const float* conf_ext, const float* grad_loss, float* loss, float* lse, float* conf, float* weight,
                     cat_stats* stats, void* dH, void* dW, int accumulate_dW, void* workspace, size_t workspace_bytes,
                     void* cuda_stream) {
    return fused_core(shape, H, W, labels, valid, conf_ext, grad_loss, loss, lse, conf, weight, stats, dH, dW, accumulate_dW,
                      workspace, workspace_bytes, cuda_stream, nullptr);
}

size_t cat_kd_workspace_bytes(const cat_shape* shape, const cat_kd_desc* desc, const int64_t* block_start_host) {
    if (check_shape(shape) != CAT_OK || check_kd(shape, desc, block_start_host) != CAT_OK) return 0;
    const FusedPlan fp = plan_fused(shape);
    return plan_kd(shape, fp, desc, block_start_host, fp.total).total;
}

int cat_kd_loss_fwd_bwd(const cat_shape* shape, const cat_kd_desc* desc, const void* H, const void* W, const int64_t* labels,
                        const uint8_t* valid, const void* Ht, const void* Wt, const int64_t* block_start_host,
                        const float* conf_ext, const float* grad_loss, float* loss, float* lse, float* conf, float* weight,
                        cat_stats* stats, void* dH, void* dW, int accumulate_dW, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    if (!desc || !block_start_host) return CAT_ERR_NULL;
    KdArgs kd;
    kd.desc = desc; kd.Ht = Ht; kd.Wt = Wt; kd.block_start_host = block_start_host; kd.user_conf_ext = conf_ext;
    return fused_core(shape, H, W, labels, valid, conf_ext, grad_loss, loss, lse, conf, weight, stats, dH, dW, accumulate_dW,
                      workspace, workspace_bytes, cuda_stream, &kd);
}

int cat_accept_len(const cat_shape* shape, const float* conf, const float* weight, float* accept_len, void* cuda_stream) {
    if (!shape || !conf || !weight || !accept_len) return CAT_ERR_NULL;
    if (shape->T <= 0 || shape->K < 1 || shape->T % shape->K != 0 || shape->T >= (1ll << 31)) return CAT_ERR_SHAPE;
    if (misaligned(conf, 4) || misaligned(weight, 4) || misaligned(accept_len, 4)) return CAT_ERR_ALIGN;
    const int n_blocks = static_cast<int>(shape->T / shape->K);
    rows::accept_len_kernel<<<static_cast<unsigned>(cdiv(n_blocks, rows::ROW_THREADS)), rows::ROW_THREADS, 0,
                              static_cast<cudaStream_t>(cuda_stream)>>>(conf, weight, accept_len, n_blocks, shape->K);
    return cudaGetLastError() == cudaSuccess ? CAT_OK : CAT_ERR_CUDA;
}

int cat_conf_fwd(const cat_shape* shape, const void* Ht, const void* Wt, const int64_t* labels, const uint8_t* valid,
                 float* conf_seq, float* lse_seq, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!shape || !Ht || !Wt || !labels || !conf_seq || !lse_seq) return CAT_ERR_NULL;
    const cat_shape one = per_position_shape(shape);
    const int sc = check_shape(&one);
    if (sc != CAT_OK) return sc;
    const size_t fwd_bytes = align256(plan_fwd(&one).total);
    const size_t need = fwd_bytes + align256(sizeof(float) * (static_cast<size_t>(one.T) + 64));
    if (!workspace || misaligned(workspace, 256) || workspace_bytes < need) return CAT_ERR_WORKSPACE;
    // with K = 1 every weight is 1 and the loss is the target's own mean cross-entropy: both land in scratch
    float* tail = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + fwd_bytes);
    float* loss_tmp = tail;
    float* weight_tmp = tail + 64;
    return cat_loss_fwd(&one, Ht, Wt, labels, valid, nullptr, loss_tmp, lse_seq, conf_seq, weight_tmp, nullptr, workspace,
                        fwd_bytes, cuda_stream);
}

int cat_conf_window(const float* conf_seq, int64_t L, const int64_t* block_start, int64_t n_blocks, int32_t K,
                    float* conf_ext, void* cuda_stream) {
    if (!conf_seq || !block_start || !conf_ext) return CAT_ERR_NULL;
    if (L <= 0 || n_blocks <= 0 || K < 1 || n_blocks * K >= (1ll << 31)) return CAT_ERR_SHAPE;
    if (misaligned(conf_seq, 4) || misaligned(block_start, 8) || misaligned(conf_ext, 4)) return CAT_ERR_ALIGN;
    const long long n_rows = n_blocks * K;
    rows::conf_window_kernel<<<static_cast<unsigned>(cdiv(n_rows, rows::ROW_THREADS)), rows::ROW_THREADS, 0,
                               static_cast<cudaStream_t>(cuda_stream)>>>(conf_seq, L, reinterpret_cast<const long long*>(block_start),
                                                                         n_rows, K, conf_ext);
    return cudaGetLastError() == cudaSuccess ? CAT_OK : CAT_ERR_CUDA;
}

int cat_loss_fwd_static(const cat_shape* shape, const void* H, const void* W, const int64_t* labels, const uint8_t* valid,
                        const float* conf_ext, float* loss, float* lse, float* conf, float* weight, cat_stats* stats,
                        void* cuda_stream) {
    if (!shape) return CAT_ERR_NULL;
    const int sc = check_shape(shape);
    if (sc != CAT_OK) return sc;
    const size_t need = plan_fwd(shape).total;
    if (need > static_cast<size_t>(CAT_STATIC_SCRATCH_BYTES)) return CAT_ERR_LIMIT;
    if (!H || !W || !labels || !loss || !lse || !conf || !weight) return CAT_ERR_NULL;
    int sms = 0;
    const int dc = check_device(&sms);
    if (dc != CAT_OK) return dc;
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != CAT_OK) return rc;
    // every call clears the status header it relies on (inside cat_loss_fwd); everything else
    // in the scratch is fully rewritten before it is read
    return cat_loss_fwd(shape, H, W, labels, valid, conf_ext, loss, lse, conf, weight, stats, scratch,
                        static_cast<size_t>(CAT_STATIC_SCRATCH_BYTES), cuda_stream);
}

int cat_die_map(int32_t* worker_of_tpc, int capacity, int32_t* n_first_die, void* cuda_stream) {
    int sms = 0;
    const int dc = check_device(&sms);
    if (dc != CAT_OK) return dc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ensure_die_map(sms, st);
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
    die::Map m;
    if (cudaMemcpyFromSymbol(&m, die::g_map, sizeof(m)) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
    if (m.valid != 1 || m.n_tpc <= 0 || m.n_tpc > die::MAX_SM / 2) return 0;
    for (int t = 0; worker_of_tpc && t < m.n_tpc && t < capacity; ++t) worker_of_tpc[t] = m.worker_of_tpc[t];
    if (n_first_die) *n_first_die = m.n_die0;
    return m.n_tpc;
}

}  // extern "C"

// Self-test of the kernels' time-out path: one CTA (or one CTA pair, as the GEMMs are configured) runs the
// GEMM kernel's set-up, role split and teardown around waits that nothing will ever satisfy.
template <int CG>
static int launch_wait_probe(int role, unsigned long long short_ns, unsigned long long long_ns, int* status,
                             unsigned long long* elapsed, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CG, 1, 1);
    cfg.blockDim = dim3(tc::NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, tc::wait_probe_kernel<CG>, role, short_ns, long_ns, status, elapsed) != cudaSuccess) {
        cudaGetLastError();
        return CAT_ERR_CUDA;
    }
    return CAT_OK;
}

extern "C" {

int cat_selftest_wait_timeout(int role, uint64_t short_ns, uint64_t long_ns, int32_t* status, uint64_t* elapsed_ns,
                              void* cuda_stream) {
    if (!status || !elapsed_ns) return CAT_ERR_NULL;
    if (role < 0 || role > 2 || short_ns == 0 || short_ns > 100000000ull || long_ns < short_ns || long_ns > 5000000000ull)
        return CAT_ERR_SHAPE;
    if (misaligned(status, 4) || misaligned(elapsed_ns, 8)) return CAT_ERR_ALIGN;
    int sms = 0;
    const int dc = check_device(&sms);
    if (dc != CAT_OK) return dc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), st) != cudaSuccess) { cudaGetLastError(); return CAT_ERR_CUDA; }
    unsigned long long* el = reinterpret_cast<unsigned long long*>(elapsed_ns);
    return cta_group() == 2 ? launch_wait_probe<2>(role, short_ns, long_ns, status, el, st)
                            : launch_wait_probe<1>(role, short_ns, long_ns, status, el, st);
}

}  // extern "C"
