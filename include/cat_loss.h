/*
 * cat_loss.h -- C ABI of the fused LM-head + Confidence-Adaptive Token (CAT) weighted
 * cross-entropy for NVIDIA B200 (sm_100a).
 *
 * The operation is the training objective of the PARD-2 parallel draft model
 * (Section 3.2, Eq. 9-11; batch form Section 3.3, Eq. 12).  For T = B*K rows laid out
 * draft block after draft block (row r = b*K + k, k = 0..K-1 the draft position):
 *
 *     z[r, v]  = sum_i H[r, i] * W[v, i]                     logits over the whole vocabulary
 *     lse[r]   = log sum_v exp z[r, v]
 *     conf[r]  = exp(z[r, y_r] - lse[r])                     confidence in the label  (Eq. 9, evaluated
 *                                                            with this head; or supplied, see conf_ext)
 *     weight[r]= prod_{j<k, row bK+j valid} conf[bK+j]       exclusive prefix product, 1 at k = 0 (Eq. 10)
 *     loss     = (1/N) sum_{valid r} weight[r] * (lse[r] - z[r, y_r])      (Eq. 11; N = #valid rows)
 *
 * and, with the weights held constant (the sentence after Eq. 10: stop-gradient),
 *
 *     dz[r, v] = g * weight[r]/N * (exp(z[r,v] - lse[r]) - [v == y_r]),   dH = dz W,   dW = dz^T H.
 *
 * A row is valid iff valid[r] != 0 (or valid == NULL) and 0 <= labels[r] < V.  Invalid rows
 * get weight 0, add nothing to the loss or to the gradients, and count as the factor 1 in
 * the prefix product of their block.  The T x V logits are never stored.
 *
 * General conventions
 *   - Every data pointer is a DEVICE pointer owned by the caller, valid on the current
 *     device, unless a parameter says "host".  cat_shape is read on the host.
 *   - Nothing is allocated or freed here and no state is kept between calls, with two exceptions:
 *     cat_loss_fwd_static owns a fixed device array inside the library image and remembers, per
 *     device, that array's address (see there); and the first tensor-core GEMM on a device measures
 *     which SMs share an L2 partition and keeps the result in the library image (see cat_die_map).
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and the call returns without synchronising.
 *   - Argument errors that the host can see return a negative cat_status before anything is
 *     launched; CAT_ERR_CUDA (a failed CUDA call) may come back after part of the work was
 *     enqueued.  Nothing throws.  Conditions only the device can see (a wait inside a kernel that ran
 *     out of time) are written to cat_stats.device_status / the workspace status word;
 *     kernels never trap.
 *   - Layout: H is [T, d] row-major with row pitch ldH elements, W is [V, d] row-major with
 *     row pitch ldW elements.  For CAT_BF16: d % 8 == 0, ldH % 8 == 0, ldW % 8 == 0 and
 *     16-byte aligned base pointers (TMA rules).  For CAT_F32: 4-byte alignment only.
 *   - T % K == 0, K >= 1.  T, V < 2^31; d <= 65536.
 */
#ifndef CAT_LOSS_H_
#define CAT_LOSS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CAT_OK = 0,
    CAT_ERR_NULL = -1,       /* a required pointer is NULL                                  */
    CAT_ERR_SHAPE = -2,      /* T, d, V, K out of range, T % K != 0, pitch < d               */
    CAT_ERR_DTYPE = -3,      /* unknown dtype code or unsupported combination                */
    CAT_ERR_ALIGN = -4,      /* pointer or pitch alignment rule broken                       */
    CAT_ERR_WORKSPACE = -5,  /* workspace NULL or smaller than cat_loss_workspace_bytes()    */
    CAT_ERR_ARCH = -6,       /* current device is not compute capability 10.x                */
    CAT_ERR_CUDA = -7,       /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
    CAT_ERR_TIMEOUT = -8,    /* reported in device_status: a bounded wait in a kernel expired */
    CAT_ERR_LIMIT = -9       /* problem needs more scratch than a fixed-capacity entry point owns */
} cat_status;

typedef enum { CAT_BF16 = 0, CAT_F32 = 1 } cat_dtype;

/* How the per-row weight is formed. */
typedef enum {
    CAT_WEIGHT_CONFIDENCE = 0,   /* Eq. 10: exclusive product of the confidences of the block's earlier rows */
    CAT_WEIGHT_FIXED_DECAY = 1   /* decay_gamma^k for draft position k: the fixed position-wise decay the
                                    paper compares CAT with (Section 4.3, Table 3, gamma_t = gamma^(t-1))   */
} cat_weight_mode;

/* Problem description, read on the host. */
typedef struct {
    int64_t T;         /* rows = draft blocks * K                                   */
    int64_t d;         /* hidden size (contraction length of the logits)             */
    int64_t V;         /* vocabulary size                                            */
    int32_t K;         /* draft positions per block                                  */
    int32_t in_dtype;  /* cat_dtype of H, W and dH.  CAT_BF16: tensor-core path with
                          fp32 accumulation.  CAT_F32: fp32 FFMA path, fp32 throughout */
    int32_t dW_dtype;  /* cat_dtype of dW: CAT_F32 (default) or CAT_BF16 (bf16 inputs only) */
    int32_t slab_mib;  /* cap, in MiB, on the large scratch slab (dz slab of cat_loss_bwd,
                          logits slab of cat_loss_fwd_bwd); 0 = default (2048 / 3072).
                          Smaller caps mean more, smaller slabs.                          */
    int64_t ldH;       /* row pitch of H and dH in elements, >= d                     */
    int64_t ldW;       /* row pitch of W and dW in elements, >= d                     */
    int32_t weight_mode;  /* cat_weight_mode; 0 = the CAT weights of Eq. 10                */
    float   decay_gamma;  /* CAT_WEIGHT_FIXED_DECAY only: weight of position k is the binary32
                             product ((1*gamma)*gamma)*... of k factors; k counts positions, so a
                             masked row still moves the exponent on.  Must be finite and >= 0.
                             conf[] still reports the head's (or conf_ext's) confidences.        */
} cat_shape;

/* Per-call statistics written by cat_loss_fwd (device memory, 32 bytes). */
typedef struct {
    int64_t n_valid;          /* N: rows that took part                                              */
    int64_t n_bad_labels;     /* rows with valid[r] != 0 whose label is outside [0, V)                */
    float   sum_weight;       /* sum_r weight[r]                                                      */
    float   est_accept_len;   /* mean over blocks of sum_k weight*conf: the estimate of Eq. 8         */
    int32_t device_status;    /* CAT_OK or CAT_ERR_TIMEOUT                                            */
    int32_t reserved;
} cat_stats;

/*
 * Bytes of scratch the given pass needs for this shape: pass 0 = cat_loss_fwd,
 * pass 1 = cat_loss_bwd, pass 2 = cat_loss_fwd_bwd, pass 3 = cat_conf_fwd.  Returns 0 if the shape is invalid.  The scratch holds the
 * per-(row, vocabulary split) softmax partials in the forward pass, and in the backward
 * pass one bounded slab of dz (bf16: rows x a slice of the vocabulary, at most about
 * 2 GiB) plus an fp32 dH accumulator when the vocabulary is processed in more than one
 * slab.  It never grows with T*V.
 */
size_t cat_loss_workspace_bytes(const cat_shape* shape, int pass);

/*
 * Forward pass: Eq. 9, Eq. 10, Eq. 11 as written at the top of this file.
 *   H, W      [T, d], [V, d] of shape->in_dtype                               (device, in)
 *   labels    [T] int64 token ids y_r                                          (device, in)
 *   valid     [T] uint8, nonzero = row takes part; NULL = all rows             (device, in)
 *   conf_ext  [T] fp32 confidences computed elsewhere (the paper's target-model
 *             confidences, Eq. 9); NULL = use this head's own probability       (device, in)
 *   loss      [1] fp32                                                          (device, out)
 *   lse       [T] fp32 log-sum-exp of each row's logits                         (device, out)
 *   conf      [T] fp32 confidence used in the product (1 for invalid rows)      (device, out)
 *   weight    [T] fp32 CAT weight, the binary32 left-to-right product of conf
 *             inside each block (0 for invalid rows)                            (device, out)
 *   stats     optional cat_stats                                                (device, out)
 *   workspace at least cat_loss_workspace_bytes(shape, 0) bytes, 256-byte aligned (device, scratch)
 * lse and weight are the only state the backward pass needs.
 * Returns CAT_OK or a negative cat_status.
 */
int cat_loss_fwd(const cat_shape* shape, const void* H, const void* W,
                 const int64_t* labels, const uint8_t* valid, const float* conf_ext,
                 float* loss, float* lse, float* conf, float* weight, cat_stats* stats,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward pass: gradients of g * loss with the weights as constants (stop-gradient,
 * Section 3.2).  The logits are recomputed slice by slice of the vocabulary;
 * dz = weight * (softmax - one-hot) feeds the dH and dW contractions.
 *   lse, weight  [T] fp32 as written by cat_loss_fwd                            (device, in)
 *   grad_loss    [1] fp32 upstream scalar g (e.g. the paper's beta of Eq. 12);
 *                NULL = 1.0                                                      (device, in)
 *   dH           [T, d] of in_dtype, pitch ldH; fully overwritten                (device, out)
 *   dW           [V, d] of dW_dtype, pitch ldW; overwritten, or added to when
 *                accumulate_dW != 0                                              (device, in/out)
 *   workspace    at least cat_loss_workspace_bytes(shape, 1) bytes, 256-byte aligned
 * After the call completes, the first int32 of the workspace holds CAT_OK or
 * CAT_ERR_TIMEOUT (a bounded wait inside a kernel expired; outputs are then undefined).
 * Returns CAT_OK or a negative cat_status.
 */
int cat_loss_bwd(const cat_shape* shape, const void* H, const void* W,
                 const int64_t* labels, const uint8_t* valid,
                 const float* lse, const float* weight, const float* grad_loss,
                 void* dH, void* dW, int accumulate_dW,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * cat_loss_bwd that also tells the caller when each part of dW is final, so that a data-parallel
 * trainer can start summing that part across GPUs while the rest is still being computed.  The
 * backward pass walks the vocabulary in cat_loss_bwd_slabs() slabs; the rows
 * [v_begin[i], v_begin[i+1]) of dW are complete once slab i's dW GEMM has run, and
 * slab_events[i] is recorded on `cuda_stream` right after it.
 *   slab_events  HOST array of n_events cudaEvent_t (as void*), created by the caller        (host, in)
 *   n_events     must equal cat_loss_bwd_slabs(shape, NULL, 0)
 * Everything else as cat_loss_bwd.  dH is final only when the whole call has run.
 */
int cat_loss_bwd_events(const cat_shape* shape, const void* H, const void* W,
                        const int64_t* labels, const uint8_t* valid,
                        const float* lse, const float* weight, const float* grad_loss,
                        void* dH, void* dW, int accumulate_dW,
                        void* workspace, size_t workspace_bytes, void* cuda_stream,
                        void* const* slab_events, int n_events);

/*
 * Number of vocabulary slabs of cat_loss_bwd for this shape (0 if the shape is invalid); if
 * v_begin != NULL the first vocabulary row of up to `capacity` slabs is written to it (host
 * array).  Slab i covers rows [v_begin[i], min(v_begin[i+1], V)).
 */
int cat_loss_bwd_slabs(const cat_shape* shape, int64_t* v_begin, int capacity);

/*
 * N of Eq. 11's batch mean: the number of rows with valid[r] != 0 (or valid == NULL) and
 * 0 <= labels[r] < V, written to *n_valid (device int64).  A data-parallel caller sums it over
 * its ranks to get the global normaliser before the backward pass.  Only T and V of `shape` are used.
 */
int cat_count_valid(const cat_shape* shape, const int64_t* labels, const uint8_t* valid, int64_t* n_valid,
                    void* cuda_stream);

/*
 * Forward and backward in one call, without recomputing the logits (same results as
 * cat_loss_fwd followed by cat_loss_bwd, within rounding).  Rows are processed in slabs of
 * whole draft blocks.  For each slab the logits GEMM also writes e[r, v] = exp(z[r, v] - ref[r]) as
 * bf16, the softmax numerators relative to a per-row reference fixed before the GEMM (the row's
 * label logit, an fp32 dot product).  Once lse and the CAT weights of the slab's blocks are known
 * (Eq. 9, Eq. 10), dz = weight * (softmax - one-hot) is a[r] * e'[r, v] with the per-row factor
 * a[r] = weight[r] * exp(ref[r] - lse[r]) and e' = e with its label entry lowered by
 * exp(lse[r] - ref[r]) (patched in place from the fp32 label logit): the dH GEMM applies a[r] in its
 * epilogue, the dW GEMM takes a[r] * H[r, :] as its second operand, and no second pass over the slab
 * is needed.  dH is written once per slab, dW accumulated over slabs in fp32.  Executed work is the
 * 6*T*d*V flops of the three contractions instead of 8*T*d*V; the price is one slab of 16-bit values
 * in the workspace (at most about slab_mib MiB, default 3072, and always at least two slabs once T
 * exceeds one slab unit, so a T x V matrix never exists at once) and bf16 rounding of the stored
 * numerators (relative 2^-9, the same as rounding dz to bf16).  e is formed as exp(z - m) * exp(m - ref),
 * m the running row maximum, with m - ref capped at 79.7 so that e stays finite for any input: only a
 * row whose label is more than 79.7 nats below
 * the row's largest logit (label probability under 1e-34) gets a damped gradient, and none at all
 * once exp(ref - lse) underflows binary32 (label probability under about 1e-45, where the fp32
 * confidence is zero as well); its loss and lse are exact.  cat_loss_fwd + cat_loss_bwd have no such
 * limit.
 * Arguments as in cat_loss_fwd and cat_loss_bwd; workspace of
 * cat_loss_workspace_bytes(shape, 2) bytes; cat_loss_launch_count(shape, 2) kernels.
 * For CAT_F32 inputs this runs the fp32 forward and backward passes back to back.
 */
int cat_loss_fwd_bwd(const cat_shape* shape, const void* H, const void* W,
                     const int64_t* labels, const uint8_t* valid, const float* conf_ext,
                     const float* grad_loss,
                     float* loss, float* lse, float* conf, float* weight, cat_stats* stats,
                     void* dH, void* dW, int accumulate_dW,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * cat_loss_fwd_bwd with timing marks, for measuring the stages of the one-call path in place (the
 * benchmark uses it to time the dominant GEMM inside its step loop).  The call walks the rows in
 * cat_loss_fused_slabs() slabs; caller-owned events are recorded on `cuda_stream` in this order:
 *     [0] start, [1] after the set-up kernel, then per slab s (base = 2 + 6 s):
 *     [base] label-logit reference, [base+1] logits GEMM, [base+2] row kernel(s) (lse, Eq. 9, Eq. 10),
 *     [base+3] per-row factor / label patch / scaled H rows, [base+4] dH GEMM, [base+5] dW GEMM;
 *     the last one after the final loss reduction.
 *   stage_events  HOST array of n_events cudaEvent_t (as void*), created with timing enabled  (host, in)
 *   n_events      must equal 6 * cat_loss_fused_slabs(shape, NULL, 0) + 3
 * bf16 inputs only.  Everything else, results included, as cat_loss_fwd_bwd.
 */
int cat_loss_fwd_bwd_events(const cat_shape* shape, const void* H, const void* W,
                            const int64_t* labels, const uint8_t* valid, const float* conf_ext,
                            const float* grad_loss,
                            float* loss, float* lse, float* conf, float* weight, cat_stats* stats,
                            void* dH, void* dW, int accumulate_dW,
                            void* workspace, size_t workspace_bytes, void* cuda_stream,
                            void* const* stage_events, int n_events);

/*
 * Number of row slabs of cat_loss_fwd_bwd for this shape (0 if the shape is invalid or not bf16); if
 * row_begin != NULL the first row of up to `capacity` slabs is written to it (host array).  Slab i
 * covers rows [row_begin[i], min(row_begin[i+1], T)).
 */
int cat_loss_fused_slabs(const cat_shape* shape, int64_t* row_begin, int capacity);

/*
 * cat_loss_fwd for callers that cannot hand over a workspace.  (The paper has no counterpart:
 * this is a packaging variant of the forward pass above, same arithmetic, same outputs.)
 *
 * Who needs it: code that runs where device memory may not be allocated at call time -- a
 * plug-in living inside another framework's memory pool that has already claimed the whole
 * GPU, a service whose policy forbids cudaMalloc after start-up because it synchronises the
 * device and can fail late, or a host with a fixed memory budget.  Such callers own their
 * inputs and outputs but have nowhere to get scratch from.
 *
 * Instead of a caller-supplied workspace, the forward pass's scratch (softmax partials per
 * row and vocabulary split, label logits, per-CTA loss partials) lives in one array that is
 * part of the library image: CAT_STATIC_SCRATCH_BYTES of device memory on every GPU that
 * loads the library, held until the process exits.  The call allocates and frees nothing.
 *
 *   - Arguments are those of cat_loss_fwd without `workspace` / `workspace_bytes`.
 *   - Shapes whose cat_loss_workspace_bytes(shape, 0) exceeds CAT_STATIC_SCRATCH_BYTES are
 *     refused with CAT_ERR_LIMIT before anything is launched (config 2, T=16384 x V=128256,
 *     needs 16.7 MB and fits; T=65536 rows of the same head need 33.6 MB and do not).
 *   - The first call on each device looks up the array's device address (once per device,
 *     with that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array and it keeps whatever the last call left in it; the
 *     words that must start at zero are cleared by every call.  Two calls whose GPU work
 *     overlaps (different streams, or different host threads) race on it: serialise them.
 *   - The device status word of this call sits in the built-in array, out of the caller's reach:
 *     pass `stats` to see it (cat_stats.device_status); with stats == NULL a timed-out wait inside
 *     a kernel goes unreported.
 */
#define CAT_STATIC_SCRATCH_BYTES (32u << 20)
int cat_loss_fwd_static(const cat_shape* shape, const void* H, const void* W,
                        const int64_t* labels, const uint8_t* valid, const float* conf_ext,
                        float* loss, float* lse, float* conf, float* weight, cat_stats* stats,
                        void* cuda_stream);

/*
 * Per-block estimate of the expected acceptance length, Eq. 8 with the estimates of Eq. 9 and
 * Eq. 10 in place of the acceptance rates:  accept_len[b] = sum_k weight[bK+k] * conf[bK+k].
 * (cat_stats.est_accept_len is the mean of these.)  Only T and K of `shape` are used.
 *   conf, weight  [T] fp32 as written by cat_loss_fwd / cat_loss_fwd_bwd       (device, in)
 *   accept_len    [T / K] fp32                                                  (device, out)
 * One kernel, no workspace.  Returns CAT_OK or a negative cat_status.
 */
int cat_accept_len(const cat_shape* shape, const float* conf, const float* weight, float* accept_len,
                   void* cuda_stream);

/*
 * Confidence producer for the paper's own reading of Eq. 9: the probability that the TARGET
 * model gives the ground-truth token at every position of the (flattened) training sequences,
 *     conf_seq[i] = softmax(Ht[i, :] . Wt^T)[labels[i]],
 * computed with the same vocabulary-chunked GEMM and online softmax as cat_loss_fwd, never
 * storing the logits.  `shape` describes the target head: T = number of positions L, d = the
 * target's hidden size, V, in_dtype, ldH/ldW pitches; K, dW_dtype and weight_mode are ignored.
 *   Ht, Wt     [L, d], [V, d] target hidden states and target LM head            (device, in)
 *   labels     [L] int64: the token that follows position i's prefix               (device, in)
 *   valid      [L] uint8 or NULL                                                   (device, in)
 *   conf_seq   [L] fp32 (1 for masked positions / labels outside [0, V))           (device, out)
 *   lse_seq    [L] fp32 log-sum-exp of the target logits                           (device, out)
 *   workspace  at least cat_loss_workspace_bytes(shape, 3) bytes, 256-byte aligned
 * Returns CAT_OK or a negative cat_status; the workspace's first int32 holds the device status.
 */
int cat_conf_fwd(const cat_shape* shape, const void* Ht, const void* Wt, const int64_t* labels,
                 const uint8_t* valid, float* conf_seq, float* lse_seq,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Lays per-position confidences out as draft rows, which turns Eq. 10 into the prefix-indexed
 * weight s_{n,k} of Eq. 12 (a product over a window that slides with the prefix position n):
 *     conf_ext[b*K + k] = conf_seq[block_start[b] + k]   if 0 <= block_start[b] + k < L, else 1.
 * Pass the result as `conf_ext` to cat_loss_fwd / cat_loss_fwd_bwd.
 *   conf_seq     [L] fp32                                                         (device, in)
 *   block_start  [n_blocks] int64: index in conf_seq of the block's first drafted token (device, in)
 *   conf_ext     [n_blocks * K] fp32                                              (device, out)
 * One kernel, no workspace.  Returns CAT_OK or a negative cat_status.
 */
int cat_conf_window(const float* conf_seq, int64_t L, const int64_t* block_start, int64_t n_blocks,
                    int32_t K, float* conf_ext, void* cuda_stream);

/*
 * The full training loss of Section 3.3, Eq. 12: cross-entropy plus distillation from the target
 * model, both under the CAT weight,
 *     loss = (1/N) sum_r weight[r] * (beta * CE_r + KD_r),      KD_r = KL(p_t || q_r) = sum_v p_t[v] (log p_t[v] - log q_r[v]),
 * q_r = softmax(H[r,:] W^T) the draft's distribution and p_t = softmax(Ht[t,:] Wt^T) the target's
 * at the sequence position the row predicts.  The paper names the distillation loss without
 * printing it; the forward KL at temperature 1 is this library's reading.  Draft row (block b,
 * position k) refers to target position t = block_start[b] + k, so one row of target logits serves
 * every draft row that predicts that position and the target GEMM covers L positions, not T rows.
 * A row whose target position is outside [0, L) is an invalid row.  Gradients (weights constant,
 * no gradient to the target side):
 *     dz[r, v] = g * weight[r]/N * ((1 + beta) q_r[v] - beta [v == y_r] - p_t[v]),  dH = dz W,  dW = dz^T H.
 * Confidences for the weights (Eq. 9): conf_ext if given; else, by desc->conf_source, the target's
 * probability of the row's label (Eq. 9 as printed) or the draft's own.
 *
 * Works like cat_loss_fwd_bwd (row slabs, logits kept as fp16, three contractions) plus, per slab,
 * a second vocabulary-chunked logits GEMM on the target side whose fp16 logits are kept for the
 * slab.  bf16 inputs only (CAT_ERR_DTYPE otherwise).
 */
typedef enum { CAT_CONF_TARGET = 0, CAT_CONF_DRAFT = 1 } cat_conf_source;

typedef struct {
    int64_t L;            /* target positions = rows of Ht                                      */
    int64_t d_t;          /* target hidden size (d_t % 8 == 0)                                  */
    int64_t ldHt, ldWt;   /* row pitches of Ht and Wt in elements (>= d_t, multiples of 8)      */
    float   beta;         /* weight of the cross-entropy term in Eq. 12 (the paper trains with 0.1) */
    int32_t conf_source;  /* cat_conf_source, used when conf_ext == NULL                        */
} cat_kd_desc;

/*
 * Scratch bytes of cat_kd_loss_fwd_bwd for this problem (0 if anything is invalid).  Needs the
 * block starts because the target slab is sized by the widest range of positions one draft slab
 * refers to.  `block_start_host`: HOST pointer, T/K entries, non-decreasing.
 */
size_t cat_kd_workspace_bytes(const cat_shape* shape, const cat_kd_desc* desc, const int64_t* block_start_host);

/*
 *   shape, H, W, labels, valid, grad_loss, lse, conf, weight, stats, dH, dW, accumulate_dW:
 *                     as in cat_loss_fwd_bwd (device pointers)
 *   desc              target-side sizes, beta, confidence source                        (host, in)
 *   Ht, Wt            [L, d_t], [V, d_t] bf16 target hidden states and target LM head    (device, in)
 *   block_start_host  [T/K] int64, HOST pointer, non-decreasing: sequence position of each block's
 *                     first drafted token.  Read on the host during the call (slab planning) and
 *                     copied to the device by one cudaMemcpyAsync on the stream: keep the array
 *                     unchanged until the stream has passed that copy (for pageable memory that is
 *                     when the call returns, for pinned memory it is not), and do not make this
 *                     call while the stream is being captured.
 *   conf_ext          [T] fp32 or NULL                                                   (device, in)
 *   loss              [3] fp32: total, its cross-entropy part (1/N) sum w CE, its distillation
 *                     part (1/N) sum w KD; total = beta * loss[1] + loss[2]              (device, out)
 *   workspace         at least cat_kd_workspace_bytes(...) bytes, 256-byte aligned       (device, scratch)
 * Returns CAT_OK or a negative cat_status (CAT_ERR_SHAPE also for unsorted block starts).
 */
int cat_kd_loss_fwd_bwd(const cat_shape* shape, const cat_kd_desc* desc, const void* H, const void* W,
                        const int64_t* labels, const uint8_t* valid, const void* Ht, const void* Wt,
                        const int64_t* block_start_host, const float* conf_ext, const float* grad_loss,
                        float* loss, float* lse, float* conf, float* weight, cat_stats* stats,
                        void* dH, void* dW, int accumulate_dW,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Number of kernels of this library that the given pass (0 = cat_loss_fwd, 1 = cat_loss_bwd,
 * 2 = cat_loss_fwd_bwd) launches for this shape: the logits GEMM, the per-row kernels and the final reduction in
 * the forward pass; one set-up kernel plus three GEMMs per vocabulary slab in the backward
 * pass.  Host-only; returns 0 for an invalid shape.
 */
int cat_loss_launch_count(const cat_shape* shape, int pass);

/*
 * What the library has measured about the current device's two L2 partitions (no counterpart in the
 * paper: it concerns how this library's GEMM kernels are placed on a B200).  The first tensor-core GEMM
 * launched on a device is preceded, on the same stream, by two small kernels (about 0.2 ms, once per device
 * and process, skipped while the stream is being captured) that time atomics from every SM and sort the SMs
 * into the two dies; the persistent GEMM kernels then number their CTA pairs die by die, because
 * neighbouring pairs share operand tiles and a tile shared across the dies is fetched into both L2
 * partitions.  Results do not depend on it (every pair claims its index with an atomic and falls back to
 * the next free one); DRAM traffic and time do.  This call runs the measurement if it has not run yet,
 * WAITS for `cuda_stream`, and reports the table:
 *   worker_of_tpc  HOST array of `capacity` int32, or NULL: entry t is the worker index suggested to the CTA
 *                  pair running on SMs 2t and 2t+1                                             (host, out)
 *   n_first_die    HOST int32, or NULL: number of TPCs on the die of SM 0                       (host, out)
 * Returns the number of TPCs the table covers (74 on a full B200), 0 if the measurement was not clean
 * enough to be used (the kernels then number their pairs by blockIdx), or a negative cat_status.
 */
int cat_die_map(int32_t* worker_of_tpc, int capacity, int32_t* n_first_die, void* cuda_stream);

/*
 * Self-test of the error path that cat_stats.device_status / the workspace status word report (no
 * counterpart in the paper: it concerns this library's kernels only).  Every wait inside the
 * tensor-core kernels is bounded; one that runs out raises an abort flag that the other warp roles
 * of the CTA watch, records CAT_ERR_TIMEOUT, and the CTA (or CTA pair) leaves through the normal
 * teardown.  This call runs exactly that sequence -- the GEMM kernel's set-up, role split, bounded
 * waits, abort flag and teardown -- in one CTA (or one pair, as the GEMMs are configured) with no
 * copy and no tensor-core work in flight, around barriers that nothing signals:
 *   role        0 = the TMA-producer lane, 1 = the MMA-issuing lane, 2 = the epilogue warps: the role
 *               whose wait gets the limit short_ns; the others get long_ns and must leave early,
 *               through the abort flag
 *   short_ns    1 .. 1e8 (0.1 s);  long_ns  short_ns .. 5e9: anything else is CAT_ERR_SHAPE
 *   status      [1] int32: cleared by the call, CAT_ERR_TIMEOUT once the kernel has run  (device, out)
 *   elapsed_ns  [12] uint64, entry cta * 6 + warp: nanoseconds that warp waited; bit 63 is set if
 *               its wait was (wrongly) satisfied; one CTA writes 6 entries, a pair 12     (device, out)
 * The kernel returns by itself after about short_ns; nothing traps and the context stays usable.
 */
int cat_selftest_wait_timeout(int role, uint64_t short_ns, uint64_t long_ns, int32_t* status,
                              uint64_t* elapsed_ns, void* cuda_stream);

/* Static, NUL-terminated description of a cat_status value (host pointer, never freed). */
const char* cat_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* CAT_LOSS_H_ */
