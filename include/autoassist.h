/*
 * autoassist.h — C ABI of the B200 (sm_100a) instance-shrinking batch generator of
 * AutoAssist (Zhang, Yu, Dhillon, arXiv 1905.03381).
 *
 * One training step of the generator, as the paper defines it:
 *   1. score a pool of candidate instances with the light-weight Assistant g(x; phi)
 *      (Sec. "Learning to generate smart training batches"; logistic regression in Sec. "Image classification", bag-of-words classifier in Sec. "Machine Translation"),
 *   2. accept each candidate by the Bernoulli rule of Algorithm 1 (Assistant.sample_batch)
 *      with base probability gamma, i.e. with probability gamma + (1 - gamma) g,
 *   3. append the accepted candidates to the batch B in list order (Algorithm 1),
 *   4. obtain the Boss's loss f on every instance of B (Sec. "Asynchronous joint learning with CPU/GPU": the (i, f_i) pairs pushed
 *      to the AssistantQueue) — here: row cross-entropy of caller-supplied logits, summed
 *      over the token rows of a sentence for sequence tasks,
 *   5. turn the losses into labels z = 1[f > T] (Sec. "Learning to generate smart training batches") and take one gradient step on the
 *      Assistant's cross-entropy objective (Eq. "sec-loss"; Algorithm 2: gradient, update).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless a comment says HOST.
 *     The library never allocates or frees device memory; scratch space is the caller's
 *     workspace handed to aa_create.
 *   - Every call only enqueues kernels on the context's CUDA stream and returns.  Results
 *     are ordered after earlier work on that stream.  out_count is a device scalar, so no
 *     call forces a host synchronisation.
 *   - Argument errors return a non-zero aa_status at once and enqueue nothing.  Conditions
 *     found on the device (scan wait gave up, label or column out of range, more survivors
 *     than capacity) latch a code in a device status word that aa_device_status reads;
 *     no kernel traps or aborts.
 *   - One context per stream; calls on one context must not overlap in time.  Screening calls of
 *     two contexts that overlap on one GPU are allowed, but each sizes its grid for an idle GPU:
 *     when they compete for SMs a look-back wait can run out, which latches AA_ERR_SCAN_TIMEOUT
 *     (the batch of that call is invalid; repeat the call).
 *   - out_idx, out_count and the mask are pure functions of (features, parameters, mix,
 *     seed, step, id_base): Philox4x32-10 is keyed by seed with counter (instance id, step).
 */
#ifndef AUTOASSIST_H
#define AUTOASSIST_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct aa_ctx aa_ctx;

typedef enum {
    AA_OK = 0,
    AA_ERR_INVALID_ARG = 1,   /* null pointer, negative size, misaligned or inconsistent argument */
    AA_ERR_UNSUPPORTED = 2,   /* valid request this build has no kernel for */
    AA_ERR_CUDA = 3,          /* a CUDA runtime call failed */
    AA_ERR_WORKSPACE = 4,     /* workspace too small for this call */
    AA_ERR_SCAN_TIMEOUT = 5,  /* device: a tile gave up waiting for its predecessor's prefix */
    AA_ERR_BAD_INDEX = 6,     /* device: label >= cols, CSR column >= d, or row index out of range */
    AA_ERR_CAPACITY = 7       /* device: more survivors than out_idx capacity (count is still exact) */
} aa_status;

typedef enum { AA_F32 = 0, AA_BF16 = 1 } aa_dtype;
typedef enum { AA_FEAT_DENSE = 0, AA_FEAT_CSR = 1 } aa_feat_kind;
typedef enum { AA_ASSIST_LINEAR = 0, AA_ASSIST_MLP = 1 } aa_assist_kind;
typedef enum { AA_THRESH_VALUE = 0, AA_THRESH_BATCH_MEAN = 1 } aa_thresh_mode;

/*
 * Feature rows of the candidate instances (the x_i that g(x_i; phi) is evaluated on, Sec. "Learning to generate smart training batches").
 * Dense: row-major [n x d], element type dtype, row r starts at dense + r*row_stride elements.
 *        The 128-bit load path needs dense 16-byte aligned and row_stride*sizeof(element)
 *        a multiple of 16; anything else takes a slower element-wise path.
 * CSR:   indptr[n+1], col[nnz] in [0, d), val[nnz] fp32 (the bag-of-words counts of Sec. "Machine Translation").
 *        Repeated columns in a row add.  nnz = indptr[n] as known on the host (it only steers
 *        how many lanes share a row; 0 = unknown).
 * row_idx: optional candidate list.  Candidate k is stored row row_idx[k], k in [0, n_rows)
 *        (the slice of the shuffled index list that Sec. "Learning to generate smart training batches" walks).  NULL: candidate k is
 *        row k and n_rows is ignored.
 * id_base: instance id of stored row 0.  The Philox counter of a candidate is id_base + row,
 *        so a shard of a larger data set draws the same decisions as the whole.
 */
typedef struct {
    int32_t kind;            /* aa_feat_kind */
    int32_t dtype;           /* aa_dtype of dense values */
    int64_t n;               /* stored rows */
    int64_t d;               /* feature dimension */
    const void* dense;
    int64_t row_stride;      /* elements */
    const int32_t* indptr;
    const int32_t* col;
    const float* val;
    int64_t nnz;
    const int32_t* row_idx;
    int64_t n_rows;
    int64_t id_base;
} aa_feat;

/*
 * Assistant parameters phi, caller-owned, updated in place by aa_assistant_step.
 * Linear (logistic regression / bag-of-words): g = sigmoid(w . x + b), w[d] and b[1] fp32.
 * MLP: g = sigmoid(w2 . relu(W1 x + b1) + b2); W1 is [hidden x d] row-major (one hidden unit
 *      per row), kept as an fp32 master W1 and a bf16 copy W1_bf16 that scoring reads;
 *      b1[hidden], w2[hidden], b2[1] fp32.  (The paper only asks for a light-weight model,
 *      Secs. "Assistant for instance selection" and "Learning to generate smart training batches"; the two-layer form is this library's dense-contraction case.)
 */
typedef struct {
    int32_t kind;            /* aa_assist_kind */
    int32_t reserved;
    int64_t d;
    int64_t hidden;
    float* w;
    float* b;
    float* W1;
    void* W1_bf16;
    float* b1;
    float* w2;
    float* b2;
} aa_assistant;

/* Boss outputs for the batch: row-major [rows x cols] logits, row r at data + r*row_stride elements. */
typedef struct {
    const void* data;
    int32_t dtype;           /* aa_dtype */
    int32_t reserved;
    int64_t rows;
    int64_t cols;
    int64_t row_stride;      /* elements */
} aa_logits;

/* HOST string for a status code. */
const char* aa_status_string(aa_status s);

/*
 * Bytes of device workspace a context needs to serve pools of up to max_rows candidates /
 * logit rows, feature dimension up to max_d and hidden width up to max_hidden (0 if the MLP
 * Assistant is not used).  bytes is a HOST pointer.
 */
aa_status aa_workspace_bytes(int64_t max_rows, int64_t max_d, int64_t max_hidden, size_t* bytes);

/*
 * Create a context on the current device for the same limits that sized the workspace.
 * workspace: device memory of at least aa_workspace_bytes(max_rows, max_d, max_hidden) bytes,
 * 256-byte aligned, owned by the caller and kept alive until aa_destroy; its control block is
 * cleared on the stream here (the call synchronises the stream once).  cuda_stream: a
 * cudaStream_t (NULL = the legacy default stream).  ctx is a HOST pointer.
 */
aa_status aa_create(aa_ctx** ctx, int64_t max_rows, int64_t max_d, int64_t max_hidden,
                    void* workspace, size_t bytes, void* cuda_stream);
aa_status aa_destroy(aa_ctx* ctx);

/*
 * Steps 1-3 fused: Assistant score, Bernoulli shrink (Algorithm 1), ordered batch list.
 *   keep_k  = (c < mix) or ((c - mix)/(1 - mix) < g_k)   <=>   c < mix + (1 - mix) g_k,
 *   c       = top 24 bits of Philox4x32-10(key = seed, counter = (id_base + row_k, step)) * 2^-24,
 * evaluated in fp32.  out_idx[0..M) receives the stored row numbers of the kept candidates in
 * candidate order (ascending when row_idx is NULL); out_count[0] = M.  capacity = entries
 * out_idx can hold; survivors beyond it are counted but not written and AA_ERR_CAPACITY is
 * latched.  out_score (nullable): fp32 pre-activation s_k per candidate.  out_mask (nullable):
 * one byte per candidate, 1 = kept.  mix in [0, 1].
 */
aa_status aa_score_shrink(aa_ctx* ctx, const aa_feat* feat, const aa_assistant* assistant, float mix,
                          uint64_t seed, uint64_t step,
                          int32_t* out_idx, int64_t capacity, int32_t* out_count,
                          float* out_score, uint8_t* out_mask);

/*
 * Steps 2-3 alone on precomputed pre-activations score[0..n): same rule, same outputs.
 * Candidate k has instance id id_base + k.
 */
aa_status aa_shrink_compact(aa_ctx* ctx, const float* score, int64_t n, int64_t id_base, float mix,
                            uint64_t seed, uint64_t step,
                            int32_t* out_idx, int64_t capacity, int32_t* out_count, uint8_t* out_mask);

/*
 * Hard shrinking (Sec. "Instance Shrinking in Stochastic Gradient Descent", Eq. "shrinking_grad"; the SK method of Sec. "Shrinking experiment under convex setting"): an instance is used
 * only if its objective value or gradient magnitude is at least T.  value[i] is that quantity for
 * instance i (e.g. the losses of aa_instance_loss); out_idx receives the ascending list of i with
 * value[i] >= threshold, out_count its length, out_mask (nullable) one byte per instance.  No random
 * draw is involved; NaN values are dropped.  Capacity overflow latches AA_ERR_CAPACITY as in
 * aa_score_shrink.  aa_sk_threshold gives the schedule T_k = G / k of the convergence theorem
 * (Sec. "Theoretical Analysis", Theorem 1) for step k >= 1 (HOST helper).
 */
aa_status aa_threshold_compact(aa_ctx* ctx, const float* value, int64_t n, float threshold,
                               int32_t* out_idx, int64_t capacity, int32_t* out_count, uint8_t* out_mask);
float aa_sk_threshold(float G, int64_t k);

/*
 * Batch cut + cursor: the batch Algorithm 1 (Assistant.sample_batch) returns, cut out of the ordered
 * survivor list of a screened pool.  Algorithm 1 stops as soon as the batch holds batch_size
 * instances, so its batch is the first batch_size entries of the list and its walk over the
 * (shuffled) candidate list ends right after the last one taken; the next call starts there.
 * For sequence tasks (Sec. "Machine Translation": batches of a given number of tokens) the batch is the longest prefix
 * of the list whose sentence lengths add up to at most token_budget.
 *   idx, count_dev : out_idx / out_count of aa_score_shrink (candidate k = stored row k, i.e. no
 *                    candidate list); idx_capacity bounds the device count.  n_cand = pool size.
 *   batch_size     : most instances in the batch (0 = no limit).
 *   lengths        : nullable; lengths[r] = tokens of stored row r (n_stored rows, negative counts
 *                    as 0); with it token_budget applies.  A list entry outside the rows latches
 *                    AA_ERR_BAD_INDEX and counts as length 0.
 *   out_m[0]       : instances in the batch, b.
 *   out_consumed[0]: candidates the walk covered: idx[b-1] + 1 when a limit ended it (0 if not even
 *                    the first survivor fits), n_cand when the survivors ran out first.
 *   out_offsets    : nullable (needs lengths), offsets_capacity entries: out_offsets[k] = tokens of
 *                    the first k batch instances, k = 0..b — the offsets aa_instance_loss takes.
 * All outputs are device memory; nothing is read back.
 */
aa_status aa_batch_cut(aa_ctx* ctx, const int32_t* idx, const int32_t* count_dev, int64_t idx_capacity, int64_t n_cand,
                       int64_t batch_size, const int32_t* lengths, int64_t n_stored, int64_t token_budget,
                       int32_t* out_m, int32_t* out_consumed, int32_t* out_offsets, int64_t offsets_capacity);

/*
 * aa_shrink_compact for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of the entry point above.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits — a plug-in or callback inside a
 * host application that owns the whole memory pool, a real-time loop that must not enter the
 * allocator, a process that starts after the device memory has been handed out.  Such a caller
 * cannot provide the workspace that aa_create wants, so this variant takes no context: its scan
 * state (a control block and one look-back word per 1024-candidate tile, 33 KB) is a fixed array
 * inside the library, present on every device that loads the library for the life of the process.
 * The call itself allocates and frees nothing on host or device.
 *
 *   - n may be at most AA_STATIC_MAX_CANDIDATES; a larger n returns AA_ERR_WORKSPACE and enqueues
 *     nothing.  Split a larger pool into consecutive calls with id_base advanced by the rows done.
 *   - Inputs and outputs are the caller's device buffers exactly as for aa_shrink_compact; results
 *     are bit-identical to it for the same arguments.
 *   - out_status (nullable, device int32): receives the condition latched by this call
 *     (AA_OK, AA_ERR_CAPACITY, AA_ERR_SCAN_TIMEOUT), ordered on the stream like the other outputs.
 *   - cuda_stream: the cudaStream_t to enqueue on (NULL = legacy default stream), on the CURRENT device.
 *   - The first call on each device looks up the array's device address and the launch shape
 *     (a few host-side CUDA queries); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call clears the part it uses before its
 *     kernel runs, so calls that follow each other on one stream are independent; calls that can
 *     overlap on the GPU (different streams, different host threads without ordering) race on the
 *     array and give wrong batches.  Serialise them.
 */
#define AA_STATIC_MAX_CANDIDATES (1 << 22)
aa_status aa_shrink_compact_static(const float* score, int64_t n, int64_t id_base, float mix,
                                   uint64_t seed, uint64_t step,
                                   int32_t* out_idx, int64_t capacity, int32_t* out_count, uint8_t* out_mask,
                                   int32_t* out_status, void* cuda_stream);

/*
 * Step 4: per-instance Boss loss.  Row r: l_r = log sum_c exp(logit[r][c]) - logit[r][labels[r]]
 * (one pass, running maximum, fp32).  labels[r] < 0 marks padding (contributes 0); labels[r] >=
 * cols contributes 0 and latches AA_ERR_BAD_INDEX.
 *   offsets == NULL: out_loss[r] = l_r for r in [0, rows).
 *   offsets != NULL: offsets[n_seg+1] ascending token-row offsets; out_loss[s] = sum of l_r over
 *                    rows [offsets[s], offsets[s+1]) (a sentence's summed token loss); an empty
 *                    segment gives 0.
 * count_dev (nullable): device int32; only the first min(*count_dev, rows) rows (offsets == NULL)
 * are evaluated — lets the accepted count of aa_score_shrink size the work without a host read.
 */
aa_status aa_instance_loss(aa_ctx* ctx, const aa_logits* logits, const int32_t* labels,
                           const int32_t* offsets, int64_t n_seg, const int32_t* count_dev,
                           float* out_loss);

/*
 * Step 4 on a batch list: the Boss losses of the batch instances when the logits (and labels) are
 * stored for the whole pool (Sec. "Asynchronous joint learning with CPU/GPU": the losses {f(x_i, y_i)} of the instances i in B).
 *   out_loss[k] = l_r with r = row_idx[k], for k in [0, M), M = min(*count_dev, n_rows) when
 *   count_dev is given, else n_rows; labels[r] is the label of stored row r.
 * row_idx: device int32 list (e.g. out_idx of aa_score_shrink); an entry outside [0, logits->rows)
 * gives 0 and latches AA_ERR_BAD_INDEX.  Label rules as in aa_instance_loss.  out_loss holds
 * n_rows entries; entries at and beyond M are left untouched.
 */
aa_status aa_instance_loss_rows(aa_ctx* ctx, const aa_logits* logits, const int32_t* labels,
                                const int32_t* row_idx, int64_t n_rows, const int32_t* count_dev,
                                float* out_loss);

/*
 * Step 5: labels and one SGD step of the Assistant on the batch (Algorithm 2: gradient, update).
 * Batch instance i is stored row feat->row_idx[i] (or row i), i in [0, M), M = min(*count_dev,
 * feat->n_rows) when count_dev is given, else feat->n_rows (or feat->n without row_idx).
 *   T   = threshold (AA_THRESH_VALUE) or the mean of loss[0..M) (AA_THRESH_BATCH_MEAN),
 *   z_i = 1 if loss[i] > T else 0,  r_i = sigmoid(s_i) - z_i under the CURRENT parameters,
 *   w  <- w - lr * (1/M) sum_i r_i x_i,   b <- b - lr * (1/M) sum_i r_i   (MLP: back-propagated
 *   through both layers, fp32 masters updated, W1_bf16 re-rounded to nearest even).
 * M = 0 leaves the parameters unchanged.
 */
aa_status aa_assistant_step(aa_ctx* ctx, const aa_feat* feat, const float* loss, const int32_t* count_dev,
                            aa_assistant* assistant, float lr, int32_t thresh_mode, float threshold);

/*
 * Step 5 for the sequential schedule, where the parameters have not changed since the pool was screened
 * (Algorithm 1 evaluates g(x_i; phi) for the candidates; Algorithm 2's gradient needs the same g(x_i; phi) for the
 * batch instances as long as phi is the same): score[r] is the pre-activation s_r of STORED row r under the current
 * parameters, as aa_score_shrink wrote it to out_score when it screened these rows without a candidate list.  The
 * residual of batch instance i is then r_i = sigmoid(score[row_i]) - z_i and the dot products are not recomputed;
 * everything else is aa_assistant_step.  The caller vouches that score belongs to the current parameters: after any
 * update in between (a deeper Boss queue, a second step on one screen) use aa_assistant_step.  score = NULL is
 * aa_assistant_step.  Kernels that have no use for the scores (CSR rows, rows that are not 16-byte aligned bf16 of
 * 256..3072 features) recompute the pre-activations, so the result is the same up to rounding.
 *
 * Two-layer Assistant: back-propagation also needs the gates [a_iu > 0] of the hidden layer.  aa_score_shrink leaves
 * them in this context's workspace (one bit per stored row and hidden unit) whenever it screens a dense pool without a
 * candidate list.  The step uses score and those gates, and runs no forward pass, when the LAST two-layer screening on
 * this context covered exactly these features (same base pointer, row count and W1_bf16 pointer), no two-layer update
 * has gone through the context since, d is a multiple of 128 and the fp32 W1 is 16-byte aligned; grad w2 then comes
 * from  sum_i r_i relu(a_iu) = sum_k W1b_uk G_uk + b1_u sum_i r_i [a_iu > 0]  with G the W1-gradient contraction.  In
 * every other case the forward pass is evaluated as in aa_assistant_step and score is not read.
 */
aa_status aa_assistant_step_scored(aa_ctx* ctx, const aa_feat* feat, const float* loss, const int32_t* count_dev,
                                   const float* score, aa_assistant* assistant, float lr, int32_t thresh_mode,
                                   float threshold);

/*
 * Step 5 with Adam in place of SGD (the paper trained its Assistants with Adam, Sec. "Image classification").  Labels and gradient exactly as
 * in aa_assistant_step; the update of every parameter p with mean gradient g is
 *   m <- beta1 m + (1 - beta1) g,   v <- beta2 v + (1 - beta2) g^2,
 *   p <- p - lr (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps),      t = state->t + 1,
 * in fp32.  state (HOST struct) is caller-owned: m and v are DEVICE arrays laid out like the flattened parameters
 * (linear: w[d] then b, d + 1 floats; two-layer: W1[hidden*d], b1[hidden], w2[hidden], b2, hidden*(d+2) + 1 floats),
 * zero before the first step; the call advances state->t.  A batch that turns out empty on the device leaves parameters
 * and moments unchanged (t still advances).  With CSR features every weight is updated, not only the batch's columns:
 * a first moment keeps moving its weight while it decays.
 */
typedef struct {
    float beta1, beta2, eps;
    int32_t reserved;
    int64_t t;               /* steps taken so far */
    float* m;
    float* v;
} aa_adam;
aa_status aa_assistant_step_adam(aa_ctx* ctx, const aa_feat* feat, const float* loss, const int32_t* count_dev,
                                 aa_assistant* assistant, aa_adam* state, float lr, int32_t thresh_mode, float threshold);

/*
 * Feature map of the convolutional Assistant (Sec. "Learning to generate smart training batches", closing paragraph:
 * for image tasks the Assistant may be a convolution layer that shares its parameters with the Boss, followed by a
 * pooling layer and a single linear layer).  The paper gives no sizes; this library's reading:
 *   images : dense rows (fp32 or bf16), one instance per row, stored channel-major: element (ci * height + y) * width + x;
 *            images->d = c_in * height * width; images->row_idx must be NULL (every stored row is evaluated).
 *   conv   : the Boss's convolution: weight[c_out][c_in][ksize][ksize] and bias[c_out] (nullable) in fp32, DEVICE memory,
 *            ksize 1, 3 or 5, stride 1, zero padding (ksize - 1) / 2, followed by the rectifier max(., 0);
 *            pool: side of the non-overlapping average-pooling windows (divides height and width).
 *   out_phi: row i receives phi_i[co][y / pool][x / pool] (c_out * (height / pool) * (width / pool) fp32 values),
 *            rows phi_stride elements apart.
 * The single linear layer is the linear Assistant on phi: screen with aa_score_shrink on a dense fp32 descriptor of
 * out_phi, update with aa_assistant_step on the same (only that layer trains; the convolution weights stay the Boss's).
 */
typedef struct {
    int32_t c_in, height, width;
    int32_t c_out, ksize, pool;
    const float* weight;
    const float* bias;
} aa_conv;
aa_status aa_conv_pool_features(aa_ctx* ctx, const aa_feat* images, const aa_conv* conv, float* out_phi, int64_t phi_stride);

/*
 * One whole step for callers whose data lives in HOST memory (pinned memory for full copy speed):
 * copies the candidate features, the Boss logits and the labels to the device staging buffer,
 * runs steps 1-5 above (dense linear Assistant), copies the batch list, its count, the
 * per-instance losses and nothing else back, and synchronises the stream before returning.
 *   feat->dense, logits->data, labels, out_idx, out_count, out_loss: HOST pointers.
 *   logits holds one row per candidate of the pool; row k is the Boss output for the k-th
 *   accepted instance (the first M rows are used).  feat->row_idx must be NULL.
 *   assistant: DEVICE parameters, updated in place.  staging: DEVICE memory of at least
 *   aa_step_host_staging_bytes(...) bytes, 256-byte aligned, owned by the caller.
 *   out_idx holds feat->n entries, out_loss feat->n entries, out_count one.
 */
aa_status aa_step_host_staging_bytes(const aa_feat* feat, const aa_logits* logits, size_t* bytes);
aa_status aa_step_host(aa_ctx* ctx, const aa_feat* feat, aa_assistant* assistant, float mix,
                       uint64_t seed, uint64_t step, const aa_logits* logits, const int32_t* labels,
                       float lr, int32_t thresh_mode, float threshold,
                       int32_t* out_idx, int32_t* out_count, float* out_loss,
                       void* staging, size_t staging_bytes);

/*
 * Synchronises the context's stream, returns the first device-side condition latched since the
 * last call in *latched (HOST pointer; AA_OK if none) and clears it.
 */
aa_status aa_device_status(aa_ctx* ctx, int32_t* latched);

/* Kernels launched through this context so far (HOST counter). */
int64_t aa_launch_count(const aa_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* AUTOASSIST_H */
