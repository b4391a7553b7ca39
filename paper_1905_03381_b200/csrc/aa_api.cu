// C ABI of the AutoAssist batch-generator library: context, workspace layout, argument checks.
// Every entry point validates on the host, then enqueues kernels on the context's stream.
#include <new>
#include <stdio.h>
#include <math.h>
#include <string.h>

#include "aa_internal.cuh"

namespace aa {

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    size_t tile_state_off, row_scratch_off, partials_off, total;
    size_t mlp_pt_off, mlp_small_off, mlp_part_off, mlp_part_bytes, mlp_gate_off;   // two-layer Assistant step (max_hidden > 0)
    int64_t max_tiles, partial_floats;
};

Layout make_layout(int64_t max_rows, int64_t max_d, int64_t max_hidden) {
    Layout L;
    L.max_tiles = (max_rows + 15) / 16 + 1;   // the smallest compaction tile is 16 candidates
    size_t off = sizeof(Control);
    L.tile_state_off = off;
    off = align_up(off + sizeof(unsigned long long) * (size_t)L.max_tiles, 256);
    L.row_scratch_off = off;
    off = align_up(off + sizeof(float) * (size_t)(max_rows > 0 ? max_rows : 1), 256);
    L.partials_off = off;
    // per-CTA gradient partials: up to kMaxParts copies of a padded weight vector, at most 64 MiB
    const int64_t d_pad = max_d + 9;
    int64_t floats = (int64_t)kMaxParts * d_pad;
    const int64_t cap = (64ll << 20) / 4;
    if (floats > cap) floats = cap;
    if (floats < 2 * d_pad) floats = 2 * d_pad;
    L.partial_floats = floats;
    off = align_up(off + sizeof(float) * (size_t)floats, 256);
    L.mlp_pt_off = L.mlp_small_off = L.mlp_part_off = L.mlp_part_bytes = L.mlp_gate_off = 0;
    if (max_hidden > 0) {
        size_t pt_bytes = 0, small_bytes = 0;
        L.mlp_part_bytes = mlp_step_workspace_bytes(max_rows, max_d, max_hidden, &pt_bytes, &small_bytes, &L.mlp_gate_off);
        L.mlp_pt_off = off;    off = align_up(off + pt_bytes, 1024);
        L.mlp_small_off = off; off = align_up(off + small_bytes, 256);
        L.mlp_part_off = off;  off = align_up(off + L.mlp_part_bytes, 256);
    }
    L.total = off;
    return L;
}

struct OccEntry {
    const void* kernel;
    int threads;
    size_t smem;
    int ctas;
};
constexpr int kOccSlots = 64;

}  // namespace

}  // namespace aa

struct aa_ctx {
    aa::aa_ctx_impl impl;
    aa::OccEntry occ[aa::kOccSlots];
    int occ_used;
};

namespace aa {

int resident_ctas(aa_ctx_impl* c, const void* kernel, int threads, size_t dyn_smem) {
    aa_ctx* ctx = reinterpret_cast<aa_ctx*>(c);   // impl is the first member
    for (int i = 0; i < ctx->occ_used; ++i) {
        const OccEntry& e = ctx->occ[i];
        if (e.kernel == kernel && e.threads == threads && e.smem == dyn_smem) return e.ctas;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, dyn_smem) != cudaSuccess) return -1;
    if (per_sm < 1) return -1;
    const int ctas = per_sm * c->sm_count;
    if (ctx->occ_used < kOccSlots) ctx->occ[ctx->occ_used++] = OccEntry{kernel, threads, dyn_smem, ctas};
    return ctas;
}

cudaError_t launch_overlapped(aa_ctx_impl* c, const void* kernel, dim3 grid, dim3 block, void** args, size_t smem, bool cooperative) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute attrs[2];
    unsigned int n = 0;
    attrs[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cooperative) {
        attrs[n].id = cudaLaunchAttributeCooperative;
        attrs[n].val.cooperative = 1;
        ++n;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = n;
    return cudaLaunchKernelExC(&cfg, kernel, args);
}

namespace {

bool valid_mix(float mix) { return mix >= 0.0f && mix <= 1.0f; }

// Fills the parts of ShrinkParams that come from the caller's arguments.
aa_status base_shrink_params(ShrinkParams& sp, int64_t n_cand, int64_t n_stored, const int32_t* row_idx, int64_t id_base,
                             float mix, uint64_t seed, uint64_t step, int32_t* out_idx, int64_t capacity,
                             int32_t* out_count, float* out_score, uint8_t* out_mask) {
    if (!out_count || capacity < 0 || (capacity > 0 && !out_idx) || !valid_mix(mix)) return AA_ERR_INVALID_ARG;
    if (n_cand < 0 || n_cand > 0x7FFFFFFFll) return AA_ERR_INVALID_ARG;
    memset(&sp, 0, sizeof sp);
    sp.n_cand = n_cand;
    sp.n_stored = n_stored;
    sp.row_idx = row_idx;
    sp.id_base = id_base;
    sp.mix = mix;
    sp.seed_lo = (uint32_t)seed;
    sp.seed_hi = (uint32_t)(seed >> 32);
    sp.step_lo = (uint32_t)step;
    sp.step_hi = (uint32_t)(step >> 32);
    sp.out_idx = out_idx;
    sp.capacity = capacity;
    sp.out_count = out_count;
    sp.out_score = out_score;
    sp.out_mask = out_mask;
    return AA_OK;
}

aa_status check_feat(const aa_feat* f) {
    if (!f || f->n < 0 || f->d <= 0 || f->n > 0x7FFFFFFFll) return AA_ERR_INVALID_ARG;
    if (f->kind == AA_FEAT_DENSE) {
        if (f->dtype != AA_F32 && f->dtype != AA_BF16) return AA_ERR_INVALID_ARG;
        if (f->n > 0 && (!f->dense || f->row_stride < f->d)) return AA_ERR_INVALID_ARG;
        const uintptr_t es = f->dtype == AA_BF16 ? 2 : 4;
        if ((uintptr_t)f->dense % es) return AA_ERR_INVALID_ARG;
    } else if (f->kind == AA_FEAT_CSR) {
        if (!f->indptr || (f->n > 0 && (!f->col || !f->val))) return AA_ERR_INVALID_ARG;
    } else {
        return AA_ERR_INVALID_ARG;
    }
    if (f->row_idx && (f->n_rows < 0 || f->n_rows > 0x7FFFFFFFll)) return AA_ERR_INVALID_ARG;
    return AA_OK;
}

}  // namespace
}  // namespace aa

using namespace aa;

extern "C" {

const char* aa_status_string(aa_status s) {
    switch (s) {
        case AA_OK: return "ok";
        case AA_ERR_INVALID_ARG: return "invalid argument";
        case AA_ERR_UNSUPPORTED: return "unsupported configuration";
        case AA_ERR_CUDA: return "CUDA runtime error";
        case AA_ERR_WORKSPACE: return "workspace too small";
        case AA_ERR_SCAN_TIMEOUT: return "device: look-back wait gave up";
        case AA_ERR_BAD_INDEX: return "device: label, column or row index out of range";
        case AA_ERR_CAPACITY: return "device: more survivors than out_idx capacity";
    }
    return "unknown status";
}

aa_status aa_workspace_bytes(int64_t max_rows, int64_t max_d, int64_t max_hidden, size_t* bytes) {
    if (!bytes || max_rows < 0 || max_d <= 0 || max_hidden < 0) return AA_ERR_INVALID_ARG;
    *bytes = make_layout(max_rows, max_d, max_hidden).total;
    return AA_OK;
}

aa_status aa_create(aa_ctx** out, int64_t max_rows, int64_t max_d, int64_t max_hidden, void* workspace, size_t bytes,
                    void* cuda_stream) {
    if (!out || !workspace || max_rows < 0 || max_d <= 0 || max_hidden < 0) return AA_ERR_INVALID_ARG;
    if ((uintptr_t)workspace % 256) return AA_ERR_INVALID_ARG;
    const Layout L = make_layout(max_rows, max_d, max_hidden);
    if (bytes < L.total) return AA_ERR_WORKSPACE;
    aa_ctx* ctx = new (std::nothrow) aa_ctx();
    if (!ctx) return AA_ERR_CUDA;
    memset(ctx, 0, sizeof *ctx);
    aa_ctx_impl& c = ctx->impl;
    if (cudaGetDevice(&c.device) != cudaSuccess ||
        cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, c.device) != cudaSuccess) {
        delete ctx;
        return AA_ERR_CUDA;
    }
    c.ws = static_cast<char*>(workspace);
    c.ws_bytes = bytes;
    c.stream = static_cast<cudaStream_t>(cuda_stream);
    c.max_rows = max_rows;
    c.max_d = max_d;
    c.max_hidden = max_hidden;
    c.ctl = reinterpret_cast<Control*>(c.ws);
    c.tile_state = reinterpret_cast<unsigned long long*>(c.ws + L.tile_state_off);
    c.max_tiles = L.max_tiles;
    c.row_scratch = reinterpret_cast<float*>(c.ws + L.row_scratch_off);
    c.partials = reinterpret_cast<float*>(c.ws + L.partials_off);
    c.partial_floats = L.partial_floats;
    if (max_hidden > 0) {
        c.mlp_pt = c.ws + L.mlp_pt_off;
        c.mlp_gate_cand = reinterpret_cast<uint32_t*>(c.ws + L.mlp_pt_off + L.mlp_gate_off);
        c.mlp_small = reinterpret_cast<float*>(c.ws + L.mlp_small_off);
        c.mlp_part = reinterpret_cast<float*>(c.ws + L.mlp_part_off);
        c.mlp_part_bytes = L.mlp_part_bytes;
    }
    // control block and look-back flags start cleared; the flag generation starts at 1
    if (cudaMemsetAsync(c.ws, 0, L.row_scratch_off, c.stream) != cudaSuccess) {
        delete ctx;
        return AA_ERR_CUDA;
    }
    const unsigned int one = 1;
    if (cudaMemcpyAsync(&c.ctl->epoch, &one, sizeof one, cudaMemcpyHostToDevice, c.stream) != cudaSuccess ||
        cudaStreamSynchronize(c.stream) != cudaSuccess) {
        delete ctx;
        return AA_ERR_CUDA;
    }
    *out = ctx;
    return AA_OK;
}

aa_status aa_destroy(aa_ctx* ctx) {
    if (!ctx) return AA_ERR_INVALID_ARG;
    delete ctx;
    return AA_OK;
}

aa_status aa_score_shrink(aa_ctx* ctx, const aa_feat* feat, const aa_assistant* a, float mix, uint64_t seed, uint64_t step,
                          int32_t* out_idx, int64_t capacity, int32_t* out_count, float* out_score, uint8_t* out_mask) {
    if (!ctx || !a) return AA_ERR_INVALID_ARG;
    aa_status st = check_feat(feat);
    if (st != AA_OK) return st;
    aa_ctx_impl* c = &ctx->impl;
    const int64_t n_cand = feat->row_idx ? feat->n_rows : feat->n;
    ShrinkParams sp;
    st = base_shrink_params(sp, n_cand, feat->n, feat->row_idx, feat->id_base, mix, seed, step, out_idx, capacity,
                            out_count, out_score, out_mask);
    if (st != AA_OK) return st;
    if (n_cand > c->max_rows || feat->d > c->max_d) return AA_ERR_WORKSPACE;
    if (a->kind == AA_ASSIST_MLP) {
        if (a->d != feat->d || a->hidden <= 0 || !a->W1_bf16 || !a->b1 || !a->w2 || !a->b2) return AA_ERR_INVALID_ARG;
        if (a->hidden > c->max_hidden) return AA_ERR_WORKSPACE;
        if (feat->kind != AA_FEAT_DENSE || feat->dtype != AA_BF16) return AA_ERR_UNSUPPORTED;
        if (n_cand == 0) return cuda_ok(cudaMemsetAsync(out_count, 0, sizeof(int32_t), c->stream));
        MlpFeat f = {feat->dense, feat->n, feat->d, feat->row_stride, a->W1_bf16, a->b1, a->w2, a->b2, a->hidden};
        return launch_score_shrink_mlp(c, f, sp);
    }
    if (a->kind != AA_ASSIST_LINEAR) return AA_ERR_INVALID_ARG;
    if (a->d != feat->d || !a->w || !a->b) return AA_ERR_INVALID_ARG;
    if (n_cand == 0) return cuda_ok(cudaMemsetAsync(out_count, 0, sizeof(int32_t), c->stream));
    if (feat->kind == AA_FEAT_DENSE) {
        DenseFeat f = {feat->dense, feat->dtype, feat->d, feat->row_stride, a->w, a->b};
        return launch_score_shrink_dense(c, f, sp);
    }
    CsrFeat f = {feat->indptr, feat->col, feat->val, feat->d, a->w, a->b, 0.0f};
    f.mean_nnz = (feat->nnz > 0 && feat->n > 0) ? (float)feat->nnz / (float)feat->n : 32.0f;
    return launch_score_shrink_csr(c, f, sp);
}

aa_status aa_shrink_compact(aa_ctx* ctx, const float* score, int64_t n, int64_t id_base, float mix, uint64_t seed,
                            uint64_t step, int32_t* out_idx, int64_t capacity, int32_t* out_count, uint8_t* out_mask) {
    if (!ctx || (n > 0 && !score)) return AA_ERR_INVALID_ARG;
    aa_ctx_impl* c = &ctx->impl;
    ShrinkParams sp;
    aa_status st = base_shrink_params(sp, n, n, nullptr, id_base, mix, seed, step, out_idx, capacity, out_count, nullptr,
                                      out_mask);
    if (st != AA_OK) return st;
    if (n > c->max_rows) return AA_ERR_WORKSPACE;
    if (n == 0) return cuda_ok(cudaMemsetAsync(out_count, 0, sizeof(int32_t), c->stream));
    return launch_shrink_from_scores(c, score, sp);
}

aa_status aa_threshold_compact(aa_ctx* ctx, const float* value, int64_t n, float threshold, int32_t* out_idx, int64_t capacity,
                               int32_t* out_count, uint8_t* out_mask) {
    if (!ctx || (n > 0 && !value) || threshold != threshold) return AA_ERR_INVALID_ARG;
    aa_ctx_impl* c = &ctx->impl;
    ShrinkParams sp;
    aa_status st = base_shrink_params(sp, n, n, nullptr, 0, 0.0f, 0, 0, out_idx, capacity, out_count, nullptr, out_mask);
    if (st != AA_OK) return st;
    sp.hard = 1;
    sp.hard_threshold = threshold;
    if (n > c->max_rows) return AA_ERR_WORKSPACE;
    if (n == 0) return cuda_ok(cudaMemsetAsync(out_count, 0, sizeof(int32_t), c->stream));
    return launch_shrink_from_scores(c, value, sp);
}

aa_status aa_batch_cut(aa_ctx* ctx, const int32_t* idx, const int32_t* count_dev, int64_t idx_capacity, int64_t n_cand,
                       int64_t batch_size, const int32_t* lengths, int64_t n_stored, int64_t token_budget, int32_t* out_m,
                       int32_t* out_consumed, int32_t* out_offsets, int64_t offsets_capacity) {
    if (!ctx || !out_m || !out_consumed || idx_capacity < 0 || n_cand < 0 || n_cand > 0x7FFFFFFFll || batch_size < 0)
        return AA_ERR_INVALID_ARG;
    if (idx_capacity > 0 && !idx) return AA_ERR_INVALID_ARG;
    if (lengths && (token_budget < 0 || n_stored < 0)) return AA_ERR_INVALID_ARG;
    if (out_offsets && (!lengths || offsets_capacity < 1)) return AA_ERR_INVALID_ARG;
    return launch_batch_cut(&ctx->impl, idx, count_dev, idx_capacity, n_cand, n_stored, batch_size, lengths, token_budget, out_m,
                            out_consumed, out_offsets, offsets_capacity);
}

aa_status aa_instance_loss(aa_ctx* ctx, const aa_logits* lg, const int32_t* labels, const int32_t* offsets, int64_t n_seg,
                           const int32_t* count_dev, float* out_loss) {
    if (!ctx || !lg || lg->rows < 0 || lg->cols <= 0 || lg->row_stride < lg->cols) return AA_ERR_INVALID_ARG;
    if (lg->dtype != AA_F32 && lg->dtype != AA_BF16) return AA_ERR_INVALID_ARG;
    if (lg->rows > 0 && (!lg->data || !labels)) return AA_ERR_INVALID_ARG;
    if ((uintptr_t)lg->data % (lg->dtype == AA_BF16 ? 2 : 4)) return AA_ERR_INVALID_ARG;
    if (lg->cols > 0x7FFFFFFFll) return AA_ERR_INVALID_ARG;
    if (offsets ? (n_seg < 0 || (n_seg > 0 && !out_loss)) : (lg->rows > 0 && !out_loss)) return AA_ERR_INVALID_ARG;
    aa_ctx_impl* c = &ctx->impl;
    if (offsets && lg->rows > c->max_rows) return AA_ERR_WORKSPACE;
    return launch_instance_loss(c, *lg, labels, offsets, n_seg, count_dev, out_loss);
}

aa_status aa_instance_loss_rows(aa_ctx* ctx, const aa_logits* lg, const int32_t* labels, const int32_t* row_idx, int64_t n_rows,
                                const int32_t* count_dev, float* out_loss) {
    if (!ctx || !lg || lg->rows < 0 || lg->cols <= 0 || lg->row_stride < lg->cols || n_rows < 0) return AA_ERR_INVALID_ARG;
    if (lg->dtype != AA_F32 && lg->dtype != AA_BF16) return AA_ERR_INVALID_ARG;
    if (n_rows > 0 && (!lg->data || !labels || !row_idx || !out_loss)) return AA_ERR_INVALID_ARG;
    if ((uintptr_t)lg->data % (lg->dtype == AA_BF16 ? 2 : 4)) return AA_ERR_INVALID_ARG;
    if (lg->cols > 0x7FFFFFFFll) return AA_ERR_INVALID_ARG;
    if (n_rows == 0) return AA_OK;
    return launch_instance_loss(&ctx->impl, *lg, labels, nullptr, 0, count_dev, out_loss, row_idx, n_rows);
}

aa_status aa_assistant_step(aa_ctx* ctx, const aa_feat* feat, const float* loss, const int32_t* count_dev, aa_assistant* a,
                            float lr, int32_t thresh_mode, float threshold) {
    if (!ctx || !a) return AA_ERR_INVALID_ARG;
    aa_status st = check_feat(feat);
    if (st != AA_OK) return st;
    if (thresh_mode != AA_THRESH_VALUE && thresh_mode != AA_THRESH_BATCH_MEAN) return AA_ERR_INVALID_ARG;
    aa_ctx_impl* c = &ctx->impl;
    const int64_t m_host = feat->row_idx ? feat->n_rows : feat->n;
    if (m_host > 0 && !loss) return AA_ERR_INVALID_ARG;
    if (a->kind == AA_ASSIST_MLP) {
        if (a->d != feat->d || a->hidden <= 0 || !a->W1 || !a->W1_bf16 || !a->b1 || !a->w2 || !a->b2) return AA_ERR_INVALID_ARG;
        if (feat->kind != AA_FEAT_DENSE || feat->dtype != AA_BF16) return AA_ERR_UNSUPPORTED;
        MlpFeat f = {feat->dense, feat->n, feat->d, feat->row_stride, a->W1_bf16, a->b1, a->w2, a->b2, a->hidden};
        return launch_assistant_step_mlp(c, f, a->W1, feat->row_idx, feat->n, m_host, count_dev, loss, lr, thresh_mode, threshold);
    }
    if (a->kind != AA_ASSIST_LINEAR) return AA_ERR_INVALID_ARG;
    if (a->d != feat->d || !a->w || !a->b) return AA_ERR_INVALID_ARG;
    if (feat->d > c->max_d) return AA_ERR_WORKSPACE;
    if (feat->kind == AA_FEAT_DENSE) {
        DenseFeat f = {feat->dense, feat->dtype, feat->d, feat->row_stride, a->w, a->b};
        return launch_assistant_step_dense(c, f, feat->row_idx, feat->n, m_host, count_dev, loss, a->w, a->b, lr,
                                           thresh_mode, threshold);
    }
    CsrFeat f = {feat->indptr, feat->col, feat->val, feat->d, a->w, a->b, 0.0f};
    f.mean_nnz = (feat->nnz > 0 && feat->n > 0) ? (float)feat->nnz / (float)feat->n : 32.0f;
    return launch_assistant_step_csr(c, f, feat->row_idx, feat->n, m_host, count_dev, loss, a->w, a->b, lr, thresh_mode,
                                     threshold);
}

aa_status aa_assistant_step_scored(aa_ctx* ctx, const aa_feat* feat, const float* loss, const int32_t* count_dev,
                                   const float* score, aa_assistant* a, float lr, int32_t thresh_mode, float threshold) {
    if (!ctx) return AA_ERR_INVALID_ARG;
    ctx->impl.step_score = score;
    const aa_status st = aa_assistant_step(ctx, feat, loss, count_dev, a, lr, thresh_mode, threshold);
    ctx->impl.step_score = nullptr;
    return st;
}

aa_status aa_assistant_step_adam(aa_ctx* ctx, const aa_feat* feat, const float* loss, const int32_t* count_dev, aa_assistant* a,
                                 aa_adam* state, float lr, int32_t thresh_mode, float threshold) {
    if (!ctx || !state || !state->m || !state->v || state->t < 0) return AA_ERR_INVALID_ARG;
    if (!(state->beta1 >= 0.0f && state->beta1 < 1.0f) || !(state->beta2 >= 0.0f && state->beta2 < 1.0f) || !(state->eps >= 0.0f))
        return AA_ERR_INVALID_ARG;
    const double t = (double)(state->t + 1);
    AdamArgs args;
    args.on = 1;
    args.beta1 = state->beta1;
    args.beta2 = state->beta2;
    args.eps = state->eps;
    args.corr1 = (float)(1.0 / (1.0 - pow((double)state->beta1, t)));
    args.corr2 = (float)(1.0 / (1.0 - pow((double)state->beta2, t)));
    args.m = state->m;
    args.v = state->v;
    ctx->impl.adam = args;
    const aa_status st = aa_assistant_step(ctx, feat, loss, count_dev, a, lr, thresh_mode, threshold);
    ctx->impl.adam.on = 0;
    if (st == AA_OK) state->t += 1;
    return st;
}

namespace {

struct HostStepLayout {
    size_t feat_off, logits_off, labels_off, idx_off, count_off, loss_off, score_off, total;
    size_t feat_bytes, logits_bytes;
};

aa_status host_step_layout(const aa_feat* feat, const aa_logits* lg, HostStepLayout& L) {
    if (!feat || !lg || feat->kind != AA_FEAT_DENSE || feat->n < 0 || feat->d <= 0) return AA_ERR_INVALID_ARG;
    if (feat->dtype != AA_F32 && feat->dtype != AA_BF16) return AA_ERR_INVALID_ARG;
    if (lg->dtype != AA_F32 && lg->dtype != AA_BF16) return AA_ERR_INVALID_ARG;
    if (feat->row_stride != feat->d || lg->row_stride != lg->cols || lg->rows < feat->n || lg->cols <= 0)
        return AA_ERR_INVALID_ARG;
    const size_t n = (size_t)feat->n;
    L.feat_bytes = n * (size_t)feat->d * (feat->dtype == AA_BF16 ? 2 : 4);
    L.logits_bytes = n * (size_t)lg->cols * (lg->dtype == AA_BF16 ? 2 : 4);
    size_t off = 0;
    L.feat_off = off;   off = align_up(off + L.feat_bytes, 256);
    L.logits_off = off; off = align_up(off + L.logits_bytes, 256);
    L.labels_off = off; off = align_up(off + n * sizeof(int32_t), 256);
    L.idx_off = off;    off = align_up(off + n * sizeof(int32_t), 256);
    L.count_off = off;  off = align_up(off + sizeof(int32_t), 256);
    L.loss_off = off;   off = align_up(off + n * sizeof(float), 256);
    L.score_off = off;  off = align_up(off + n * sizeof(float), 256);
    L.total = off;
    return AA_OK;
}

}  // namespace

aa_status aa_step_host_staging_bytes(const aa_feat* feat, const aa_logits* logits, size_t* bytes) {
    if (!bytes) return AA_ERR_INVALID_ARG;
    HostStepLayout L;
    aa_status st = host_step_layout(feat, logits, L);
    if (st != AA_OK) return st;
    *bytes = L.total;
    return AA_OK;
}

aa_status aa_step_host(aa_ctx* ctx, const aa_feat* feat, aa_assistant* a, float mix, uint64_t seed, uint64_t step,
                       const aa_logits* logits, const int32_t* labels, float lr, int32_t thresh_mode, float threshold,
                       int32_t* out_idx, int32_t* out_count, float* out_loss, void* staging, size_t staging_bytes) {
    if (!ctx || !a || !staging || (uintptr_t)staging % 256 || !out_count) return AA_ERR_INVALID_ARG;
    HostStepLayout L;
    aa_status st = host_step_layout(feat, logits, L);
    if (st != AA_OK) return st;
    if (feat->row_idx) return AA_ERR_UNSUPPORTED;
    if (staging_bytes < L.total) return AA_ERR_WORKSPACE;
    const int64_t n = feat->n;
    if (n > 0 && (!feat->dense || !logits->data || !labels || !out_idx || !out_loss)) return AA_ERR_INVALID_ARG;
    cudaStream_t s = ctx->impl.stream;
    char* base = static_cast<char*>(staging);
    int32_t* d_idx = reinterpret_cast<int32_t*>(base + L.idx_off);
    int32_t* d_count = reinterpret_cast<int32_t*>(base + L.count_off);
    float* d_loss = reinterpret_cast<float*>(base + L.loss_off);
    int32_t* d_labels = reinterpret_cast<int32_t*>(base + L.labels_off);
    if (n > 0) {
        if (cudaMemcpyAsync(base + L.feat_off, feat->dense, L.feat_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(base + L.logits_off, logits->data, L.logits_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(d_labels, labels, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, s) != cudaSuccess)
            return AA_ERR_CUDA;
    }
    aa_feat f = *feat;
    f.dense = base + L.feat_off;
    float* d_score = reinterpret_cast<float*>(base + L.score_off);
    st = aa_score_shrink(ctx, &f, a, mix, seed, step, d_idx, n, d_count, d_score, nullptr);
    if (st != AA_OK) return st;
    aa_logits lg = *logits;
    lg.data = base + L.logits_off;
    lg.rows = n;
    st = aa_instance_loss(ctx, &lg, d_labels, nullptr, 0, d_count, d_loss);
    if (st != AA_OK) return st;
    aa_feat fb = f;
    fb.row_idx = d_idx;
    fb.n_rows = n;
    // the parameters are still those of the screening above: the step takes its pre-activations
    st = aa_assistant_step_scored(ctx, &fb, d_loss, d_count, d_score, a, lr, thresh_mode, threshold);
    if (st != AA_OK) return st;
    // the count first, so that only the M live entries of the list and the losses cross the bus
    if (cudaMemcpyAsync(out_count, d_count, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return AA_ERR_CUDA;
    int64_t m = *out_count;
    if (m > n) m = n;
    if (m > 0) {
        if (cudaMemcpyAsync(out_idx, d_idx, (size_t)m * sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaMemcpyAsync(out_loss, d_loss, (size_t)m * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess)
            return AA_ERR_CUDA;
    }
    return AA_OK;
}

aa_status aa_conv_pool_features(aa_ctx* ctx, const aa_feat* images, const aa_conv* conv, float* out_phi, int64_t phi_stride) {
    if (!ctx || !conv) return AA_ERR_INVALID_ARG;
    aa_status st = check_feat(images);
    if (st != AA_OK) return st;
    if (images->kind != AA_FEAT_DENSE) return AA_ERR_INVALID_ARG;
    if (images->row_idx) return AA_ERR_UNSUPPORTED;
    if (conv->c_in <= 0 || conv->height <= 0 || conv->width <= 0 || conv->c_out <= 0 || conv->pool <= 0 || !conv->weight)
        return AA_ERR_INVALID_ARG;
    if (conv->ksize <= 0 || conv->ksize % 2 == 0 || conv->height % conv->pool || conv->width % conv->pool) return AA_ERR_INVALID_ARG;
    if ((int64_t)conv->c_in * conv->height * conv->width != images->d) return AA_ERR_INVALID_ARG;
    const int64_t feats = (int64_t)conv->c_out * (conv->height / conv->pool) * (conv->width / conv->pool);
    if (phi_stride < feats || (images->n > 0 && !out_phi)) return AA_ERR_INVALID_ARG;
    if (images->n == 0) return AA_OK;
    return launch_conv_pool_features(&ctx->impl, images->dense, images->dtype, images->n, images->row_stride, *conv, out_phi, phi_stride);
}

aa_status aa_device_status(aa_ctx* ctx, int32_t* latched) {
    if (!ctx || !latched) return AA_ERR_INVALID_ARG;
    aa_ctx_impl* c = &ctx->impl;
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, &c->ctl->status, sizeof v, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
        return AA_ERR_CUDA;
    *latched = v;
    if (v != 0) {
        // a scan that gave up may have left the ticket state half-used: re-arm everything
        const unsigned int zeros[4] = {0, 0, 0, 0};
        if (cudaMemcpyAsync(c->ctl, zeros, 2 * sizeof(unsigned int), cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
            cudaMemsetAsync(&c->ctl->status, 0, sizeof(int), c->stream) != cudaSuccess ||
            cudaMemsetAsync(&c->ctl->sums_in, 0, 3 * sizeof(unsigned int), c->stream) != cudaSuccess ||   // sums_in, grad_done, applied
            cudaStreamSynchronize(c->stream) != cudaSuccess)
            return AA_ERR_CUDA;
    }
    return AA_OK;
}

float aa_sk_threshold(float G, int64_t k) { return k >= 1 ? G / (float)k : G; }

int64_t aa_launch_count(const aa_ctx* ctx) { return ctx ? ctx->impl.launches : -1; }

}  // extern "C"
