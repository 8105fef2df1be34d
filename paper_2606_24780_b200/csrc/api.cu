// C ABI of the bt library: model object over a caller-owned workspace, the fixed launch
// schedule of the training step, and the per-operation entry points.
//
// There is no tensor class, no autograd and no allocator: the backward pass is hand-derived
// and every buffer has a fixed place in the workspace.  All kernels of one step are enqueued
// on one stream in a fixed order; the host never blocks unless the caller asks for the loss.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/bt.h"
#include "common.cuh"

using namespace bt;

namespace {

thread_local std::string g_last_error;

bt_status fail(bt_status st, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    g_last_error = buf;
    return st;
}

}  // namespace

extern "C" __attribute__((visibility("hidden"))) int bt_internal_fail_int(int status, const char* message) {
    g_last_error = message ? message : "";
    return status;
}

namespace {

#define BT_CUDA(call)                                                                           \
    do {                                                                                        \
        cudaError_t e__ = (call);                                                               \
        if (e__ != cudaSuccess) return fail(BT_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
#define BT_PTR(p)                                                                               \
    do {                                                                                        \
        if ((p) == nullptr) return fail(BT_ERR_INVALID_ARG, "%s is NULL", #p);                  \
        if (!aligned16(p)) return fail(BT_ERR_INVALID_ARG, "%s is not 16-byte aligned", #p);    \
    } while (0)
#define BT_OPT_PTR(p)                                                                           \
    do {                                                                                        \
        if ((p) != nullptr && !aligned16(p))                                                    \
            return fail(BT_ERR_INVALID_ARG, "%s is not 16-byte aligned", #p);                   \
    } while (0)

struct Tensor {
    std::string name;
    int64_t numel;
    int decay;
    int64_t off;   // float offset inside each arena
    int kind;      // 0 normal(std), 1 normal(residual std), 2 ones, 3 zeros
};

// One timed launch group of the step: category, algorithmic work, the two events around it.
struct ProfRec {
    int cat;
    double flops, bytes;
    size_t ev;  // index of the start event; the stop event follows
};
enum ProfCat {
    kCatSplit = 0, kCatEmbedFwd, kCatLnFwd, kCatGemmNT, kCatAttnFwd, kCatGeluFwd, kCatXent, kCatGemmNN, kCatGemmTN,
    kCatLnBwd, kCatGeluBwd, kCatAttnBwd, kCatColsum, kCatEmbedBwd, kCatGradNorm, kCatAdamW, kNumCats
};
const char* const kCatNames[kNumCats] = {
    "split_weights", "embedding_fwd", "layernorm_fwd", "gemm_fwd", "attention_fwd", "gelu_fwd", "softmax_xent",
    "gemm_dx", "gemm_dw", "layernorm_bwd", "gelu_bwd", "attention_bwd", "colsum", "embedding_bwd", "grad_norm",
    "adamw"};

struct LayerAct {
    float *x, *mean1, *rstd1, *a_s, *qkv, *qkv_s, *o_s, *lse, *x1, *mean2, *rstd2, *m_s, *h, *g_s;
};

// Bump allocator over the workspace; with base == nullptr it only measures.
struct Bump {
    uint8_t* base;
    size_t off = 0;
    template <typename T>
    T* take(size_t count) {
        off = (off + 255) & ~(size_t)255;
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += count * sizeof(T);
        return p;
    }
};

}  // namespace

// Gradient buckets of the data-parallel step (Algorithm 1).  The gradients of one model lie in one
// flat arena in registry order, and the backward pass finishes them in (almost exactly) the reverse
// of that order, so a bucket needs no memory of its own: it is a contiguous range of the arena,
// bucket 0 at the arena's end (first ready), the last bucket at its start (the tied embedding, ready
// last).  Ranges are cut at tensor boundaries while a tensor fits under the cap; a larger tensor is
// cut into equal ranges under the cap (all of them ready together).  `pending` counts the tensors that overlap
// a bucket and are not ready yet; buckets are released strictly in order (the launch gate).
struct bt_ddp_plan {
    struct Bucket { int64_t offset, count; int n_tensors, pending; };
    std::vector<Bucket> buckets;
    std::vector<int64_t> t_off, t_len;          // arena range of every tensor (padded length)
    std::vector<int> t_first, t_last;           // buckets a tensor overlaps
    std::vector<uint8_t> t_ready;
    int next_bucket = 0;
    int64_t P = 0;
};

struct bt_model {
    bt_config cfg;
    cudaStream_t stream;
    int L, C, H, T, V, Vp, F, maxB;
    std::vector<Tensor> tensors;
    int64_t P;  // padded parameter count (multiple of 1024)
    size_t part_bytes[7];   // workspace sections, see bt_workspace_part_bytes
    float *params, *grads, *mom1, *mom2, *wsplit, *wsplit_t, *gacc, *loss_acc;
    MatDesc* mat_descs;   // device table of the weight matrices (for the split in both orientations)
    int n_mats, n_mat_tiles;
    uint8_t* decay_flags;
    std::vector<LayerAct> act;
    float *xL, *meanf, *rstdf, *xf_s, *logits, *dlogits_s, *losses, *loss, *norm_out;
    float *dres, *dres_s, *dtmp, *do_s, *dqkv_s, *dh_s, *dg, *dh_groups, *dvec, *attn_rg;
    float *partials, *ln_scratch, *colsum_scratch;
    void* norm_scratch;
    size_t partial_floats;
    int* err_word;
    int32_t *tok_stage, *tgt_stage;
    uint8_t* emb_table;   // [Vp][chunks] byte table of the embedding backward
    bool debug_sync;      // BT_FLAG_DEBUG or BT_DEBUG=1: every step call synchronises and reports device errors
    int64_t step;
    int curB;
    const int32_t* cur_tok;
    bool have_forward;
    long long launches_at_create;
    // optional per-kernel timing (CUDA events around every launch of the step)
    // data-parallel gradient exchange (null: single replica)
    bt_ddp_plan* ddp;
    bt_allreduce_fn ddp_fn;
    void* ddp_user;
    cudaStream_t ddp_stream;
    std::vector<cudaEvent_t> ddp_ready_ev;   // one per bucket, recorded on the compute stream
    cudaEvent_t ddp_done_ev;                 // recorded on the communication stream after the last bucket
    bool ddp_sync;                           // this backward exchanges gradients (false on all but the last micro-step)
    float ddp_acc_weight;                    // > 0: the last micro-step's accumulation is folded in per bucket
    bool prof_on;
    std::vector<ProfRec> prof_recs;
    std::vector<cudaEvent_t> prof_events;
    size_t prof_used;
};

bool bt::pdl_enabled() {
    static const bool on = []() {
        const char* v = getenv("BT_PDL");
        return !(v && v[0] == '0');
    }();
    return on;
}

namespace {

void build_registry(const bt_config& c, std::vector<Tensor>& out, int64_t& P) {
    const int64_t C = c.d_model, F = 4 * (int64_t)c.d_model;
    int64_t off = 0;
    auto add = [&](const std::string& n, int64_t numel, int decay, int kind) {
        out.push_back(Tensor{n, numel, decay, off, kind});
        off += (numel + 1023) / 1024 * 1024;
    };
    add("wte", (int64_t)c.padded_vocab_size * C, 1, 0);
    add("wpe", (int64_t)c.seq_len * C, 1, 0);
    for (int l = 0; l < c.n_layers; ++l) {
        std::string p = "h" + std::to_string(l) + ".";
        add(p + "ln1.g", C, 0, 2);
        add(p + "ln1.b", C, 0, 3);
        add(p + "attn.qkv.w", 3 * C * C, 1, 0);
        add(p + "attn.qkv.b", 3 * C, 0, 3);
        add(p + "attn.proj.w", C * C, 1, 1);
        add(p + "attn.proj.b", C, 0, 3);
        add(p + "ln2.g", C, 0, 2);
        add(p + "ln2.b", C, 0, 3);
        add(p + "mlp.fc.w", F * C, 1, 0);
        add(p + "mlp.fc.b", F, 0, 3);
        add(p + "mlp.proj.w", C * F, 1, 1);
        add(p + "mlp.proj.b", C, 0, 3);
    }
    add("lnf.g", C, 0, 2);
    add("lnf.b", C, 0, 3);
    P = off;
}

bt_status validate(const bt_config* c) {
    if (!c) return fail(BT_ERR_INVALID_ARG, "config is NULL");
    if (c->n_layers < 1 || c->d_model < 1 || c->n_heads < 1 || c->seq_len < 1 || c->vocab_size < 1 ||
        c->max_batch < 1)
        return fail(BT_ERR_INVALID_ARG, "config: sizes must be positive");
    if (c->d_model % c->n_heads) return fail(BT_ERR_INVALID_ARG, "config: d_model %% n_heads != 0");
    int d = c->d_model / c->n_heads;
    if (d != 16 && d != 32 && d != 64 && d != 128)
        return fail(BT_ERR_UNSUPPORTED, "config: head_dim %d not in {16,32,64,128}", d);
    if (c->d_model % 32) return fail(BT_ERR_INVALID_ARG, "config: d_model %% 32 != 0");
    if (c->d_model > 4096) return fail(BT_ERR_UNSUPPORTED, "config: d_model > 4096 not compiled");
    if (1 + 4 * (int64_t)c->n_layers > kMaxSplitMats) return fail(BT_ERR_UNSUPPORTED, "config: more than 63 layers");
    if (c->padded_vocab_size < c->vocab_size) return fail(BT_ERR_INVALID_ARG, "config: padded_vocab < vocab");
    if (c->padded_vocab_size % 32) return fail(BT_ERR_INVALID_ARG, "config: padded_vocab %% 32 != 0");
    if ((c->flags & BT_FLAG_LOGITS_IN_PLACE) && c->padded_vocab_size > softmax_xent_max_in_place_columns())
        return fail(BT_ERR_UNSUPPORTED, "config: BT_FLAG_LOGITS_IN_PLACE needs padded_vocab <= %d", softmax_xent_max_in_place_columns());
    if ((int64_t)c->max_batch * c->seq_len > (1 << 24))
        return fail(BT_ERR_UNSUPPORTED, "config: more than 2^24 tokens per step");
    return BT_OK;
}

// Carves the workspace.  Called with base == nullptr to measure.
size_t layout(bt_model* m, uint8_t* base) {
    Bump b{base};
    const int64_t C = m->C, F = m->F, N = (int64_t)m->maxB * m->T, Vp = m->Vp, P = m->P;
    // the raw (single-plane) qkv exists only for the attention kernels that read it: the warp-MMA
    // kernels of head_dim 16 / 32 and the reference kernels behind the test flags
    const int hd = (int)(C / m->H);
    const bool raw_qkv = (m->cfg.flags & (BT_FLAG_ATTN_SIMT | BT_FLAG_GEMM_SIMT)) != 0 || (hd != 64 && hd != 128);
    size_t mark = 0;
    auto section = [&](int part) { m->part_bytes[part] = b.off - mark; mark = b.off; };
    m->params = b.take<float>(P);
    m->grads = b.take<float>(P);
    m->mom1 = b.take<float>(P);
    m->mom2 = b.take<float>(P);
    section(0);                      // parameters, gradients, both moments
    m->wsplit = b.take<float>(2 * P);
    m->wsplit_t = b.take<float>(2 * P);
    section(1);                      // TF32 hi/lo planes of the weights, both orientations
    m->gacc = b.take<float>(P);      // gradient accumulator of the micro-step loop
    m->loss_acc = b.take<float>(4);
    m->mat_descs = b.take<MatDesc>(kMaxSplitMats);
    m->decay_flags = b.take<uint8_t>(P / 1024);
    section(2);                      // gradient accumulator, tables
    m->act.resize(m->L);
    // BT_FLAG_RECOMPUTE_LN: the LayerNorm outputs (hi/lo planes) are not kept per layer; one buffer
    // serves every layer and the backward pass re-runs the LayerNorm forward from the saved input
    // and statistics where a weight-gradient product needs them
    const bool recompute_ln = (m->cfg.flags & BT_FLAG_RECOMPUTE_LN) != 0;
    float* ln_shared = recompute_ln ? b.take<float>(2 * N * C) : nullptr;
    // BT_FLAG_RECOMPUTE_GELU: likewise for the GELU output planes (the largest saved activation); the
    // backward pass forms them again from the pre-activation h, which is kept anyway
    const bool recompute_gelu = (m->cfg.flags & BT_FLAG_RECOMPUTE_GELU) != 0;
    float* gelu_shared = recompute_gelu ? b.take<float>(2 * N * F) : nullptr;
    for (int l = 0; l < m->L; ++l) {
        LayerAct& a = m->act[l];
        a.x = b.take<float>(N * C);
        a.mean1 = b.take<float>(N);
        a.rstd1 = b.take<float>(N);
        a.a_s = recompute_ln ? ln_shared : b.take<float>(2 * N * C);
        a.qkv = raw_qkv ? b.take<float>(N * 3 * C) : nullptr;
        a.qkv_s = b.take<float>(2 * N * 3 * C);
        a.o_s = b.take<float>(2 * N * C);
        a.lse = b.take<float>((int64_t)m->maxB * m->H * m->T);
        a.x1 = b.take<float>(N * C);
        a.mean2 = b.take<float>(N);
        a.rstd2 = b.take<float>(N);
        a.m_s = recompute_ln ? ln_shared : b.take<float>(2 * N * C);
        a.h = b.take<float>(N * F);
        a.g_s = recompute_gelu ? gelu_shared : b.take<float>(2 * N * F);
    }
    m->xL = b.take<float>(N * C);
    m->meanf = b.take<float>(N);
    m->rstdf = b.take<float>(N);
    m->xf_s = b.take<float>(2 * N * C);
    section(3);                      // activations kept for the backward pass
    // BT_FLAG_LOGITS_IN_PLACE: the hi plane of the logit gradient overwrites the logits (the loss kernel
    // holds a whole row in registers before it writes anything)
    m->dlogits_s = b.take<float>(2 * N * Vp);
    m->logits = (m->cfg.flags & BT_FLAG_LOGITS_IN_PLACE) ? m->dlogits_s : b.take<float>(N * Vp);
    m->losses = b.take<float>(N);
    m->loss = b.take<float>(4);
    m->norm_out = b.take<float>(4);
    section(4);                      // logits, their gradient planes, per-row losses
    m->dres = b.take<float>(N * C);
    m->dres_s = b.take<float>(2 * N * C);
    m->dtmp = b.take<float>(N * C);
    m->do_s = b.take<float>(2 * N * C);
    m->dqkv_s = b.take<float>(2 * N * 3 * C);
    m->dh_s = b.take<float>(2 * N * F);
    // d g (the GELU output's gradient) exists as an array only with the FMA reference GEMM; the
    // tensor-core GEMM applies GELU' in its epilogue and leaves column sums per 32-row group instead
    const bool simt_gemm = (m->cfg.flags & BT_FLAG_GEMM_SIMT) != 0;
    m->dg = simt_gemm ? b.take<float>(N * F) : nullptr;
    m->dh_groups = simt_gemm ? nullptr : b.take<float>(((N + 31) / 32) * F);
    m->dvec = b.take<float>((int64_t)m->maxB * m->H * m->T);
    m->attn_rg = b.take<float>(attention_bwd_rowgroups(m->maxB, m->T) * 3 * m->C);
    section(5);                      // backward temporaries (reused by every layer)
    m->partial_floats = gemm_tc_partial_floats_bound();
    // the LM head's input gradient sums over the padded vocabulary: room for the K ranges that keep its
    // accumulation chains within the planner's cap at any token count
    // (and for its weight gradient, which sums over the tokens)
    if (!simt_gemm) {
        const size_t need_dx = gemm_tc_partial_floats_for_chain_cap(N, C, m->Vp);
        const size_t need_dw = gemm_tc_partial_floats_for_chain_cap(m->Vp, C, N);
        if (need_dx > m->partial_floats) m->partial_floats = need_dx;
        if (need_dw > m->partial_floats) m->partial_floats = need_dw;
    }
    m->partials = b.take<float>(m->partial_floats);
    m->ln_scratch = b.take<float>(layernorm_bwd_scratch_floats(N, (int)C));
    size_t cs = colsum_scratch_floats(N, (int)F);
    if (colsum_scratch_floats(N, (int)C) > cs) cs = colsum_scratch_floats(N, (int)C);
    if (colsum_scratch_floats(N, 3 * (int)C) > cs) cs = colsum_scratch_floats(N, 3 * (int)C);
    const size_t cs_rg = colsum_scratch_floats(attention_bwd_rowgroups(m->maxB, m->T), 3 * (int)C);
    if (cs_rg > cs) cs = cs_rg;
    m->colsum_scratch = b.take<float>(cs);
    m->norm_scratch = b.take<uint8_t>(grad_norm_scratch_bytes(P));
    m->err_word = b.take<int>(4);
    m->tok_stage = b.take<int32_t>(N);
    m->tgt_stage = b.take<int32_t>(N);
    m->emb_table = b.take<uint8_t>(embedding_bwd_scratch_bytes(N, 0, (int)Vp));
    b.off = (b.off + 255) & ~(size_t)255;
    section(6);                      // split-K partial sums, reduction scratch, id staging, embedding table
    return b.off;
}

void fill_dims(bt_model* m, const bt_config* cfg) {
    m->cfg = *cfg;
    m->L = cfg->n_layers; m->C = cfg->d_model; m->H = cfg->n_heads; m->T = cfg->seq_len;
    m->V = cfg->vocab_size; m->Vp = cfg->padded_vocab_size; m->F = 4 * cfg->d_model; m->maxB = cfg->max_batch;
    m->tensors.clear();
    build_registry(*cfg, m->tensors, m->P);
}

const Tensor* find_tensor(const bt_model* m, const char* name) {
    for (const Tensor& t : m->tensors)
        if (t.name == name) return &t;
    return nullptr;
}
inline Tensor& layer_tensor(bt_model* m, int l, int k) { return m->tensors[2 + 12 * l + k]; }
enum { LN1G = 0, LN1B, QKVW, QKVB, PROJW, PROJB, LN2G, LN2B, FCW, FCB, PRW, PRB };

inline SplitMat weight_mat(bt_model* m, const Tensor& t, int64_t rows, int64_t cols) {
    return SplitMat{m->wsplit + t.off, m->P, rows, cols, cols};
}
// The transposed copy of a [rows, cols] weight: [cols, rows] row-major.
inline SplitMat weight_mat_t(bt_model* m, const Tensor& t, int64_t rows, int64_t cols) {
    return SplitMat{m->wsplit_t + t.off, m->P, cols, rows, rows};
}
inline SplitMat act_mat(const float* hi, int64_t rows, int64_t cols, int64_t plane_rows) {
    return SplitMat{hi, plane_rows * cols, rows, cols, cols};
}

void prof_begin(bt_model* m, int cat, double flops, double bytes) {
    if (!m->prof_on) return;
    if (m->prof_used + 2 > m->prof_events.size()) {
        for (int i = 0; i < 2; ++i) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { m->prof_on = false; return; }
            m->prof_events.push_back(e);
        }
    }
    m->prof_recs.push_back(ProfRec{cat, flops, bytes, m->prof_used});
    cudaEventRecord(m->prof_events[m->prof_used], m->stream);
    m->prof_used += 2;
}
void prof_end(bt_model* m) {
    if (!m->prof_on) return;
    cudaEventRecord(m->prof_events[m->prof_recs.back().ev + 1], m->stream);
}
// One launch group of the step: timed when profiling is on, error-checked always.
#define BT_STEP(cat, flops, bytes, call)                                                        \
    do {                                                                                        \
        prof_begin(m, cat, (double)(flops), (double)(bytes));                                   \
        cudaError_t e__ = (call);                                                               \
        prof_end(m);                                                                            \
        if (e__ != cudaSuccess) return fail(BT_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

inline double gemm_flops(int64_t M, int64_t N, int64_t K) { return 2.0 * (double)M * (double)N * (double)K; }
inline double gemm_bytes(int64_t M, int64_t N, int64_t K) {
    return 8.0 * ((double)M * K + (double)N * K) + 4.0 * (double)M * N;  // hi+lo operands, FP32 output
}
// Causal attention forward: QK^T and PV over the lower triangle including the diagonal.
inline double attn_fwd_flops(int64_t B, int64_t H, int64_t T, int64_t d) {
    return 4.0 * (double)B * H * d * ((double)T * (T + 1) / 2.0);
}

// The forward pass keeps GELU'(h) in the place of h = m Wfc^T + bfc unless h is needed again (GELU
// recomputed in the backward pass) or the FMA reference GEMM, which has no fused epilogues, runs.
inline bool h_holds_gelu_grad(const bt_model* m) {
    return !(m->cfg.flags & (BT_FLAG_GEMM_SIMT | BT_FLAG_RECOMPUTE_GELU));
}

// D = op(A) op(B) (+bias)(+residual) through the tensor-core kernel or the FMA reference.
cudaError_t gemm_raw(bt_model* m, int layout, int64_t M, int64_t N, int64_t K, SplitMat A, SplitMat B, float* D,
                 const float* bias, const float* residual, float* d_split = nullptr, int act = 0,
                 float* col_partial = nullptr) {
    if (m->cfg.flags & BT_FLAG_GEMM_SIMT) {
        // the FMA reference writes the raw output; the planes are made by a separate pass
        cudaError_t e = launch_gemm_simt(layout, M, N, K, A, B, D, N, bias, residual, m->stream);
        if (e == cudaSuccess && d_split) {
            if (act) e = launch_gelu_fwd(D, M * N, act == 2, nullptr, d_split, d_split + M * N, m->stream);
            else e = launch_split(D, d_split, d_split + M * N, M * N, m->stream);
        }
        return e;
    }
    return launch_gemm_tc(layout, M, N, K, A, B, D, N, bias, residual, m->partials, m->partial_floats, m->err_word,
                          m->stream, d_split, M * N, -1, act, col_partial);
}

// Timing category by role: the forward products (Y = X W^T, run as NN on the transposed weight
// copy), the input gradients (NN on the weight) and the weight gradients (TN).
#define BT_GEMM_CAT(fwd, layout) ((fwd) ? kCatGemmNT : (layout) == kTN ? kCatGemmTN : kCatGemmNN)
#define BT_GEMM(layout, M, N, K, A, B, D, bias, res)                                                        \
    BT_STEP(BT_GEMM_CAT(gemm_is_fwd, layout), gemm_flops(M, N, K), gemm_bytes(M, N, K),                         \
            gemm_raw(m, layout, M, N, K, A, B, D, bias, res))
// same, the output also written as TF32 hi/lo planes at DS
#define BT_GEMM_SPLIT_OUT(layout, M, N, K, A, B, D, DS, bias, res)                                           \
    BT_STEP(BT_GEMM_CAT(gemm_is_fwd, layout), gemm_flops(M, N, K), gemm_bytes(M, N, K) + 8.0 * (M) * (N),       \
            gemm_raw(m, layout, M, N, K, A, B, D, bias, res, DS))

// The device error words: [0] code of the first bounded wait that ran out, [1] position + 1 of a
// token id outside [0, vocab_size), [2] row + 1 of a target id outside it.  Reading them
// synchronises the stream; words that were set are reported once and cleared, so that the model
// stays usable after the caller has dealt with the error.
bt_status check_device_error(bt_model* m) {
    int err[4] = {0, 0, 0, 0};
    BT_CUDA(cudaMemcpyAsync(err, m->err_word, sizeof(err), cudaMemcpyDeviceToHost, m->stream));
    BT_CUDA(cudaStreamSynchronize(m->stream));
    if (err[0] == 0 && err[1] == 0 && err[2] == 0) return BT_OK;
    BT_CUDA(cudaMemsetAsync(m->err_word, 0, sizeof(err), m->stream));
    if (err[0] != 0) return fail(BT_ERR_DEVICE_TIMEOUT, "a bounded device-side wait ran out (code %d)", err[0]);
    if (err[1] != 0)
        return fail(BT_ERR_INVALID_ARG, "token id outside [0, %d) at position %d (treated as id 0)", m->V, err[1] - 1);
    return fail(BT_ERR_INVALID_ARG, "target id outside [0, %d) at position %d (treated as id 0)", m->V, err[2] - 1);
}

// Position of the first id outside [0, vocab) in a host array, or -1.
int64_t first_bad_id(const int32_t* ids, int64_t n, int32_t vocab) {
    for (int64_t i = 0; i < n; ++i)
        if ((uint32_t)ids[i] >= (uint32_t)vocab) return i;
    return -1;
}

bool debug_env() {
    static const bool on = []() {
        const char* v = getenv("BT_DEBUG");
        return v && v[0] != '\0' && v[0] != '0';
    }();
    return on;
}

// ------------------------------------------------------------------ data-parallel buckets
bt_status build_ddp_plan(const bt_config* cfg, int64_t cap_bytes, bt_ddp_plan** out) {
    if (!out) return fail(BT_ERR_INVALID_ARG, "ddp plan: out is NULL");
    *out = nullptr;
    bt_status st = validate(cfg);
    if (st != BT_OK) return st;
    if (cap_bytes < 4096) return fail(BT_ERR_INVALID_ARG, "ddp plan: bucket cap below 4096 bytes");
    std::vector<Tensor> reg;
    int64_t P = 0;
    build_registry(*cfg, reg, P);
    bt_ddp_plan* plan = new bt_ddp_plan();
    plan->P = P;
    const int n = (int)reg.size();
    plan->t_off.resize(n); plan->t_len.resize(n); plan->t_first.assign(n, -1); plan->t_last.assign(n, -1);
    plan->t_ready.assign(n, 0);
    for (int i = 0; i < n; ++i) {
        plan->t_off[i] = reg[i].off;
        plan->t_len[i] = (i + 1 < n ? reg[i + 1].off : P) - reg[i].off;
    }
    const int64_t cap = cap_bytes / 4 / 1024 * 1024;          // floats, a multiple of the tensor alignment
    // walk the registry backwards = gradient-ready order; `lo` is the start of the open bucket
    int64_t hi = P;          // end of the open bucket
    int64_t lo = P;
    int open_tensors = 0;
    auto close = [&]() {
        if (hi > lo) plan->buckets.push_back(bt_ddp_plan::Bucket{lo, hi - lo, open_tensors, open_tensors});
        hi = lo;
        open_tensors = 0;
    };
    for (int i = n - 1; i >= 0; --i) {
        const int64_t len = plan->t_len[i];
        if (len > cap) {                                      // larger than a bucket: equal ranges of its own, each under the cap
            close();
            plan->t_first[i] = (int)plan->buckets.size();
            int64_t end = plan->t_off[i] + len;
            const int64_t pieces = (len + cap - 1) / cap;
            const int64_t piece = ((len + pieces - 1) / pieces + 1023) / 1024 * 1024;   // equal ranges, each under the cap
            while (end > plan->t_off[i]) {
                const int64_t start = std::max(plan->t_off[i], end - piece);
                plan->buckets.push_back(bt_ddp_plan::Bucket{start, end - start, 1, 1});
                end = start;
            }
            plan->t_last[i] = (int)plan->buckets.size() - 1;
            hi = lo = plan->t_off[i];
            continue;
        }
        if (open_tensors > 0 && (hi - lo) + len > cap) close();
        lo = plan->t_off[i];
        ++open_tensors;
        plan->t_first[i] = plan->t_last[i] = (int)plan->buckets.size();   // index the open bucket will get
    }
    close();
    *out = plan;
    return BT_OK;
}

// The hook of Algorithm 1 on the host side of one model: marks a tensor ready and launches the
// exchange of every bucket the gate releases.
bt_status ddp_launch_bucket(bt_model* m, int b) {
    const bt_ddp_plan::Bucket& bk = m->ddp->buckets[(size_t)b];
    float* g = m->grads + bk.offset;
    if (m->ddp_acc_weight > 0.f)     // last micro-step: g = acc + w g for this range (the loss is handled by the caller)
        BT_CUDA(launch_grad_accumulate(m->gacc + bk.offset, g, bk.count, m->ddp_acc_weight, 2, nullptr, nullptr, m->stream));
    BT_CUDA(cudaEventRecord(m->ddp_ready_ev[(size_t)b], m->stream));
    BT_CUDA(cudaStreamWaitEvent(m->ddp_stream, m->ddp_ready_ev[(size_t)b], 0));
    if (m->ddp_fn(m->ddp_user, g, bk.count, b, (void*)m->ddp_stream) != 0)
        return fail(BT_ERR_CUDA, "ddp: the all-reduce callback failed on bucket %d", b);
    if (b + 1 == (int)m->ddp->buckets.size()) {   // the optimizer step must see every averaged bucket
        BT_CUDA(cudaEventRecord(m->ddp_done_ev, m->ddp_stream));
        BT_CUDA(cudaStreamWaitEvent(m->stream, m->ddp_done_ev, 0));
    }
    return BT_OK;
}
bt_status ddp_ready(bt_model* m, std::initializer_list<int> tensors) {
    if (!m->ddp || !m->ddp_sync) return BT_OK;
    std::vector<int32_t> launch(m->ddp->buckets.size());
    for (int t : tensors) {
        const int32_t n = bt_ddp_plan_mark_ready(m->ddp, t, launch.data());
        if (n < 0) return fail(BT_ERR_INVALID_ARG, "ddp: tensor %d marked ready twice", t);
        for (int32_t i = 0; i < n; ++i) {
            bt_status st = ddp_launch_bucket(m, launch[(size_t)i]);
            if (st != BT_OK) return st;
        }
    }
    return BT_OK;
}
#define BT_DDP_READY(...)                                  \
    do {                                                   \
        bt_status st__ = ddp_ready(m, {__VA_ARGS__});      \
        if (st__ != BT_OK) return st__;                    \
    } while (0)

}  // namespace

// =============================================================================== data-parallel plan (host only)

extern "C" bt_status bt_ddp_plan_create(const bt_config* cfg, int64_t bucket_cap_bytes, bt_ddp_plan** out) {
    return build_ddp_plan(cfg, bucket_cap_bytes, out);
}
extern "C" void bt_ddp_plan_destroy(bt_ddp_plan* plan) { delete plan; }
extern "C" int32_t bt_ddp_plan_num_buckets(const bt_ddp_plan* plan) { return plan ? (int32_t)plan->buckets.size() : 0; }
extern "C" bt_status bt_ddp_plan_bucket(const bt_ddp_plan* plan, int32_t b, int64_t* offset, int64_t* count,
                                        int32_t* n_tensors) {
    if (!plan) return fail(BT_ERR_INVALID_ARG, "ddp plan is NULL");
    if (b < 0 || b >= (int32_t)plan->buckets.size()) return fail(BT_ERR_NOT_FOUND, "bucket %d out of range", b);
    if (offset) *offset = plan->buckets[(size_t)b].offset;
    if (count) *count = plan->buckets[(size_t)b].count;
    if (n_tensors) *n_tensors = plan->buckets[(size_t)b].n_tensors;
    return BT_OK;
}
extern "C" bt_status bt_ddp_plan_tensor(const bt_ddp_plan* plan, int32_t tensor, int64_t* offset, int64_t* padded_len) {
    if (!plan) return fail(BT_ERR_INVALID_ARG, "ddp plan is NULL");
    if (tensor < 0 || tensor >= (int32_t)plan->t_off.size()) return fail(BT_ERR_NOT_FOUND, "tensor %d out of range", tensor);
    if (offset) *offset = plan->t_off[(size_t)tensor];
    if (padded_len) *padded_len = plan->t_len[(size_t)tensor];
    return BT_OK;
}
extern "C" void bt_ddp_plan_reset(bt_ddp_plan* plan) {
    if (!plan) return;
    for (auto& b : plan->buckets) b.pending = b.n_tensors;
    std::fill(plan->t_ready.begin(), plan->t_ready.end(), (uint8_t)0);
    plan->next_bucket = 0;
}
extern "C" int32_t bt_ddp_plan_mark_ready(bt_ddp_plan* plan, int32_t tensor, int32_t* launch) {
    if (!plan || !launch || tensor < 0 || tensor >= (int32_t)plan->t_off.size()) return -1;
    if (plan->t_ready[(size_t)tensor]) return -1;
    plan->t_ready[(size_t)tensor] = 1;
    for (int b = plan->t_first[(size_t)tensor]; b <= plan->t_last[(size_t)tensor]; ++b) plan->buckets[(size_t)b].pending -= 1;
    int32_t n = 0;
    while (plan->next_bucket < (int)plan->buckets.size() && plan->buckets[(size_t)plan->next_bucket].pending == 0)
        launch[n++] = plan->next_bucket++;      // the in-order launch gate
    return n;
}

// =============================================================================== model lifetime

extern "C" size_t bt_workspace_bytes(const bt_config* cfg) {
    if (validate(cfg) != BT_OK) return 0;
    bt_model tmp{};
    fill_dims(&tmp, cfg);
    return layout(&tmp, nullptr);
}

extern "C" size_t bt_workspace_part_bytes(const bt_config* cfg, int32_t part) {
    if (part < 0 || part > 6 || validate(cfg) != BT_OK) return 0;
    bt_model tmp{};
    fill_dims(&tmp, cfg);
    layout(&tmp, nullptr);
    return tmp.part_bytes[part];
}

extern "C" bt_status bt_model_create(const bt_config* cfg, void* d_workspace, size_t workspace_bytes, void* stream,
                                     bt_model** out) {
    if (!out) return fail(BT_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    bt_status st = validate(cfg);
    if (st != BT_OK) return st;
    if (!d_workspace) return fail(BT_ERR_INVALID_ARG, "workspace is NULL");
    if (reinterpret_cast<uintptr_t>(d_workspace) & 255u) return fail(BT_ERR_INVALID_ARG, "workspace not 256-byte aligned");
    bt_model* m = new bt_model{};
    fill_dims(m, cfg);
    size_t need = layout(m, nullptr);
    if (workspace_bytes < need) {
        delete m;
        return fail(BT_ERR_OOM, "workspace too small: %zu < %zu bytes", workspace_bytes, need);
    }
    if (!(cfg->flags & BT_FLAG_GEMM_SIMT)) {
        char err[256];
        if (!gemm_tc_init(err, sizeof(err))) {
            delete m;
            return fail(BT_ERR_CUDA, "tensor-core GEMM unavailable: %s", err);
        }
    }
    layout(m, static_cast<uint8_t*>(d_workspace));
    m->stream = static_cast<cudaStream_t>(stream);
    m->step = 0;
    m->curB = 0;
    m->have_forward = false;
    m->launches_at_create = g_launches.load();
    m->prof_on = false;
    m->prof_used = 0;
    m->ddp = nullptr;
    m->ddp_fn = nullptr;
    m->ddp_user = nullptr;
    m->ddp_stream = nullptr;
    m->ddp_done_ev = nullptr;
    m->ddp_sync = false;
    m->ddp_acc_weight = 0.f;
    m->debug_sync = (cfg->flags & BT_FLAG_DEBUG) != 0 || debug_env();
    std::vector<uint8_t> flags((size_t)(m->P / 1024), 0);
    for (const Tensor& t : m->tensors)
        if (t.decay)
            for (int64_t c = t.off / 1024; c < (t.off + t.numel + 1023) / 1024; ++c) flags[(size_t)c] = 1;
    // table of the GEMM weight matrices, with their 64x64 tiles numbered consecutively
    std::vector<MatDesc> descs;
    int tiles = 0;
    auto add_mat = [&](const Tensor& t, int rows, int cols) {
        MatDesc d{(long long)t.off, rows, cols, tiles, (cols + 63) / 64};
        tiles += ((rows + 63) / 64) * d.tiles_c;
        descs.push_back(d);
    };
    add_mat(m->tensors[0], m->Vp, m->C);
    for (int l = 0; l < m->L; ++l) {
        add_mat(layer_tensor(m, l, QKVW), 3 * m->C, m->C);
        add_mat(layer_tensor(m, l, PROJW), m->C, m->C);
        add_mat(layer_tensor(m, l, FCW), m->F, m->C);
        add_mat(layer_tensor(m, l, PRW), m->C, m->F);
    }
    m->n_mats = (int)descs.size();
    m->n_mat_tiles = tiles;
    cudaError_t e = cudaMemcpyAsync(m->decay_flags, flags.data(), flags.size(), cudaMemcpyHostToDevice, m->stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(m->mat_descs, descs.data(), descs.size() * sizeof(MatDesc), cudaMemcpyHostToDevice, m->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m->params, 0, (size_t)m->P * 4 * sizeof(float), m->stream);  // p,g,m,v
    if (e == cudaSuccess) e = cudaMemsetAsync(m->err_word, 0, 4 * sizeof(int), m->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(m->stream);
    if (e != cudaSuccess) {
        delete m;
        return fail(BT_ERR_CUDA, "workspace initialisation failed: %s", cudaGetErrorString(e));
    }
    *out = m;
    return BT_OK;
}

extern "C" void bt_model_destroy(bt_model* m) {
    if (!m) return;
    for (cudaEvent_t e : m->prof_events) cudaEventDestroy(e);
    bt_ddp_detach(m);
    delete m;
}

extern "C" bt_status bt_ddp_attach(bt_model* m, int64_t bucket_cap_bytes, bt_allreduce_fn fn, void* user,
                                   void* comm_stream) {
    if (!m || !fn) return fail(BT_ERR_INVALID_ARG, "ddp_attach: NULL argument");
    if ((cudaStream_t)comm_stream == m->stream)
        return fail(BT_ERR_INVALID_ARG, "ddp_attach: the communication stream must differ from the model's stream");
    bt_ddp_detach(m);
    bt_ddp_plan* plan = nullptr;
    bt_status st = build_ddp_plan(&m->cfg, bucket_cap_bytes, &plan);
    if (st != BT_OK) return st;
    std::vector<cudaEvent_t> evs(plan->buckets.size(), nullptr);
    cudaError_t e = cudaEventCreateWithFlags(&m->ddp_done_ev, cudaEventDisableTiming);
    for (size_t i = 0; i < evs.size() && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&evs[i], cudaEventDisableTiming);
    if (e != cudaSuccess) {
        for (cudaEvent_t ev : evs) if (ev) cudaEventDestroy(ev);
        if (m->ddp_done_ev) cudaEventDestroy(m->ddp_done_ev);
        m->ddp_done_ev = nullptr;
        delete plan;
        return fail(BT_ERR_CUDA, "ddp_attach: event creation failed: %s", cudaGetErrorString(e));
    }
    m->ddp = plan;
    m->ddp_ready_ev = evs;
    m->ddp_fn = fn;
    m->ddp_user = user;
    m->ddp_stream = (cudaStream_t)comm_stream;
    return BT_OK;
}

extern "C" bt_status bt_ddp_detach(bt_model* m) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    if (!m->ddp) return BT_OK;
    for (cudaEvent_t ev : m->ddp_ready_ev) cudaEventDestroy(ev);
    m->ddp_ready_ev.clear();
    if (m->ddp_done_ev) cudaEventDestroy(m->ddp_done_ev);
    m->ddp_done_ev = nullptr;
    delete m->ddp;
    m->ddp = nullptr;
    m->ddp_fn = nullptr;
    return BT_OK;
}

extern "C" bt_status bt_arena_ptr(bt_model* m, int32_t kind, float** d_ptr, int64_t* count) {
    if (!m || !d_ptr) return fail(BT_ERR_INVALID_ARG, "NULL argument");
    float* base = kind == 0 ? m->params : kind == 1 ? m->grads : kind == 2 ? m->mom1 : kind == 3 ? m->mom2 : nullptr;
    if (!base) return fail(BT_ERR_INVALID_ARG, "kind %d not in 0..3", kind);
    *d_ptr = base;
    if (count) *count = m->P;
    return BT_OK;
}

extern "C" bt_status bt_model_init(bt_model* m, uint64_t seed) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    const float std0 = 0.02f, std1 = 0.02f / sqrtf(2.0f * (float)m->L);
    BT_CUDA(cudaMemsetAsync(m->params, 0, (size_t)m->P * 4 * sizeof(float), m->stream));
    for (const Tensor& t : m->tensors) {
        float* p = m->params + t.off;
        if (t.kind == 0) BT_CUDA(launch_init_normal(p, t.numel, std0, seed, (uint64_t)t.off, m->stream));
        else if (t.kind == 1) BT_CUDA(launch_init_normal(p, t.numel, std1, seed, (uint64_t)t.off, m->stream));
        else if (t.kind == 2) BT_CUDA(launch_fill(p, t.numel, 1.0f, m->stream));
    }
    m->step = 0;
    return BT_OK;
}

extern "C" int32_t bt_num_tensors(const bt_model* m) { return m ? (int32_t)m->tensors.size() : 0; }

extern "C" bt_status bt_tensor_info(const bt_model* m, int32_t i, const char** name, int64_t* numel, int32_t* decay) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    if (i < 0 || i >= (int32_t)m->tensors.size()) return fail(BT_ERR_NOT_FOUND, "tensor index %d out of range", i);
    if (name) *name = m->tensors[i].name.c_str();
    if (numel) *numel = m->tensors[i].numel;
    if (decay) *decay = m->tensors[i].decay;
    return BT_OK;
}

extern "C" bt_status bt_tensor_ptr(bt_model* m, const char* name, int32_t kind, float** d_ptr) {
    if (!m || !name || !d_ptr) return fail(BT_ERR_INVALID_ARG, "NULL argument");
    const Tensor* t = find_tensor(m, name);
    if (!t) return fail(BT_ERR_NOT_FOUND, "no tensor named '%s'", name);
    float* base = kind == 0 ? m->params : kind == 1 ? m->grads : kind == 2 ? m->mom1 : kind == 3 ? m->mom2 : nullptr;
    if (!base) return fail(BT_ERR_INVALID_ARG, "kind %d not in 0..3", kind);
    *d_ptr = base + t->off;
    return BT_OK;
}

extern "C" bt_status bt_activation_ptr(bt_model* m, const char* name, int32_t layer, float** d_ptr, int64_t* numel) {
    if (!m || !name || !d_ptr) return fail(BT_ERR_INVALID_ARG, "NULL argument");
    const int64_t N = (int64_t)m->curB * m->T, C = m->C, F = m->F;
    std::string n(name);
    float* p = nullptr;
    int64_t ne = 0;
    if (n == "xL") { p = m->xL; ne = N * C; }
    else if (n == "xf") { p = m->xf_s; ne = N * C; }
    else if (n == "logits") {
        if (m->cfg.flags & BT_FLAG_LOGITS_IN_PLACE)
            return fail(BT_ERR_NOT_FOUND, "the logits are not kept with BT_FLAG_LOGITS_IN_PLACE (their gradient overwrites them)");
        p = m->logits; ne = N * m->Vp;
    }
    else if (n == "dlogits") { p = m->dlogits_s; ne = N * m->Vp; }
    else if (n == "losses") { p = m->losses; ne = N; }
    else {
        if (layer < 0 || layer >= m->L) return fail(BT_ERR_NOT_FOUND, "layer %d out of range", layer);
        LayerAct& a = m->act[layer];
        if (n == "x") { p = a.x; ne = N * C; }
        else if (n == "qkv_split") { p = a.qkv_s; ne = N * 3 * C; }
        else if (n == "a") { p = a.a_s; ne = N * C; }
        else if (n == "qkv") {
            if (!a.qkv) return fail(BT_ERR_NOT_FOUND, "the raw qkv array is not kept in this configuration (use qkv_split)");
            p = a.qkv; ne = N * 3 * C;
        }
        else if (n == "o") { p = a.o_s; ne = N * C; }
        else if (n == "lse") { p = a.lse; ne = (int64_t)m->curB * m->H * m->T; }
        else if (n == "x1") { p = a.x1; ne = N * C; }
        else if (n == "m") { p = a.m_s; ne = N * C; }
        else if (n == "h") { p = a.h; ne = N * F; }
        else if (n == "g") { p = a.g_s; ne = N * F; }
        else if (n == "ln1.mean") { p = a.mean1; ne = N; }
        else if (n == "ln1.rstd") { p = a.rstd1; ne = N; }
        else if (n == "ln2.mean") { p = a.mean2; ne = N; }
        else if (n == "ln2.rstd") { p = a.rstd2; ne = N; }
        else return fail(BT_ERR_NOT_FOUND, "no activation named '%s'", name);
    }
    *d_ptr = p;
    if (numel) *numel = ne;
    return BT_OK;
}

extern "C" int64_t bt_get_step(const bt_model* m) { return m ? m->step : -1; }
extern "C" bt_status bt_set_step(bt_model* m, int64_t t) {
    if (!m || t < 0) return fail(BT_ERR_INVALID_ARG, "bad argument");
    m->step = t;
    return BT_OK;
}
extern "C" int64_t bt_launch_count(const bt_model* m) { return m ? g_launches.load() - m->launches_at_create : 0; }
extern "C" const char* bt_last_error(void) { return g_last_error.c_str(); }

extern "C" bt_status bt_profile_enable(bt_model* m, int32_t on) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    BT_CUDA(cudaStreamSynchronize(m->stream));
    m->prof_on = on != 0;
    m->prof_recs.clear();
    m->prof_used = 0;
    return BT_OK;
}
extern "C" int32_t bt_profile_num_categories(void) { return kNumCats; }
extern "C" const char* bt_profile_category_name(int32_t cat) {
    return (cat >= 0 && cat < kNumCats) ? kCatNames[cat] : nullptr;
}
extern "C" bt_status bt_profile_read(bt_model* m, int32_t cat, double* ms_total, int64_t* launches, double* flops,
                                     double* bytes) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    if (cat < 0 || cat >= kNumCats) return fail(BT_ERR_NOT_FOUND, "category %d out of range", cat);
    BT_CUDA(cudaStreamSynchronize(m->stream));
    double ms = 0.0, fl = 0.0, by = 0.0;
    int64_t n = 0;
    for (const ProfRec& r : m->prof_recs) {
        if (r.cat != cat) continue;
        float t = 0.f;
        BT_CUDA(cudaEventElapsedTime(&t, m->prof_events[r.ev], m->prof_events[r.ev + 1]));
        ms += t; fl += r.flops; by += r.bytes; ++n;
    }
    if (ms_total) *ms_total = ms;
    if (launches) *launches = n;
    if (flops) *flops = fl;
    if (bytes) *bytes = by;
    return BT_OK;
}

// =============================================================================== the step

extern "C" bt_status bt_forward(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                                float* h_loss) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    if (!d_tokens || !d_targets) return fail(BT_ERR_INVALID_ARG, "tokens/targets NULL");
    if (B < 1 || B > m->maxB) return fail(BT_ERR_INVALID_ARG, "batch %d not in [1, %d]", B, m->maxB);
    cudaStream_t s = m->stream;
    const int C = m->C, F = m->F, T = m->T, H = m->H, Vp = m->Vp;
    const int64_t N = (int64_t)B * T;
    constexpr bool gemm_is_fwd = true;   // timing category of this function's GEMMs
    const bool simt_attn = (m->cfg.flags & BT_FLAG_ATTN_SIMT) != 0;
    const int tanh_form = (m->cfg.flags & BT_FLAG_GELU_TANH) ? 1 : 0;
    // the tcgen05 attention kernels read qkv only as hi/lo planes; the raw copy is written only
    // for the kernels that need it
    const bool raw_qkv = simt_attn || ((C / H) != 64 && (C / H) != 128) || (m->cfg.flags & BT_FLAG_GEMM_SIMT);

    // hi/lo planes of every parameter (weights are GEMM operands; one streaming pass)
    BT_STEP(kCatSplit, 0, 20.0 * m->P, launch_split_matrices(m->params, m->wsplit, m->wsplit_t, m->P, m->mat_descs, m->n_mats,
                                  m->n_mat_tiles, s));
    BT_STEP(kCatEmbedFwd, N * C, 12.0 * N * C, launch_embedding_fwd(d_tokens, m->params + m->tensors[0].off, m->params + m->tensors[1].off, N, T, C,
                                 m->V, m->act[0].x, m->err_word + 1, s));
    for (int l = 0; l < m->L; ++l) {
        LayerAct& a = m->act[l];
        float* xout = (l + 1 < m->L) ? m->act[l + 1].x : m->xL;
        auto P = [&](int k) { return m->params + layer_tensor(m, l, k).off; };
        BT_STEP(kCatLnFwd, 0, 12.0 * N * C, launch_layernorm_fwd(a.x, P(LN1G), P(LN1B), N, C, nullptr, a.a_s, a.a_s + N * C, a.mean1, a.rstd1, s));
        BT_GEMM_SPLIT_OUT(kNN, N, 3 * C, C, act_mat(a.a_s, N, C, N), weight_mat_t(m, layer_tensor(m, l, QKVW), 3 * C, C),
                          raw_qkv ? a.qkv : nullptr, a.qkv_s, P(QKVB), nullptr);
        BT_STEP(kCatAttnFwd, attn_fwd_flops(B, H, T, C / H), 20.0 * N * C, launch_attention_fwd(raw_qkv ? a.qkv : nullptr, a.qkv_s, N * 3 * C, B, T, C, H, nullptr, a.o_s, a.o_s + N * C, a.lse, simt_attn,
                                     m->err_word, s));
        BT_GEMM(kNN, N, C, C, act_mat(a.o_s, N, C, N), weight_mat_t(m, layer_tensor(m, l, PROJW), C, C), a.x1,
                     P(PROJB), a.x);
        BT_STEP(kCatLnFwd, 0, 12.0 * N * C, launch_layernorm_fwd(a.x1, P(LN2G), P(LN2B), N, C, nullptr, a.m_s, a.m_s + N * C, a.mean2, a.rstd2, s));
        // g = GELU(h), h = m Wfc^T + bfc, leaves the epilogue as hi/lo planes; what the backward needs of h
        // is GELU'(h), which the same epilogue writes in its place (h itself when GELU is recomputed later)
        BT_STEP(kCatGemmNT, gemm_flops(N, F, C), gemm_bytes(N, F, C) + 8.0 * N * F,
                gemm_raw(m, kNN, N, F, C, act_mat(a.m_s, N, C, N), weight_mat_t(m, layer_tensor(m, l, FCW), F, C), a.h,
                         P(FCB), nullptr, a.g_s, (tanh_form ? 2 : 1) + (h_holds_gelu_grad(m) ? 2 : 0)));
        BT_GEMM(kNN, N, C, F, act_mat(a.g_s, N, F, N), weight_mat_t(m, layer_tensor(m, l, PRW), C, F), xout,
                     P(PRB), a.x1);
    }
    const Tensor& lnfg = m->tensors[m->tensors.size() - 2];
    const Tensor& lnfb = m->tensors[m->tensors.size() - 1];
    BT_STEP(kCatLnFwd, 0, 12.0 * N * C, launch_layernorm_fwd(m->xL, m->params + lnfg.off, m->params + lnfb.off, N, C, nullptr, m->xf_s,
                                 m->xf_s + N * C, m->meanf, m->rstdf, s));
    BT_GEMM(kNN, N, Vp, C, act_mat(m->xf_s, N, C, N), weight_mat_t(m, m->tensors[0], Vp, C), m->logits, nullptr,
                 nullptr);
    BT_STEP(kCatXent, 0, 12.0 * N * Vp, launch_softmax_xent(m->logits, d_targets, N, Vp, 1.0f / (float)N, m->losses, m->loss, nullptr,
                                m->dlogits_s, m->dlogits_s + N * Vp, m->V, m->err_word + 2, s));
    m->curB = B;
    m->cur_tok = d_tokens;
    m->have_forward = true;
    if (h_loss) return bt_get_loss(m, h_loss);
    if (m->debug_sync) return check_device_error(m);
    return BT_OK;
}

extern "C" bt_status bt_get_loss(bt_model* m, float* h_loss) {
    if (!m || !h_loss) return fail(BT_ERR_INVALID_ARG, "NULL argument");
    BT_CUDA(cudaMemcpyAsync(h_loss, m->loss, sizeof(float), cudaMemcpyDeviceToHost, m->stream));
    return check_device_error(m);
}

static bt_status backward_impl(bt_model* m);

extern "C" bt_status bt_backward(bt_model* m) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    m->ddp_sync = true;          // a plain backward always exchanges gradients when ranks are attached
    m->ddp_acc_weight = 0.f;
    return backward_impl(m);
}

static bt_status backward_impl(bt_model* m) {
    if (!m->have_forward) return fail(BT_ERR_INVALID_ARG, "bt_backward without a preceding bt_forward");
    cudaStream_t s = m->stream;
    constexpr bool gemm_is_fwd = false;  // timing category of this function's GEMMs
    const int B = m->curB, C = m->C, F = m->F, T = m->T, H = m->H, Vp = m->Vp;
    const int64_t N = (int64_t)B * T;
    const bool simt_attn = (m->cfg.flags & BT_FLAG_ATTN_SIMT) != 0;
    const int tanh_form = (m->cfg.flags & BT_FLAG_GELU_TANH) ? 1 : 0;
    const bool raw_qkv = simt_attn || ((C / H) != 64 && (C / H) != 128) || (m->cfg.flags & BT_FLAG_GEMM_SIMT);
    const bool recompute_ln = (m->cfg.flags & BT_FLAG_RECOMPUTE_LN) != 0;
    const bool recompute_gelu = (m->cfg.flags & BT_FLAG_RECOMPUTE_GELU) != 0;
    auto G = [&](const Tensor& t) { return m->grads + t.off; };
    // data-parallel exchange: registry indices of the tensors whose gradients each launch group finishes
    const int nT = (int)m->tensors.size();
    auto LI = [&](int l, int k) { return 2 + 12 * l + k; };
    if (m->ddp && m->ddp_sync) bt_ddp_plan_reset(m->ddp);

    // LM head: dxf = dlogits . wte ; dwte = dlogits^T . xf
    SplitMat dlog = act_mat(m->dlogits_s, N, Vp, N);
    BT_GEMM(kNN, N, C, Vp, dlog, weight_mat(m, m->tensors[0], Vp, C), m->dtmp, nullptr, nullptr);
    BT_GEMM(kTN, Vp, C, N, dlog, act_mat(m->xf_s, N, C, N), G(m->tensors[0]), nullptr, nullptr);
    const Tensor& lnfg = m->tensors[m->tensors.size() - 2];
    const Tensor& lnfb = m->tensors[m->tensors.size() - 1];
    // Every LayerNorm backward also sums the columns of the residual gradient it writes: that is
    // the bias gradient of the projection whose output this residual stream position is.
    BT_STEP(kCatLnBwd, 0, 24.0 * N * C, launch_layernorm_bwd(m->dtmp, m->xL, m->params + lnfg.off, m->meanf, m->rstdf, nullptr, N, C, m->dres,
                                 m->dres_s, m->dres_s + N * C, G(lnfg), G(lnfb), G(layer_tensor(m, m->L - 1, PRB)), m->ln_scratch, s));
    BT_DDP_READY(nT - 1, nT - 2, LI(m->L - 1, PRB));
    SplitMat dres = act_mat(m->dres_s, N, C, N);
    for (int l = m->L - 1; l >= 0; --l) {
        LayerAct& a = m->act[l];
        auto LT = [&](int k) -> Tensor& { return layer_tensor(m, l, k); };
        // MLP down-projection: x_out = x1 + g . Wpr^T + bpr
        // d h = (d x_out . Wpr) o GELU'(h): the GELU backward runs in the product's epilogue (a plain
        // multiplication where the forward pass left GELU'(h)), which also leaves the column sums of
        // d h per 32-row group (added up below: the gradient of bfc)
        const bool fused_gelu_bwd = m->dg == nullptr;
        if (fused_gelu_bwd)
            BT_STEP(kCatGemmNN, gemm_flops(N, F, C), gemm_bytes(N, F, C) + 8.0 * N * F,
                    gemm_raw(m, kNN, N, F, C, dres, weight_mat(m, LT(PRW), C, F), nullptr, nullptr, a.h, m->dh_s,
                             h_holds_gelu_grad(m) ? 7 : tanh_form ? 6 : 5, m->dh_groups));
        else
            BT_GEMM(kNN, N, F, C, dres, weight_mat(m, LT(PRW), C, F), m->dg, nullptr, nullptr);
        if (recompute_gelu)   // g = GELU(h) again, as hi/lo planes (the same function of the same values as the epilogue's)
            BT_STEP(kCatGeluFwd, 0, 12.0 * N * F, launch_gelu_fwd(a.h, N * F, tanh_form, nullptr, a.g_s, a.g_s + N * F, s));
        BT_GEMM(kTN, C, F, N, dres, act_mat(a.g_s, N, F, N), G(LT(PRW)), nullptr, nullptr);
        BT_DDP_READY(LI(l, PRW));
        if (fused_gelu_bwd)
            BT_STEP(kCatColsum, 0, 4.0 * ((N + 31) / 32) * F, launch_colsum_stage2(m->dh_groups, (int)((N + 31) / 32), (int)F, G(LT(FCB)), s));
        else   // d h, with its column sums taken in the same pass
            BT_STEP(kCatGeluBwd, 0, 16.0 * N * F, launch_gelu_bwd_colsum(a.h, m->dg, N, F, tanh_form, nullptr, m->dh_s, m->dh_s + N * F,
                                           G(LT(FCB)), m->colsum_scratch, s));
        BT_DDP_READY(LI(l, FCB));
        // MLP up-projection: h = m . Wfc^T + bfc
        SplitMat dh = act_mat(m->dh_s, N, F, N);
        BT_GEMM(kNN, N, C, F, dh, weight_mat(m, LT(FCW), F, C), m->dtmp, nullptr, nullptr);
        if (recompute_ln)   // m = LN2(x1) again (bit-identical to the forward's: same kernel, same inputs)
            BT_STEP(kCatLnFwd, 0, 12.0 * N * C, launch_layernorm_fwd(a.x1, m->params + LT(LN2G).off, m->params + LT(LN2B).off, N, C, nullptr,
                                                                       a.m_s, a.m_s + N * C, nullptr, nullptr, s));
        BT_GEMM(kTN, F, C, N, dh, act_mat(a.m_s, N, C, N), G(LT(FCW)), nullptr, nullptr);
        BT_DDP_READY(LI(l, FCW));
        // LN2 and the residual: d x1 = d x_out + LN2'(dm)
        BT_STEP(kCatLnBwd, 0, 24.0 * N * C, launch_layernorm_bwd(m->dtmp, a.x1, m->params + LT(LN2G).off, a.mean2, a.rstd2, m->dres, N, C, m->dres,
                                     m->dres_s, m->dres_s + N * C, G(LT(LN2G)), G(LT(LN2B)), G(LT(PROJB)), m->ln_scratch, s));
        BT_DDP_READY(LI(l, LN2B), LI(l, LN2G), LI(l, PROJB));
        // attention output projection: x1 = x + o . Wo^T + bo
        // d o, raw for the FMA / warp-MMA attention kernels, as hi/lo planes for the tcgen05 ones
        BT_GEMM_SPLIT_OUT(kNN, N, C, C, dres, weight_mat(m, LT(PROJW), C, C), raw_qkv ? m->dtmp : nullptr, m->do_s, nullptr,
                          nullptr);
        BT_GEMM(kTN, C, C, N, dres, act_mat(a.o_s, N, C, N), G(LT(PROJW)), nullptr, nullptr);
        BT_DDP_READY(LI(l, PROJW));
        bool rg_written = false;
        BT_STEP(kCatAttnBwd, 2.5 * attn_fwd_flops(B, H, T, C / H), 48.0 * N * C, launch_attention_bwd(raw_qkv ? a.qkv : nullptr, a.qkv_s, N * 3 * C, a.o_s, a.o_s + N * C, a.lse,
                                     raw_qkv ? m->dtmp : nullptr, m->do_s, N * C, B, T,
                                     C, H, nullptr, m->dqkv_s, m->dqkv_s + N * 3 * C, m->dvec, simt_attn, m->err_word, s,
                                     m->attn_rg, &rg_written));
        // QKV projection: qkv = a . Wqkv^T + bqkv
        SplitMat dqkv = act_mat(m->dqkv_s, N, 3 * C, N);
        BT_GEMM(kNN, N, C, 3 * C, dqkv, weight_mat(m, LT(QKVW), 3 * C, C), m->dtmp, nullptr, nullptr);
        if (recompute_ln)   // a = LN1(x) again
            BT_STEP(kCatLnFwd, 0, 12.0 * N * C, launch_layernorm_fwd(a.x, m->params + LT(LN1G).off, m->params + LT(LN1B).off, N, C, nullptr,
                                                                       a.a_s, a.a_s + N * C, nullptr, nullptr, s));
        BT_GEMM(kTN, 3 * C, C, N, dqkv, act_mat(a.a_s, N, C, N), G(LT(QKVW)), nullptr, nullptr);
        // d bqkv: from the attention kernels' per-row-group sums when they wrote them, else a pass over dqkv
        if (rg_written)
            BT_STEP(kCatColsum, 0, 12.0 * attention_bwd_rowgroups(B, T) * C,
                    launch_colsum(m->attn_rg, nullptr, attention_bwd_rowgroups(B, T), 3 * C, G(LT(QKVB)), m->colsum_scratch, s));
        else
            BT_STEP(kCatColsum, 0, 24.0 * N * C, launch_colsum(m->dqkv_s, m->dqkv_s + N * 3 * C, N, 3 * C, G(LT(QKVB)), m->colsum_scratch, s));
        BT_DDP_READY(LI(l, QKVB), LI(l, QKVW));
        // LN1 and the residual: d x = d x1 + LN1'(da)
        BT_STEP(kCatLnBwd, 0, 24.0 * N * C, launch_layernorm_bwd(m->dtmp, a.x, m->params + LT(LN1G).off, a.mean1, a.rstd1, m->dres, N, C, m->dres,
                                     m->dres_s, m->dres_s + N * C, G(LT(LN1G)), G(LT(LN1B)),
                                     l > 0 ? G(layer_tensor(m, l - 1, PRB)) : nullptr, m->ln_scratch, s));
        BT_DDP_READY(LI(l, LN1B), LI(l, LN1G));
        if (l > 0) BT_DDP_READY(LI(l - 1, PRB));
    }
    // embeddings: dwte (already holding the LM-head part) += gather-transpose, dwpe = sum over sequences
    BT_STEP(kCatEmbedBwd, 0, 8.0 * N * C, launch_embedding_bwd(m->cur_tok, m->dres, N, T, C, m->V, Vp, G(m->tensors[0]), G(m->tensors[1]),
                                                              m->dtmp, m->emb_table, s));
    BT_DDP_READY(1, 0);
    if (m->debug_sync) return check_device_error(m);
    return BT_OK;
}

extern "C" bt_status bt_adamw_step(bt_model* m, const bt_adamw_config* opt, float* h_grad_norm) {
    if (!m || !opt) return fail(BT_ERR_INVALID_ARG, "NULL argument");
    if (!(opt->beta1 >= 0.f && opt->beta1 < 1.f) || !(opt->beta2 >= 0.f && opt->beta2 < 1.f) || !(opt->eps > 0.f))
        return fail(BT_ERR_INVALID_ARG, "AdamW: betas must lie in [0,1) and eps must be positive");
    cudaStream_t s = m->stream;
    BT_STEP(kCatGradNorm, 0, 4.0 * m->P, launch_grad_norm(m->grads, m->P, opt->grad_clip, m->norm_out, m->norm_scratch, s));
    m->step += 1;
    AdamParams hp;
    hp.lr = opt->lr; hp.beta1 = opt->beta1; hp.beta2 = opt->beta2; hp.eps = opt->eps; hp.weight_decay = opt->weight_decay;
    hp.inv_c1 = (float)(1.0 / (1.0 - std::pow((double)opt->beta1, (double)m->step)));
    hp.inv_c2 = (float)(1.0 / (1.0 - std::pow((double)opt->beta2, (double)m->step)));
    BT_STEP(kCatAdamW, 0, 28.0 * m->P, launch_adamw_flat(m->params, m->grads, m->mom1, m->mom2, m->P, m->decay_flags, hp, m->norm_out + 1, s));
    if (h_grad_norm) {
        BT_CUDA(cudaMemcpyAsync(h_grad_norm, m->norm_out, sizeof(float), cudaMemcpyDeviceToHost, s));
        return check_device_error(m);
    }
    if (m->debug_sync) return check_device_error(m);
    return BT_OK;
}

extern "C" bt_status bt_train_step(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                                   const bt_adamw_config* opt, float* h_loss) {
    bt_status st = bt_forward(m, d_tokens, d_targets, B, nullptr);
    if (st != BT_OK) return st;
    st = bt_backward(m);
    if (st != BT_OK) return st;
    st = bt_adamw_step(m, opt, nullptr);
    if (st != BT_OK) return st;
    if (h_loss) return bt_get_loss(m, h_loss);
    return BT_OK;
}

extern "C" bt_status bt_micro_step(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                                   int32_t micro_index, int32_t n_micro, float* h_loss) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    if (n_micro < 1 || micro_index < 0 || micro_index >= n_micro)
        return fail(BT_ERR_INVALID_ARG, "micro step %d of %d", micro_index, n_micro);
    bt_status st = bt_forward(m, d_tokens, d_targets, B, nullptr);
    if (st != BT_OK) return st;
    // Algorithm 1: gradients are exchanged on the last micro-step only; there the accumulation
    // g = acc + g / n is applied bucket by bucket, just before each bucket's all-reduce
    const bool last = micro_index == n_micro - 1;
    const bool per_bucket = m->ddp != nullptr && last && n_micro > 1;
    m->ddp_sync = last;
    m->ddp_acc_weight = per_bucket ? 1.0f / (float)n_micro : 0.f;
    st = backward_impl(m);
    m->ddp_acc_weight = 0.f;
    if (st != BT_OK) return st;
    if (n_micro > 1) {
        const int mode = micro_index == 0 ? 0 : last ? 2 : 1;
        // with buckets the gradient ranges are already folded in: only the loss word is left (n = 0)
        BT_CUDA(launch_grad_accumulate(m->gacc, m->grads, per_bucket ? 0 : m->P, 1.0f / (float)n_micro, mode, m->loss_acc,
                                       m->loss, m->stream));
    }
    if (h_loss) return bt_get_loss(m, h_loss);
    return BT_OK;
}

extern "C" bt_status bt_train_step_accum(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                                         int32_t n_micro, const bt_adamw_config* opt, float* h_loss) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    if (n_micro < 1) return fail(BT_ERR_INVALID_ARG, "n_micro < 1");
    for (int32_t i = 0; i < n_micro; ++i) {
        const int64_t off = (int64_t)i * B * m->T;
        bt_status st = bt_micro_step(m, d_tokens + off, d_targets + off, B, i, n_micro, nullptr);
        if (st != BT_OK) return st;
    }
    bt_status st = bt_adamw_step(m, opt, nullptr);
    if (st != BT_OK) return st;
    if (h_loss) return bt_get_loss(m, h_loss);
    return BT_OK;
}

extern "C" float bt_lr_at(const bt_lr_schedule* s, int64_t step) {
    if (!s || step < 1) return 0.0f;
    if (s->warmup_steps > 0 && step <= s->warmup_steps) return s->max_lr * (float)((double)step / (double)s->warmup_steps);
    if (step >= s->max_steps || s->max_steps <= s->warmup_steps) return s->min_lr;
    const double frac = (double)(step - s->warmup_steps) / (double)(s->max_steps - s->warmup_steps);
    return (float)((double)s->min_lr + 0.5 * (1.0 + std::cos(3.14159265358979323846 * frac)) * ((double)s->max_lr - (double)s->min_lr));
}

extern "C" bt_status bt_train_step_host(bt_model* m, const int32_t* h_tokens, const int32_t* h_targets, int32_t B,
                                        const bt_adamw_config* opt, float* h_loss) {
    if (!m || !h_tokens || !h_targets) return fail(BT_ERR_INVALID_ARG, "NULL argument");
    if (B < 1 || B > m->maxB) return fail(BT_ERR_INVALID_ARG, "batch %d not in [1, %d]", B, m->maxB);
    const size_t bytes = (size_t)B * m->T * sizeof(int32_t);
    // the ids are on the host here: check them before anything is enqueued
    int64_t bad = first_bad_id(h_tokens, (int64_t)B * m->T, m->V);
    if (bad >= 0) return fail(BT_ERR_INVALID_ARG, "token id %d outside [0, %d) at position %lld", h_tokens[bad], m->V, (long long)bad);
    bad = first_bad_id(h_targets, (int64_t)B * m->T, m->V);
    if (bad >= 0) return fail(BT_ERR_INVALID_ARG, "target id %d outside [0, %d) at position %lld", h_targets[bad], m->V, (long long)bad);
    BT_CUDA(cudaMemcpyAsync(m->tok_stage, h_tokens, bytes, cudaMemcpyHostToDevice, m->stream));
    BT_CUDA(cudaMemcpyAsync(m->tgt_stage, h_targets, bytes, cudaMemcpyHostToDevice, m->stream));
    return bt_train_step(m, m->tok_stage, m->tgt_stage, B, opt, h_loss);
}

extern "C" bt_status bt_selftest_bounded_wait(bt_model* m, float limit_ms) {
    if (!m) return fail(BT_ERR_INVALID_ARG, "model is NULL");
    if (!(limit_ms > 0.f) || limit_ms > 1000.f) return fail(BT_ERR_INVALID_ARG, "limit_ms must lie in (0, 1000]");
    BT_CUDA(launch_bounded_wait_probe(m->err_word, (unsigned long long)((double)limit_ms * 1e6), kSelftestWaitCode, m->stream));
    return check_device_error(m);
}

extern "C" bt_status bt_probe_tf32_mma_rate(int32_t n_ctas, int32_t iters, int64_t* d_clocks, int32_t* d_err,
                                            void* stream) {
    if (!d_clocks || !d_err) return fail(BT_ERR_INVALID_ARG, "probe: NULL argument");
    if (reinterpret_cast<uintptr_t>(d_clocks) & 7u) return fail(BT_ERR_INVALID_ARG, "probe: d_clocks not 8-byte aligned");
    if (n_ctas < 1 || n_ctas > 4096 || iters < 16 || iters > (1 << 20))
        return fail(BT_ERR_INVALID_ARG, "probe: n_ctas in [1, 4096], iters in [16, 2^20]");
    BT_CUDA(launch_tf32_rate_probe(n_ctas, iters, reinterpret_cast<long long*>(d_clocks), d_err, (cudaStream_t)stream));
    return BT_OK;
}

extern "C" bt_status bt_probe_mma_issue_rate(int32_t n, int32_t a_in_tmem, int32_t issuers, int32_t n_ctas, int32_t iters,
                                             int64_t* d_clocks, int32_t* d_err, void* stream) {
    if (!d_clocks || !d_err) return fail(BT_ERR_INVALID_ARG, "probe: NULL argument");
    if (reinterpret_cast<uintptr_t>(d_clocks) & 7u) return fail(BT_ERR_INVALID_ARG, "probe: d_clocks not 8-byte aligned");
    if ((n != 64 && n != 128 && n != 256) || (n == 256 && a_in_tmem) || issuers < 1 || issuers > 4)
        return fail(BT_ERR_INVALID_ARG, "probe: n in {64, 128, 256} (256: A in shared memory only), issuers in [1, 4]");
    if (n_ctas < 1 || n_ctas > 4096 || iters < 16 || iters > (1 << 20))
        return fail(BT_ERR_INVALID_ARG, "probe: n_ctas in [1, 4096], iters in [16, 2^20]");
    BT_CUDA(launch_mma_issue_probe(n, a_in_tmem ? 1 : 0, issuers, n_ctas, iters, reinterpret_cast<long long*>(d_clocks), d_err,
                                   (cudaStream_t)stream));
    return BT_OK;
}

// =============================================================================== per-op entry points

extern "C" bt_status bt_op_embedding_fwd(const int32_t* tok, const float* wte, const float* wpe, int64_t N, int32_t T,
                                         int32_t C, int32_t V, float* x, int32_t* d_bad, void* stream) {
    BT_PTR(tok); BT_PTR(wte); BT_PTR(wpe); BT_PTR(x);
    if (N < 0 || T < 1 || C < 4 || C % 4 || V < 1) return fail(BT_ERR_INVALID_ARG, "embedding_fwd: bad sizes");
    if (N == 0) return BT_OK;
    BT_CUDA(launch_embedding_fwd(tok, wte, wpe, N, T, C, V, x, d_bad, (cudaStream_t)stream));
    return BT_OK;
}

extern "C" size_t bt_op_embedding_bwd_scratch_bytes(int64_t N, int32_t C, int32_t V) {
    if (N < 1 || C < 4 || V < 1) return 0;
    return embedding_bwd_scratch_bytes(N, C, V);
}

extern "C" bt_status bt_op_embedding_bwd(const int32_t* tok, const float* dx, int64_t N, int32_t T, int32_t C, int32_t V,
                                         float* dwte, float* dwpe, void* scratch, size_t scratch_bytes, void* stream) {
    BT_PTR(tok); BT_PTR(dx); BT_PTR(dwte); BT_PTR(dwpe); BT_PTR(scratch);
    if (N < 1 || T < 1 || C < 4 || C % 4 || N % T || N > (1 << 24) || V < 1)
        return fail(BT_ERR_INVALID_ARG, "embedding_bwd: bad sizes");
    if (scratch_bytes < embedding_bwd_scratch_bytes(N, C, V)) return fail(BT_ERR_OOM, "embedding_bwd: scratch too small");
    const size_t partial_bytes = embedding_bwd_partial_bytes(N, C);
    BT_CUDA(launch_embedding_bwd(tok, dx, N, T, C, V, V, dwte, dwpe, (float*)scratch, (uint8_t*)scratch + partial_bytes,
                                 (cudaStream_t)stream));
    return BT_OK;
}

extern "C" int64_t bt_first_invalid_id(const int32_t* h_ids, int64_t n, int32_t vocab_size) {
    if ((!h_ids && n > 0) || n < 0 || vocab_size < 1) return -2;
    return first_bad_id(h_ids, n, vocab_size);
}

extern "C" bt_status bt_op_layernorm_fwd(const float* x, const float* gamma, const float* beta, int64_t N, int32_t C,
                                         float* y, float* y_split, float* mean, float* rstd, void* stream) {
    BT_PTR(x); BT_PTR(gamma); BT_PTR(beta); BT_OPT_PTR(y); BT_OPT_PTR(y_split);
    if (N < 0 || C < 4 || C % 4) return fail(BT_ERR_INVALID_ARG, "layernorm_fwd: bad sizes");
    if (C > 4096) return fail(BT_ERR_UNSUPPORTED, "layernorm_fwd: C > 4096");
    if (N == 0) return BT_OK;
    BT_CUDA(launch_layernorm_fwd(x, gamma, beta, N, C, y, y_split, y_split ? y_split + N * C : nullptr, mean, rstd,
                                 (cudaStream_t)stream));
    return BT_OK;
}

extern "C" size_t bt_op_layernorm_bwd_scratch_bytes(int64_t N, int32_t C) {
    return layernorm_bwd_scratch_floats(N, C) * sizeof(float);
}

static bt_status layernorm_bwd_impl(const float* dy, const float* x, const float* gamma, const float* mean,
                                    const float* rstd, const float* dres, int64_t N, int32_t C, float* dx,
                                    float* dx_split, float* dgamma, float* dbeta, float* dx_colsum, void* scratch,
                                    size_t scratch_bytes, void* stream) {
    BT_PTR(dy); BT_PTR(x); BT_PTR(gamma); BT_PTR(mean); BT_PTR(rstd); BT_OPT_PTR(dres); BT_OPT_PTR(dx);
    BT_OPT_PTR(dx_split); BT_PTR(dgamma); BT_PTR(dbeta); BT_OPT_PTR(dx_colsum); BT_PTR(scratch);
    if (N < 1 || C < 4 || C % 4) return fail(BT_ERR_INVALID_ARG, "layernorm_bwd: bad sizes");
    if (C > 4096) return fail(BT_ERR_UNSUPPORTED, "layernorm_bwd: C > 4096");
    if (scratch_bytes < bt_op_layernorm_bwd_scratch_bytes(N, C)) return fail(BT_ERR_OOM, "layernorm_bwd: scratch too small");
    BT_CUDA(launch_layernorm_bwd(dy, x, gamma, mean, rstd, dres, N, C, dx, dx_split,
                                 dx_split ? dx_split + N * C : nullptr, dgamma, dbeta, dx_colsum, (float*)scratch,
                                 (cudaStream_t)stream));
    return BT_OK;
}

extern "C" bt_status bt_op_layernorm_bwd(const float* dy, const float* x, const float* gamma, const float* mean,
                                         const float* rstd, const float* dres, int64_t N, int32_t C, float* dx,
                                         float* dx_split, float* dgamma, float* dbeta, void* scratch,
                                         size_t scratch_bytes, void* stream) {
    return layernorm_bwd_impl(dy, x, gamma, mean, rstd, dres, N, C, dx, dx_split, dgamma, dbeta, nullptr, scratch,
                              scratch_bytes, stream);
}

extern "C" bt_status bt_op_layernorm_bwd_colsum(const float* dy, const float* x, const float* gamma, const float* mean,
                                                const float* rstd, const float* dres, int64_t N, int32_t C, float* dx,
                                                float* dx_split, float* dgamma, float* dbeta, float* dx_colsum,
                                                void* scratch, size_t scratch_bytes, void* stream) {
    if (!dx_colsum) return fail(BT_ERR_INVALID_ARG, "layernorm_bwd_colsum: dx_colsum is NULL");
    return layernorm_bwd_impl(dy, x, gamma, mean, rstd, dres, N, C, dx, dx_split, dgamma, dbeta, dx_colsum, scratch,
                              scratch_bytes, stream);
}

namespace {
struct GemmShapes { int64_t a_rows, a_cols, b_rows, b_cols; };
GemmShapes gemm_shapes(int layout, int64_t M, int64_t N, int64_t K) {
    GemmShapes s;
    if (layout == BT_GEMM_TN) { s.a_rows = K; s.a_cols = M; } else { s.a_rows = M; s.a_cols = K; }
    if (layout == BT_GEMM_NT) { s.b_rows = N; s.b_cols = K; } else { s.b_rows = K; s.b_cols = N; }
    return s;
}
inline size_t pad256(size_t n) { return (n + 63) / 64 * 64; }  // floats
}  // namespace

extern "C" size_t bt_op_gemm_split_scratch_bytes(void) {
    return (gemm_tc_partial_floats_bound() + 64) * sizeof(float);
}

extern "C" size_t bt_op_gemm_scratch_bytes(int32_t layout, int64_t M, int64_t N, int64_t K) {
    if (layout < 0 || layout > 2 || M < 1 || N < 1 || K < 1) return 0;
    GemmShapes s = gemm_shapes(layout, M, N, K);
    return (pad256(2 * s.a_rows * s.a_cols) + pad256(2 * s.b_rows * s.b_cols)) * sizeof(float) +
           bt_op_gemm_split_scratch_bytes();
}

extern "C" bt_status bt_op_split(const float* x, int64_t n, float* x_split, void* stream) {
    BT_PTR(x); BT_PTR(x_split);
    if (n < 0 || n % 4) return fail(BT_ERR_INVALID_ARG, "split: n must be a non-negative multiple of 4");
    if (n == 0) return BT_OK;
    BT_CUDA(launch_split(x, x_split, x_split + n, n, (cudaStream_t)stream));
    return BT_OK;
}

static bt_status gemm_split_impl(int32_t layout, int64_t M, int64_t N, int64_t K, const float* A_split,
                                 const float* B_split, float* D, float* D_act_split, int32_t act, const float* bias,
                                 const float* residual, void* scratch, size_t scratch_bytes, uint32_t flags,
                                 void* stream) {
    BT_PTR(A_split); BT_PTR(B_split); BT_PTR(D); BT_OPT_PTR(D_act_split); BT_OPT_PTR(bias); BT_OPT_PTR(residual);
    BT_PTR(scratch);
    if (act < 0 || act > 4) return fail(BT_ERR_INVALID_ARG, "gemm: act %d", act);
    if (layout < 0 || layout > 2) return fail(BT_ERR_INVALID_ARG, "gemm: layout %d", layout);
    if (M < 1 || N < 1 || K < 1 || M % 4 || N % 4 || K % 4) return fail(BT_ERR_INVALID_ARG, "gemm: M, N, K must be positive multiples of 4");
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return fail(BT_ERR_INVALID_ARG, "gemm: size too large");
    if (scratch_bytes < bt_op_gemm_split_scratch_bytes()) return fail(BT_ERR_OOM, "gemm: scratch too small");
    if (reinterpret_cast<uintptr_t>(scratch) & 255u) return fail(BT_ERR_INVALID_ARG, "gemm: scratch not 256-byte aligned");
    cudaStream_t s = (cudaStream_t)stream;
    GemmShapes sh = gemm_shapes(layout, M, N, K);
    const int64_t na = sh.a_rows * sh.a_cols, nb = sh.b_rows * sh.b_cols;
    SplitMat Am{A_split, na, sh.a_rows, sh.a_cols, sh.a_cols}, Bm{B_split, nb, sh.b_rows, sh.b_cols, sh.b_cols};
    if (flags & BT_FLAG_GEMM_SIMT) {
        BT_CUDA(launch_gemm_simt(layout, M, N, K, Am, Bm, D, N, bias, residual, s));
        if (act > 2) return fail(BT_ERR_UNSUPPORTED, "gemm: act %d needs the tensor-core kernels", act);
        if (D_act_split) {
            if (act) BT_CUDA(launch_gelu_fwd(D, M * N, act == 2, nullptr, D_act_split, D_act_split + M * N, s));
            else BT_CUDA(launch_split(D, D_act_split, D_act_split + M * N, M * N, s));
        }
        return BT_OK;
    }
    if ((layout == BT_GEMM_TN && M % 32) || (layout != BT_GEMM_NT && N % 32))
        return fail(BT_ERR_UNSUPPORTED, "gemm: transposed operands need their contiguous extent to be a multiple of 32");
    char msg[256];
    if (!gemm_tc_init(msg, sizeof(msg))) return fail(BT_ERR_CUDA, "tensor-core GEMM unavailable: %s", msg);
    float* partials = (float*)scratch;
    int* err = (int*)(partials + gemm_tc_partial_floats_bound());
    BT_CUDA(cudaMemsetAsync(err, 0, sizeof(int), s));
    const int two_cta_mode = (flags & BT_FLAG_GEMM_PAIR) ? 1 : (flags & BT_FLAG_GEMM_SINGLE) ? 0 : -1;
    BT_CUDA(launch_gemm_tc(layout, M, N, K, Am, Bm, D, N, bias, residual, partials, gemm_tc_partial_floats_bound(), err, s,
                           D_act_split, M * N, two_cta_mode, act));
    return BT_OK;
}

extern "C" bt_status bt_op_gemm_split(int32_t layout, int64_t M, int64_t N, int64_t K, const float* A_split,
                                      const float* B_split, float* D, const float* bias, const float* residual,
                                      void* scratch, size_t scratch_bytes, uint32_t flags, void* stream) {
    return gemm_split_impl(layout, M, N, K, A_split, B_split, D, nullptr, 0, bias, residual, scratch, scratch_bytes,
                           flags, stream);
}

extern "C" bt_status bt_op_gemm_split_act(int32_t layout, int64_t M, int64_t N, int64_t K, const float* A_split,
                                          const float* B_split, float* D, float* D_act_split, int32_t act,
                                          const float* bias, const float* residual, void* scratch,
                                          size_t scratch_bytes, uint32_t flags, void* stream) {
    if (!D_act_split) return fail(BT_ERR_INVALID_ARG, "gemm_split_act: D_act_split is NULL");
    return gemm_split_impl(layout, M, N, K, A_split, B_split, D, D_act_split, act, bias, residual, scratch,
                           scratch_bytes, flags, stream);
}

extern "C" size_t bt_op_gemm_gelu_bwd_scratch_bytes(int64_t M, int64_t N) {
    if (M < 1 || N < 1) return 0;
    return bt_op_gemm_split_scratch_bytes() + pad256(((M + 31) / 32) * N) * sizeof(float);
}

extern "C" bt_status bt_op_gemm_gelu_bwd(int64_t M, int64_t N, int64_t K, const float* dy_split, const float* w_split,
                                         const float* h, int32_t form, float* dh_split, float* colsum,
                                         void* scratch, size_t scratch_bytes, uint32_t flags, void* stream) {
    BT_PTR(dy_split); BT_PTR(w_split); BT_PTR(h); BT_PTR(dh_split); BT_PTR(colsum); BT_PTR(scratch);
    if (M < 1 || N < 1 || K < 1 || M % 4 || N % 32 || K % 4) return fail(BT_ERR_INVALID_ARG, "gemm_gelu_bwd: bad sizes");
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return fail(BT_ERR_INVALID_ARG, "gemm_gelu_bwd: size too large");
    if (form < 0 || form > 2) return fail(BT_ERR_INVALID_ARG, "gemm_gelu_bwd: form %d", form);
    if (flags & BT_FLAG_GEMM_SIMT) return fail(BT_ERR_UNSUPPORTED, "gemm_gelu_bwd: tensor-core kernels only");
    if (scratch_bytes < bt_op_gemm_gelu_bwd_scratch_bytes(M, N)) return fail(BT_ERR_OOM, "gemm_gelu_bwd: scratch too small");
    if (reinterpret_cast<uintptr_t>(scratch) & 255u) return fail(BT_ERR_INVALID_ARG, "gemm_gelu_bwd: scratch not 256-byte aligned");
    char msg[256];
    if (!gemm_tc_init(msg, sizeof(msg))) return fail(BT_ERR_CUDA, "tensor-core GEMM unavailable: %s", msg);
    cudaStream_t s = (cudaStream_t)stream;
    float* partials = (float*)scratch;
    int* err = (int*)(partials + gemm_tc_partial_floats_bound());
    float* groups = (float*)((uint8_t*)scratch + bt_op_gemm_split_scratch_bytes());
    BT_CUDA(cudaMemsetAsync(err, 0, sizeof(int), s));
    SplitMat Am{dy_split, M * K, M, K, K}, Bm{w_split, K * N, K, N, N};
    const int two_cta_mode = (flags & BT_FLAG_GEMM_PAIR) ? 1 : (flags & BT_FLAG_GEMM_SINGLE) ? 0 : -1;
    BT_CUDA(launch_gemm_tc(BT_GEMM_NN, M, N, K, Am, Bm, nullptr, N, nullptr, h, partials, gemm_tc_partial_floats_bound(), err,
                           s, dh_split, M * N, two_cta_mode, 5 + form, groups));
    BT_CUDA(launch_colsum_stage2(groups, (int)((M + 31) / 32), (int)N, colsum, s));
    return BT_OK;
}

extern "C" bt_status bt_op_gemm_plan(int64_t M, int64_t N, int64_t K, int32_t epilogue, uint32_t flags, int32_t* out7) {
    if (!out7) return fail(BT_ERR_INVALID_ARG, "gemm_plan: NULL argument");
    if (M < 1 || N < 1 || K < 1) return fail(BT_ERR_INVALID_ARG, "gemm_plan: bad sizes");
    const int two_cta_mode = (flags & BT_FLAG_GEMM_PAIR) ? 1 : (flags & BT_FLAG_GEMM_SINGLE) ? 0 : -1;
    int out[7];
    gemm_tc_plan_info(M, N, K, /*can_split=*/!epilogue, /*can_tail=*/true, two_cta_mode, out);
    for (int i = 0; i < 7; ++i) out7[i] = out[i];
    return BT_OK;
}

extern "C" bt_status bt_op_gemm_check(const void* scratch, void* stream) {
    BT_PTR(scratch);
    const int* err = (const int*)((const float*)scratch + gemm_tc_partial_floats_bound());
    int herr = 0;
    BT_CUDA(cudaMemcpyAsync(&herr, err, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    BT_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    if (herr) return fail(BT_ERR_DEVICE_TIMEOUT, "gemm: a bounded device-side wait ran out (code %d)", herr);
    return BT_OK;
}

extern "C" bt_status bt_op_gemm(int32_t layout, int64_t M, int64_t N, int64_t K, const float* A, const float* B,
                                float* D, const float* bias, const float* residual, void* scratch,
                                size_t scratch_bytes, uint32_t flags, void* stream) {
    BT_PTR(A); BT_PTR(B); BT_PTR(scratch);
    if (layout < 0 || layout > 2) return fail(BT_ERR_INVALID_ARG, "gemm: layout %d", layout);
    if (M < 1 || N < 1 || K < 1 || M % 4 || N % 4 || K % 4) return fail(BT_ERR_INVALID_ARG, "gemm: M, N, K must be positive multiples of 4");
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return fail(BT_ERR_INVALID_ARG, "gemm: size too large");
    if (scratch_bytes < bt_op_gemm_scratch_bytes(layout, M, N, K)) return fail(BT_ERR_OOM, "gemm: scratch too small");
    if (reinterpret_cast<uintptr_t>(scratch) & 255u) return fail(BT_ERR_INVALID_ARG, "gemm: scratch not 256-byte aligned");
    GemmShapes sh = gemm_shapes(layout, M, N, K);
    float* a_s = (float*)scratch;
    float* b_s = a_s + pad256(2 * sh.a_rows * sh.a_cols);
    float* rest = b_s + pad256(2 * sh.b_rows * sh.b_cols);
    bt_status st = bt_op_split(A, sh.a_rows * sh.a_cols, a_s, stream);
    if (st == BT_OK) st = bt_op_split(B, sh.b_rows * sh.b_cols, b_s, stream);
    if (st == BT_OK)
        st = bt_op_gemm_split(layout, M, N, K, a_s, b_s, D, bias, residual, rest, bt_op_gemm_split_scratch_bytes(), flags,
                              stream);
    if (st != BT_OK) return st;
    if (flags & BT_FLAG_GEMM_SIMT) return BT_OK;
    return bt_op_gemm_check(rest, stream);
}

extern "C" bt_status bt_op_attention_fwd(const float* qkv, const float* qkv_split, int32_t B, int32_t T, int32_t C,
                                         int32_t H, float* o, float* o_split, float* lse, uint32_t flags,
                                         void* stream) {
    BT_OPT_PTR(qkv); BT_OPT_PTR(qkv_split); BT_OPT_PTR(o); BT_OPT_PTR(o_split); BT_PTR(lse);
    if (!qkv && !qkv_split) return fail(BT_ERR_INVALID_ARG, "attention_fwd: qkv and qkv_split both NULL");
    if (B < 1 || T < 1 || C < 1 || H < 1 || C % H) return fail(BT_ERR_INVALID_ARG, "attention_fwd: bad sizes");
    int d = C / H;
    if (d != 16 && d != 32 && d != 64 && d != 128) return fail(BT_ERR_UNSUPPORTED, "attention: head_dim %d", d);
    const bool simt = (flags & BT_FLAG_ATTN_SIMT) != 0;
    if (!qkv && (simt || (d != 64 && d != 128)))
        return fail(BT_ERR_INVALID_ARG, "attention_fwd: this kernel needs the raw qkv array");
    int* err = nullptr;
    if (qkv_split && (d == 64 || d == 128) && !simt) {
        char msg[256];
        if (!gemm_tc_init(msg, sizeof(msg))) return fail(BT_ERR_CUDA, "tensor-core attention unavailable: %s", msg);
        BT_CUDA(attention_tc_default_err(&err));
        BT_CUDA(cudaMemsetAsync(err, 0, sizeof(int), (cudaStream_t)stream));
    }
    BT_CUDA(launch_attention_fwd(qkv, qkv_split, (int64_t)B * T * 3 * C, B, T, C, H, o, o_split,
                                 o_split ? o_split + (int64_t)B * T * C : nullptr, lse, simt, err,
                                 (cudaStream_t)stream));
    if (err) {
        int herr = 0;
        BT_CUDA(cudaMemcpyAsync(&herr, err, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
        BT_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
        if (herr) return fail(BT_ERR_DEVICE_TIMEOUT, "attention_fwd: a bounded device-side wait ran out (code %d)", herr);
    }
    return BT_OK;
}

extern "C" bt_status bt_op_attention_bwd(const float* qkv, const float* qkv_split, const float* o, const float* lse,
                                         const float* d_o, const float* d_o_split, int32_t B, int32_t T, int32_t C,
                                         int32_t H, float* dqkv, float* dqkv_split, void* scratch,
                                         size_t scratch_bytes, uint32_t flags, void* stream) {
    BT_OPT_PTR(qkv); BT_OPT_PTR(qkv_split); BT_PTR(o); BT_PTR(lse); BT_OPT_PTR(d_o); BT_OPT_PTR(d_o_split);
    BT_OPT_PTR(dqkv); BT_OPT_PTR(dqkv_split); BT_PTR(scratch);
    if (B < 1 || T < 1 || C < 1 || H < 1 || C % H) return fail(BT_ERR_INVALID_ARG, "attention_bwd: bad sizes");
    int d = C / H;
    if (d != 16 && d != 32 && d != 64 && d != 128) return fail(BT_ERR_UNSUPPORTED, "attention: head_dim %d", d);
    if (scratch_bytes < (size_t)B * H * T * sizeof(float)) return fail(BT_ERR_OOM, "attention_bwd: scratch too small");
    if (!dqkv && !dqkv_split) return fail(BT_ERR_INVALID_ARG, "attention_bwd: no output requested");
    const bool simt = (flags & BT_FLAG_ATTN_SIMT) != 0;
    const bool tc = !simt && qkv_split && d_o_split && dqkv_split && !dqkv && (d == 64 || d == 128);
    if (!tc && (!qkv || !d_o)) return fail(BT_ERR_INVALID_ARG, "attention_bwd: this kernel needs the raw qkv and d_o arrays");
    int* err = nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    if (tc) {
        char msg[256];
        if (!gemm_tc_init(msg, sizeof(msg))) return fail(BT_ERR_CUDA, "tensor-core attention unavailable: %s", msg);
        BT_CUDA(attention_tc_default_err(&err));
        BT_CUDA(cudaMemsetAsync(err, 0, sizeof(int), s));
    }
    const int64_t n = (int64_t)B * T;
    BT_CUDA(launch_attention_bwd(qkv, qkv_split, n * 3 * C, o, nullptr, lse, d_o, d_o_split, n * C, B, T, C, H, dqkv,
                                 dqkv_split, dqkv_split ? dqkv_split + n * 3 * C : nullptr, (float*)scratch, simt, err, s));
    if (err) {
        int herr = 0;
        BT_CUDA(cudaMemcpyAsync(&herr, err, sizeof(int), cudaMemcpyDeviceToHost, s));
        BT_CUDA(cudaStreamSynchronize(s));
        if (herr) return fail(BT_ERR_DEVICE_TIMEOUT, "attention_bwd: a bounded device-side wait ran out (code %d)", herr);
    }
    return BT_OK;
}

extern "C" bt_status bt_op_gelu_fwd(const float* x, int64_t n, int32_t tanh_form, float* y, float* y_split,
                                    void* stream) {
    BT_PTR(x); BT_OPT_PTR(y); BT_OPT_PTR(y_split);
    if (n < 0 || n % 4) return fail(BT_ERR_INVALID_ARG, "gelu_fwd: n must be a non-negative multiple of 4");
    if (n == 0) return BT_OK;
    BT_CUDA(launch_gelu_fwd(x, n, tanh_form, y, y_split, y_split ? y_split + n : nullptr, (cudaStream_t)stream));
    return BT_OK;
}

extern "C" bt_status bt_op_gelu_bwd(const float* x, const float* dy, int64_t n, int32_t tanh_form, float* dx,
                                    float* dx_split, void* stream) {
    BT_PTR(x); BT_PTR(dy); BT_OPT_PTR(dx); BT_OPT_PTR(dx_split);
    if (n < 0 || n % 4) return fail(BT_ERR_INVALID_ARG, "gelu_bwd: n must be a non-negative multiple of 4");
    if (n == 0) return BT_OK;
    BT_CUDA(launch_gelu_bwd(x, dy, n, tanh_form, dx, dx_split, dx_split ? dx_split + n : nullptr, (cudaStream_t)stream));
    return BT_OK;
}

extern "C" bt_status bt_op_gelu_bwd_colsum(const float* x, const float* dy, int64_t N, int32_t C, int32_t tanh_form,
                                           float* dx, float* dx_split, float* colsum, void* scratch,
                                           size_t scratch_bytes, void* stream) {
    BT_PTR(x); BT_PTR(dy); BT_OPT_PTR(dx); BT_OPT_PTR(dx_split); BT_PTR(colsum); BT_PTR(scratch);
    if (N < 1 || C < 4 || C % 4) return fail(BT_ERR_INVALID_ARG, "gelu_bwd_colsum: bad sizes");
    if (scratch_bytes < bt_op_colsum_scratch_bytes(N, C)) return fail(BT_ERR_OOM, "gelu_bwd_colsum: scratch too small");
    BT_CUDA(launch_gelu_bwd_colsum(x, dy, N, C, tanh_form, dx, dx_split, dx_split ? dx_split + N * C : nullptr, colsum,
                                   (float*)scratch, (cudaStream_t)stream));
    return BT_OK;
}

extern "C" bt_status bt_op_softmax_xent(const float* logits, const int32_t* targets, int64_t N, int32_t Vp,
                                        float inv_count, float* losses, float* loss_mean, float* dlogits,
                                        float* dlogits_split, int32_t* d_bad, void* stream) {
    BT_PTR(logits); BT_PTR(targets); BT_PTR(losses); BT_OPT_PTR(dlogits); BT_OPT_PTR(dlogits_split);
    if (N < 1 || Vp < 4 || Vp % 4 || N > (1 << 30)) return fail(BT_ERR_INVALID_ARG, "softmax_xent: bad sizes");
    BT_CUDA(launch_softmax_xent(logits, targets, N, Vp, inv_count, losses, loss_mean, dlogits, dlogits_split,
                                dlogits_split ? dlogits_split + N * Vp : nullptr, Vp, d_bad, (cudaStream_t)stream));
    return BT_OK;
}

extern "C" size_t bt_op_colsum_scratch_bytes(int64_t N, int32_t C) { return colsum_scratch_floats(N, C) * sizeof(float); }

extern "C" bt_status bt_op_colsum(const float* x, int64_t N, int32_t C, float* out, void* scratch, size_t scratch_bytes,
                                  void* stream) {
    BT_PTR(x); BT_PTR(out); BT_PTR(scratch);
    if (N < 1 || C < 4 || C % 4) return fail(BT_ERR_INVALID_ARG, "colsum: bad sizes");
    if (scratch_bytes < bt_op_colsum_scratch_bytes(N, C)) return fail(BT_ERR_OOM, "colsum: scratch too small");
    BT_CUDA(launch_colsum(x, nullptr, N, C, out, (float*)scratch, (cudaStream_t)stream));
    return BT_OK;
}

extern "C" size_t bt_op_grad_norm_scratch_bytes(int64_t n) { return grad_norm_scratch_bytes(n); }

extern "C" bt_status bt_op_grad_norm(const float* g, int64_t n, float clip, float* out2, void* scratch,
                                     size_t scratch_bytes, void* stream) {
    BT_PTR(g); BT_PTR(out2); BT_PTR(scratch);
    if (n < 1) return fail(BT_ERR_INVALID_ARG, "grad_norm: n < 1");
    if (scratch_bytes < grad_norm_scratch_bytes(n)) return fail(BT_ERR_OOM, "grad_norm: scratch too small");
    BT_CUDA(launch_grad_norm(g, n, clip, out2, scratch, (cudaStream_t)stream));
    return BT_OK;
}

namespace bt { int adamw_chunk_elems(); }

extern "C" bt_status bt_op_adamw_multi(int32_t n_tensors, float* const* h_p, const float* const* h_g,
                                       float* const* h_m, float* const* h_v, const int64_t* h_numel,
                                       const int32_t* h_decay, const bt_adamw_config* opt, int64_t t,
                                       const float* d_scale, void* stream) {
    if (!h_p || !h_g || !h_m || !h_v || !h_numel || !h_decay || !opt) return fail(BT_ERR_INVALID_ARG, "adamw_multi: NULL argument");
    if (n_tensors < 0 || n_tensors > AdamTensorList::kMax) return fail(BT_ERR_INVALID_ARG, "adamw_multi: n_tensors not in [0, 64]");
    if (t < 1) return fail(BT_ERR_INVALID_ARG, "adamw_multi: step t must be >= 1");
    if (!(opt->beta1 >= 0.f && opt->beta1 < 1.f) || !(opt->beta2 >= 0.f && opt->beta2 < 1.f) || !(opt->eps > 0.f))
        return fail(BT_ERR_INVALID_ARG, "AdamW: betas must lie in [0,1) and eps must be positive");
    AdamTensorList tl;
    memset(&tl, 0, sizeof(tl));
    tl.n = n_tensors;
    int chunks = 0;
    const int ce = adamw_chunk_elems();
    for (int i = 0; i < n_tensors; ++i) {
        BT_PTR(h_p[i]); BT_PTR(h_g[i]); BT_PTR(h_m[i]); BT_PTR(h_v[i]);
        if (h_numel[i] < 0) return fail(BT_ERR_INVALID_ARG, "adamw_multi: negative numel");
        tl.p[i] = h_p[i]; tl.g[i] = h_g[i]; tl.m[i] = h_m[i]; tl.v[i] = h_v[i];
        tl.numel[i] = h_numel[i]; tl.decay[i] = h_decay[i];
        tl.chunk_begin[i] = chunks;
        chunks += (int)((h_numel[i] + ce - 1) / ce);
    }
    tl.chunk_begin[n_tensors] = chunks;
    AdamParams hp;
    hp.lr = opt->lr; hp.beta1 = opt->beta1; hp.beta2 = opt->beta2; hp.eps = opt->eps; hp.weight_decay = opt->weight_decay;
    hp.inv_c1 = (float)(1.0 / (1.0 - std::pow((double)opt->beta1, (double)t)));
    hp.inv_c2 = (float)(1.0 / (1.0 - std::pow((double)opt->beta2, (double)t)));
    BT_CUDA(launch_adamw_multi(tl, hp, d_scale, (cudaStream_t)stream));
    return BT_OK;
}

// Debug aid (not part of the public header): device buffer of 2 + 2*2000 uint64 that block (0,0)
// of the tcgen05 attention forward kernel fills with (tag, SM clock) records; NULL switches it off.
namespace bt { void attention_tc_set_trace(unsigned long long* p); }
extern "C" __attribute__((visibility("default"))) void bt_debug_set_attention_trace(void* d_buffer) {
    bt::attention_tc_set_trace(static_cast<unsigned long long*>(d_buffer));
}
