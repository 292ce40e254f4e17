// Host side of the C ABI declared in include/xsm.h: argument checks, workspace layout, phase tables,
// launches.  No device memory is allocated here; everything lives in the caller's workspace.
#include "../../include/xsm.h"
#include "xsm_internal.h"

#include <cuda.h>

#include <limits.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <string>
#include <vector>

using namespace xsm;

namespace {

constexpr int kSizingGrid = 256;      // CTA count assumed when sizing split-partial buffers and per-CTA marks
constexpr int kKvStagePositions = 256;
constexpr int kMinSlots = 5;          // ring slots the shared-memory plan keeps at least
constexpr int kChunkSteps = 64;       // decoding steps per persistent-kernel launch in xsm_generate

thread_local std::string g_create_error;

struct Layout {
    size_t total = 0;
    size_t phases, jobs, wkc_off, wvc_off, hk_off, hv_off, tmaps;
    size_t len, window, cand, acc_len, finished, n_gen, n_blocks, ingest_left, step_idx, block_table, free_stack,
        scalars, hist, steps, tok_log, step_tokens, step_n_new, prompt, script;
    size_t h, rope_cs;
    size_t xchg_begin, hpub, qkv, attn, qc, cattn, act, y, logits0, hlogits, part, cpart, candx, header, done, sspub, qh, hattn, gpub,
        hpart, treex, xchg_end;
    size_t stage_cond, stage_kv, stage_tok, trace, ckv_pool, hckv_pool, kv_pool;
    int n_pages = 0, max_blocks = 0, cpages = 0, tok_ld = 0, n_phases = 0, n_jobs = 0;
    size_t page_bytes = 0;
};

size_t esize(const xsm_model_config &c) { return c.dtype == 1 ? 2 : 4; }

size_t take(size_t &cur, size_t bytes) {
    size_t o = cur;
    cur = (cur + bytes + 255) / 256 * 256;
    return o;
}

// workspace_bytes == 0: size the pool for max_batch full sequences
bool make_layout(const xsm_model_config &c, size_t workspace_bytes, Layout &L) {
    const size_t B = c.max_batch, K1 = c.n_draft + 1, M = B * K1, d = c.d_model, V = c.vocab, f = c.d_ff;
    const size_t P = c.page_size, H = c.n_heads, dh = c.d_head;
    L.max_blocks = (int)((c.max_seq_len + K1 + P - 1) / P);
    L.cpages = (int)((c.n_cond + P - 1) / P);
    L.tok_ld = c.max_seq_len + (int)K1;
    const bool ca = c.head_kind == 1 && c.n_draft > 0;
    L.n_phases = c.n_layers * 8 + 3 + (c.n_draft > 0 ? 1 : 0) + (ca ? 2 : 0);
    L.n_jobs = c.n_layers * 6 + 1 + (ca ? 3 : 2) * c.n_draft;
    size_t cur = 0;
    L.phases = take(cur, sizeof(Tables));
    L.jobs = take(cur, 256);
    L.wkc_off = take(cur, sizeof(size_t) * c.n_layers);
    L.wvc_off = take(cur, sizeof(size_t) * c.n_layers);
    L.tmaps = take(cur, 128 * 2 * (size_t)(kLayerJobs + kMaxTailJobs));      // two tensor maps per job
    L.hk_off = take(cur, sizeof(size_t) * (c.n_draft + 1));
    L.hv_off = take(cur, sizeof(size_t) * (c.n_draft + 1));
    L.len = take(cur, 4 * B);
    L.window = take(cur, 4 * M);
    L.cand = take(cur, 4 * M);
    L.acc_len = take(cur, 4 * B);
    L.finished = take(cur, 4 * B);
    L.n_gen = take(cur, 4 * B);
    L.n_blocks = take(cur, 4 * B);
    L.ingest_left = take(cur, 4 * B);
    L.step_idx = take(cur, 4 * B);
    L.block_table = take(cur, 4 * B * L.max_blocks);
    L.scalars = take(cur, 256);   // n_free, n_active, status, bar
    L.hist = take(cur, 8 * B * (kMaxDraft + 1));
    L.steps = take(cur, 8 * B);
    L.tok_log = take(cur, 4 * B * L.tok_ld);
    L.step_tokens = take(cur, 4 * M);
    L.step_n_new = take(cur, 4 * B);
    L.prompt = take(cur, 4 * B * (c.max_seq_len + 1));
    L.script = take(cur, 4 * B * L.tok_ld);
    L.h = take(cur, 4 * M * d);
    L.rope_cs = take(cur, 8 * (size_t)(c.max_seq_len + K1 + 1) * (dh / 2));
    // tagged exchange buffers, cleared together at every xsm_prefill
    L.xchg_begin = cur;
    L.hpub = take(cur, 4 * M * d);
    L.qkv = take(cur, 4 * M * 3 * d);
    L.attn = take(cur, 4 * M * d);
    L.qc = take(cur, 4 * M * d);
    L.cattn = take(cur, 4 * M * d);
    L.act = take(cur, 4 * M * f);
    L.y = take(cur, 4 * M * d * (c.n_draft > 0 ? c.n_draft : 1));
    L.logits0 = take(cur, 4 * M * V);
    L.hlogits = take(cur, 4 * M * V * (c.n_draft > 0 ? c.n_draft : 1));
    const size_t part_items = B * H + kSizingGrid;      // >= B * H * S_max for every batch
    L.part = take(cur, 4 * part_items * K1 * (dh + 2));
    L.cpart = take(cur, 4 * part_items * K1 * (dh + 2));
    L.candx = take(cur, 4 * B * (K1 + 1));
    L.header = take(cur, 4 * B * kHeaderWords);
    L.done = take(cur, 4 * kSizingGrid);
    L.sspub = take(cur, 4 * (size_t)kSizingGrid * M);
    const size_t nh = ca ? (size_t)c.n_draft : 0;       // cross-attention heads: their own exchange buffers
    L.qh = take(cur, 4 * M * d * nh);
    L.hattn = take(cur, 4 * M * d * nh);
    L.gpub = take(cur, 4 * M * d * (ca ? 1 : 0));
    L.hpart = take(cur, 4 * nh * part_items * K1 * (dh + 2));
    L.treex = take(cur, 4 * B * (c.n_draft > 0 ? c.n_draft : 1) * 8 * 2);
    L.xchg_end = cur;
    L.stage_cond = take(cur, esize(c) * B * c.n_cond * c.d_cond);
    L.stage_kv = take(cur, 4 * 2 * (size_t)kKvStagePositions * d);
    L.stage_tok = take(cur, 4 * B * (c.max_seq_len + 1));
    L.trace = take(cur, 8 * (size_t)(1 + 2 * L.n_phases) * kSizingGrid);
    L.ckv_pool = take(cur, esize(c) * (size_t)c.n_layers * 2 * B * L.cpages * H * P * dh);
    L.hckv_pool = take(cur, esize(c) * nh * 2 * B * L.cpages * H * P * dh);
    L.page_bytes = esize(c) * (size_t)c.n_layers * 2 * H * P * dh;
    // the rest is the shared page pool, preceded by its free stack (4 bytes per page)
    if (workspace_bytes == 0) {
        L.n_pages = (int)(B * L.max_blocks);
    } else {
        if (workspace_bytes <= cur) return false;
        size_t n = (workspace_bytes - cur) / (L.page_bytes + 4);   // upper bound; the stack is 256-byte padded
        if (n > (size_t)INT_MAX / 2) n = INT_MAX / 2;
        while (n > 0) {
            size_t c2 = cur;
            take(c2, 4 * n);
            if (c2 + L.page_bytes * n <= workspace_bytes) break;
            --n;
        }
        if (n < (size_t)L.max_blocks) return false;
        L.n_pages = (int)n;
    }
    L.free_stack = take(cur, 4 * (size_t)L.n_pages);
    L.kv_pool = cur;
    L.total = cur + L.page_bytes * L.n_pages;
    return true;
}

const char *check_config(const xsm_model_config &c) {
    if (c.n_layers < 1 || c.d_model < 32 || c.n_heads < 1 || c.d_head < 2 || c.d_ff < 32 || c.vocab < 2 ||
        c.n_cond < 1 || c.d_cond < 32 || c.max_batch < 1 || c.max_seq_len < 1)
        return "a model dimension is out of range";
    if (c.n_heads * c.d_head != c.d_model) return "n_heads * d_head must equal d_model";
    if (c.d_model % 128 || c.d_ff % 128) return "d_model and d_ff must be multiples of 128";
    if (c.d_cond % 32) return "d_cond must be a multiple of 32";
    if ((long long)(c.d_model > c.d_ff ? c.d_model : c.d_ff) * (c.dtype == 1 ? 2 : 4) > 16384)
        return "d_model and d_ff are limited to 16 KB per weight row (8192 bf16 or 4096 fp32 elements)";
    if ((long long)c.d_model * (c.dtype == 1 ? 2 : 4) > 4096)
        return "d_model is limited to 4 KB per weight row (2048 bf16 or 1024 fp32 elements)";
    if (c.d_head != 32 && c.d_head != 64 && c.d_head != 128) return "d_head must be 32, 64 or 128";
    if (c.n_draft < 0 || c.n_draft >= XSM_MAX_DRAFT) return "n_draft must be in [0, 15]";
    if (c.head_hidden != c.d_model) return "head_hidden must equal d_model (the head block is residual)";
    if (c.head_kind != 0 && c.head_kind != 1) return "head_kind must be 0 (MLP heads) or 1 (cross-attention heads)";
    if (c.dtype != 0 && c.dtype != 1) return "dtype must be 0 (fp32) or 1 (bf16)";
    if (c.page_size < 32 || c.page_size % 32) return "page_size must be a positive multiple of 32";
    if ((long long)c.page_size * c.d_head * (c.dtype == 1 ? 2 : 4) > 16384 * (c.dtype == 1 ? 1 : 4))
        return "page_size * d_head is too large for one cache tile";
    if (c.max_batch > kMaxBatch) return "max_batch exceeds 128";
    if ((long long)c.max_batch * (c.n_draft + 1) > kMaxTokens) return "max_batch * (n_draft + 1) exceeds 128";
    if (c.vocab > (1 << 20)) return "vocab too large";
    if (!(c.rope_theta > 1.0f) || !(c.rms_eps > 0.0f)) return "rope_theta must be > 1 and rms_eps > 0";
    if (c.bos_id < 0 || c.bos_id >= c.vocab || c.eos_id >= c.vocab) return "bos_id / eos_id out of range";
    return nullptr;
}

struct WeightOffsets {
    size_t E, gf, W0;
    std::vector<size_t> g1, wq, wo, g2, wqc, wkc, wvc, woc, g3, wgate, wup, wdown, W1, Wout, hq, hk, hv, ho;
    size_t total;
};

WeightOffsets weight_offsets(const xsm_model_config &c) {
    WeightOffsets w;
    const size_t d = c.d_model, f = c.d_ff, V = c.vocab, dc = c.d_cond, hd = c.head_hidden;
    size_t o = 0;
    w.E = o; o += V * d;
    for (int l = 0; l < c.n_layers; ++l) {
        w.g1.push_back(o); o += d;
        w.wq.push_back(o); o += 3 * d * d;      // Wq, Wk, Wv are consecutive
        w.wo.push_back(o); o += d * d;
        w.g2.push_back(o); o += d;
        w.wqc.push_back(o); o += d * d;
        w.wkc.push_back(o); o += d * dc;
        w.wvc.push_back(o); o += d * dc;
        w.woc.push_back(o); o += d * d;
        w.g3.push_back(o); o += d;
        w.wgate.push_back(o); o += f * d;
        w.wup.push_back(o); o += f * d;
        w.wdown.push_back(o); o += d * f;
    }
    w.gf = o; o += d;
    w.W0 = o; o += V * d;
    for (int i = 0; i < c.n_draft; ++i) {
        if (c.head_kind == 1) {          // cross-attention head (Eq. 3): Wq, Wk, Wv, Wo of its own, then W(i)
            w.hq.push_back(o); o += d * d;
            w.hk.push_back(o); o += d * dc;
            w.hv.push_back(o); o += d * dc;
            w.ho.push_back(o); o += d * d;
            w.Wout.push_back(o); o += V * d;
        } else {
            w.W1.push_back(o); o += hd * d;
            w.Wout.push_back(o); o += V * hd;
        }
    }
    w.total = o;
    return w;
}

}  // namespace

struct xsm_ctx {
    xsm_model_config cfg;
    xsm_decode_config dc;
    Layout lay;
    WeightOffsets wo;
    const char *weights;
    char *ws;
    size_t ws_bytes;
    cudaStream_t stream;
    Dev dev;
    int grid, sm_count, smem_bytes, phase_launch, prefilled, batch;
    uint32_t serial;          // decoding steps launched since the last xsm_prefill
    int static_steps;         // the latest step kept its attention partials in the library's own scratch array
    uint64_t launches;
    std::string err;
    Tables h_tab;
    std::vector<CUtensorMap> h_tmaps;   // tcgen05 path: host copies of the jobs' tensor maps (uploaded by xsm_prefill)
    int n_stages;             // stages of one decoding step
    void *encode_tiled;       // cuTensorMapEncodeTiled of the driver (null: the tcgen05 path is not used)
    int *pinned;              // [4] n_active, status
    cudaEvent_t ev0, ev1;
    double last_wall_ms;
};

namespace {

xsm_status fail(xsm_ctx *ctx, xsm_status st, const std::string &msg) {
    if (ctx) ctx->err = msg; else g_create_error = msg;
    return st;
}
xsm_status cuda_fail(xsm_ctx *ctx, cudaError_t e, const char *what) {
    return fail(ctx, XSM_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
#define XSM_CUDA(ctx, call)                                             \
    do {                                                                \
        cudaError_t e_ = (call);                                        \
        if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #call);        \
    } while (0)

template <typename T> T *at(xsm_ctx *ctx, size_t off) { return reinterpret_cast<T *>(ctx->ws + off); }
const void *wptr(const xsm_ctx *ctx, size_t elem_off) { return ctx->weights + elem_off * esize(ctx->cfg); }

// Shared memory of the step kernel for a batch of `batch` sequences: header, ring slots, activation area
// (also the scratch of attention, verification and the cross-warp reduction), sums of squares.
// Returns nullptr or the reason why the shape cannot run.
// do the projections of this batch run on the tcgen05 path?
bool umma_shape(const xsm_model_config &c, int batch) {
    const int M = batch * (c.n_draft + 1);
    // (measured: below about 27 token rows the mma.sync paths are faster; the tensor-core path pays a fixed cost per
    // block of 64 columns that only a well-filled tile repays)
    return c.dtype == 1 && M >= kUmmaMinRows && M <= 128 && c.d_model % kUmmaK == 0 && c.d_ff % kUmmaK == 0;
}

// jobs in the tail of a step: the LM head, then per decoding head W1 and Wout, or Wq, Wo and Wout
int tail_jobs(const xsm_model_config &c) { return 1 + (c.head_kind == 1 ? 3 : 2) * c.n_draft; }

// grid: CTAs of the step kernel if known (it sizes the staging of the sums-of-squares shares on the path for at most
// eight token rows), 0: not known yet, plan for the largest
const char *plan_smem(const xsm_model_config &c, int batch, Dev &D, int &smem_bytes, int grid = 0) {
    const int K1 = c.n_draft + 1, M = batch * K1, dh = c.d_head;
    D.tab_bytes = smem_tab_bytes(tail_jobs(c));
    D.plan_bytes = smem_plan_bytes(tail_jobs(c));
    if (D.umma)      // swizzled tensor-core tiles: the ring starts on a 1024-byte boundary
        D.plan_bytes = (kSmemHeader + D.tab_bytes + D.plan_bytes + 1023) / 1024 * 1024 - kSmemHeader - D.tab_bytes;
    const int kSmemTables = D.tab_bytes, kSmemPlans = D.plan_bytes;
    if (D.umma) {
        // tcgen05 path: the activation area holds two buffers of two planes (hi, lo) of 128 token rows x 64 columns; the
        // other users of the area (attention, verification, commit) fit inside
        const int tail = (kMaxTokens + 1536) * 4;
        const int avail = kSmemMax - kSmemHeader - kSmemTables - kSmemPlans - tail;
        int need = 2 * 16 * (dh + 8) * 2 + 4 * K1 * dh * 4 + 128 * dh + (kConsumerWarps + 1) * K1 * (dh + 2) * 4;
        const int samp = (((c.vocab + 3) & ~3) + 1024) * 4;
        if (samp > need) need = samp;
        const int emb = 512 + K1 * (c.d_model / 8) * 4;
        if (emb > need) need = emb;
        int acts = kUmmaActsBytes > need ? kUmmaActsBytes : (need + 1023) / 1024 * 1024;
        int slots = (avail - acts) / kSlotBytes;
        if (slots > kMaxSlots) slots = kMaxSlots;
        if (slots < kMinSlots) return "the shape needs more shared memory than one CTA has";
        D.n_slots = slots;
        D.acts_bytes = acts;
        D.kca = c.d_model > c.d_ff ? c.d_model : c.d_ff;
        D.tile_bytes = c.page_size * dh * 2;
        D.kv_one_item = 2 * D.tile_bytes <= kSlotBytes ? 1 : 0;
        smem_bytes = kSmemHeader + kSmemTables + kSmemPlans + slots * kSlotBytes + acts + tail;
        return nullptr;
    }
    const int kmax = c.d_model > c.d_ff ? c.d_model : c.d_ff;
    // sums of squares and their partials; at most eight token rows of a bf16 model: the CTAs' shares [row][CTA]
    int tail = (kMaxTokens + 1536) * 4;
    if (grid > 0 && c.dtype == 1 && M <= 8 && grid * M <= 1536) tail = (kMaxTokens + ((grid * M + 31) & ~31)) * 4;
    const int avail = kSmemMax - kSmemHeader - kSmemTables - kSmemPlans - tail;
    // what the other users of the activation area need
    const int np = c.dtype == 1 ? (M <= 8 ? 8 : M <= 16 ? 16 : M <= 32 ? 32 : M <= 80 ? 80 : 128) : 8;
    int need = kConsumerWarps * np * 16 * 4 + 2 * 16 * M * 4;         // reduction of the projections, new residual values
    const int attn = 2 * 16 * (dh + 8) * 2 + 4 * K1 * dh * 4 + 128 * dh + (kConsumerWarps + 1) * K1 * (dh + 2) * 4;
    if (attn > need) need = attn;
    const int samp = (((c.vocab + 3) & ~3) + 1024) * 4;      // a logits row, reduction scratch, candidates, the probability tree's tables
    if (samp > need) need = samp;
    const int emb = 512 + K1 * (c.d_model / (c.dtype == 1 ? 8 : 4)) * 4;   // commit: scalars, partial sums of the new window's rows
    if (emb > need) need = emb;
    const int full = M * (kmax * 4 + 16) + (kConsumerWarps * np * 16 + kConsumerWarps * M) * 4;   // all activations of the widest projection, and the partial products behind them
    int acts = full > need ? full : need;
    if (acts > avail - kMinSlots * kSlotBytes) acts = avail - kMinSlots * kSlotBytes;
    if (acts < need) return "the shape needs more shared memory than one CTA has";
    acts = (acts + 127) / 128 * 128;
    if (acts > avail - kMinSlots * kSlotBytes) acts -= 128;
    int kca = ((acts / M - 16) / 4) / 128 * 128;
    if (kca > kmax) kca = kmax;
    if (kca < kmax && c.dtype == 1) {
        // the widest projection is staged in chunks: room for the accumulators and the per-token partial sums behind
        // a chunk, and chunks of at most 2048 columns (four rows of a chunk fit one ring slot)
        kca = (((acts - kAccumBytes - kAccumBytes / 16) / M - 16) / 4) / 128 * 128;
        if (kca > 2048) kca = 2048;
    }
    if (kca < 128) return "batch * (n_draft + 1) is too large for the activation staging area";
    if (c.dtype == 0 && kca < kmax) return "fp32 models need all activations of a projection in shared memory: reduce the batch";
    if (c.dtype == 0 && M > 24) return "fp32 models support at most 24 token rows per step";
    int slots = (avail - acts) / kSlotBytes;
    if (slots > kMaxSlots) slots = kMaxSlots;
    D.n_slots = slots;
    D.acts_bytes = acts;
    D.kca = kca;
    D.tile_bytes = c.page_size * dh * (c.dtype == 1 ? 2 : 4);
    D.kv_one_item = 2 * D.tile_bytes <= kSlotBytes ? 1 : 0;
    smem_bytes = kSmemHeader + kSmemTables + kSmemPlans + slots * kSlotBytes + acts + tail;
    return nullptr;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of a bf16 weight matrix [layers][rows][kdim] (rows of kdim elements, layers layer_bytes apart): boxes of 64
// columns x 8 rows of one layer, 128-byte swizzle (the layout the tcgen05 matrix descriptors of the step kernel name).
bool encode_weight_map(xsm_ctx *ctx, CUtensorMap *out, const void *W, int rows, int kdim, int layers, long long layer_bytes) {
    if (!ctx->encode_tiled || !W) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kdim, (cuuint64_t)rows, (cuuint64_t)(layers > 0 ? layers : 1)};
    cuuint64_t strides[2] = {(cuuint64_t)kdim * 2, (cuuint64_t)(layers > 1 ? layer_bytes : (long long)rows * kdim * 2)};
    cuuint32_t box[3] = {(cuuint32_t)kUmmaK, 8, 1}, estr[3] = {1, 1, 1};
    return ((EncodeTiledFn)ctx->encode_tiled)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(W), dims, strides, box, estr,
                                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// stage and job tables for the current batch: the eight stages of layer 0, then the tail of the step
void build_tables(xsm_ctx *ctx) {
    const xsm_model_config &c = ctx->cfg;
    const Dev &D = ctx->dev;
    const WeightOffsets &w = ctx->wo;
    const int d = c.d_model, f = c.d_ff, V = c.vocab, K = c.n_draft, L = c.n_layers;
    const size_t M = D.M;
    const int hw = 3 * L + 1;      // writes of the residual stream per step: the embedding and three per layer
    Tables &T = ctx->h_tab;
    memset(&T, 0, sizeof(T));
    T.layer_bytes = L > 1 ? (long long)((w.wq[1] - w.wq[0]) * esize(c)) : 0;
    T.gain_last = wptr(ctx, w.gf);
    int n_jobs = 0, n_stages = 0;
    auto job = [&](const void *W, const void *W2, int rows, int kdim, const float *x, const void *gain, float *out,
                   int out_ld, int epi, TagRef in, int in_jinc, TagRef outt, int out_jinc, const void *gain_out = nullptr,
                   int out_plain = 0) -> GemvJob & {
        GemvJob &j = T.jobs[n_jobs++];
        j.W = W; j.W2 = W2; j.x = x; j.gain = gain; j.out = out; j.hm = epi == EPI_ADD ? D.h : nullptr;
        j.rows = rows; j.kdim = kdim; j.out_ld = out_ld; j.epi = epi; j.in = in; j.outt = outt;
        j.in_jinc = in_jinc; j.out_jinc = out_jinc; j.gain_out = gain_out; j.out_plain = out_plain;
        return j;
    };
    auto gemv1 = [&](int j0, int n) {
        Stage &s = T.stages[n_stages++];
        s.kind = ST_GEMV; s.job0 = j0; s.njobs = n;
    };
    auto attn = [&](int kind) {
        Stage &s = T.stages[n_stages++];
        s.kind = kind;
        s.in = TagRef{L, 0}; s.outt = TagRef{L, 0}; s.part = TagRef{L, 0}; s.jinc = 1;
    };
    // layer 0.  Buffers written once per layer have write index serial * L + l, the residual stream 3 l + which.
    // A stage that adds to the residual stream publishes it with the gain of the RMSNorm that reads it next.
    const TagRef per_layer{L, 0};
    job(wptr(ctx, w.wq[0]), nullptr, 3 * d, d, D.hpub, wptr(ctx, w.g1[0]), D.qkv, 3 * d, EPI_STORE, TagRef{hw, 0}, 3, per_layer, 1);
    gemv1(0, 1);
    attn(ST_ATTN_SELF);
    job(wptr(ctx, w.wo[0]), nullptr, d, d, D.attn, nullptr, D.hpub, d, EPI_ADD, per_layer, 1, TagRef{hw, 1}, 3, wptr(ctx, w.g2[0]));
    gemv1(1, 1);
    job(wptr(ctx, w.wqc[0]), nullptr, d, d, D.hpub, wptr(ctx, w.g2[0]), D.qc, d, EPI_STORE, TagRef{hw, 1}, 3, per_layer, 1);
    gemv1(2, 1);
    attn(ST_ATTN_CROSS);
    job(wptr(ctx, w.woc[0]), nullptr, d, d, D.cattn, nullptr, D.hpub, d, EPI_ADD, per_layer, 1, TagRef{hw, 2}, 3, wptr(ctx, w.g3[0]));
    gemv1(3, 1);
    job(wptr(ctx, w.wgate[0]), wptr(ctx, w.wup[0]), f, d, D.hpub, wptr(ctx, w.g3[0]), D.act, f, EPI_GATEUP, TagRef{hw, 2}, 3,
        per_layer, 1);
    gemv1(4, 1);
    {   // the down projection's published copy is read through the first RMSNorm of the NEXT layer (or the final one)
        GemvJob &j = job(wptr(ctx, w.wdown[0]), nullptr, d, f, D.act, nullptr, D.hpub, d, EPI_ADD, per_layer, 1, TagRef{hw, 3}, 3,
                         wptr(ctx, w.g1[0]));
        j.gain_out_step = T.layer_bytes != 0 ? T.layer_bytes : 1;
        gemv1(5, 1);
    }
    // tail
    const TagRef once{1, 0};
    int j0 = n_jobs;
    job(wptr(ctx, w.W0), nullptr, V, d, D.hpub, wptr(ctx, w.gf), D.logits0, V, EPI_STORE, TagRef{hw, 3 * L}, 0, once, 0, nullptr, 1);
    if (c.head_kind == 1 && K > 0) {
        // cross-attention heads (Eq. 3): q = Wq g beside the LM head (every CTA also publishes its columns of g), the
        // heads' attention over their own keys and values of the condition, y = g + Wo a
        for (int i = 0; i < K; ++i)
            job(wptr(ctx, w.hq[i]), nullptr, d, d, D.hpub, wptr(ctx, w.gf), D.qh + (size_t)i * M * d, d, EPI_STORE, TagRef{hw, 3 * L}, 0, once, 0);
        gemv1(j0, 1 + K);
        T.stages[n_stages - 1].norm_out = 1;
        {
            Stage &s = T.stages[n_stages++];
            s.kind = ST_ATTN_HEAD;
            s.in = once; s.outt = once; s.part = once; s.jinc = 0;
        }
        j0 = n_jobs;
        for (int i = 0; i < K; ++i)
            job(wptr(ctx, w.ho[i]), nullptr, d, d, D.hattn + (size_t)i * M * d, nullptr, D.y + (size_t)i * M * d, d, EPI_ADDG, once, 0, once, 0)
                .res = D.gpub;
        gemv1(j0, K);
    } else {
        for (int i = 0; i < K; ++i)
            job(wptr(ctx, w.W1[i]), nullptr, d, d, D.hpub, wptr(ctx, w.gf), D.y + (size_t)i * M * d, d, EPI_HEADY,
                TagRef{hw, 3 * L}, 0, once, 0);
        gemv1(j0, 1 + K);
    }
    if (K > 0) {
        j0 = n_jobs;
        for (int i = 0; i < K; ++i)
            job(wptr(ctx, w.Wout[i]), nullptr, V, d, D.y + (size_t)i * M * d, nullptr, D.hlogits + (size_t)i * M * V, V,
                EPI_STORE, once, 0, once, 0, nullptr, 1);
        gemv1(j0, K);
    }
    T.stages[n_stages++].kind = ST_SAMPLE;
    T.stages[n_stages++].kind = ST_COMMIT;
    T.n_tail_stages = n_stages - kLayerStages;
    T.n_tail_jobs = n_jobs - kLayerJobs;
    ctx->n_stages = kLayerStages * L + T.n_tail_stages;
    if (ctx->dev.umma) {
        // tcgen05 path: the weights come by TMA; one tensor map per matrix (all layers of a layer job in one map)
        ctx->h_tmaps.assign(2 * (size_t)n_jobs, CUtensorMap{});
        char *d_maps = ctx->ws + ctx->lay.tmaps;
        bool ok = true;
        for (int i = 0; i < n_jobs && ok; ++i) {
            GemvJob &j = T.jobs[i];
            const int layers = i < kLayerJobs ? L : 1;
            ok = encode_weight_map(ctx, &ctx->h_tmaps[2 * i], j.W, j.rows, j.kdim, layers, T.layer_bytes);
            j.tmap = d_maps + 128 * (2 * (size_t)i);
            if (ok && j.W2 != nullptr) {
                ok = encode_weight_map(ctx, &ctx->h_tmaps[2 * i + 1], j.W2, j.rows, j.kdim, layers, T.layer_bytes);
                j.tmap2 = d_maps + 128 * (2 * (size_t)i + 1);
            }
        }
        if (!ok) {        // no tensor maps: the projections take the mma.sync path
            ctx->dev.umma = 0;
            for (int i = 0; i < n_jobs; ++i) T.jobs[i].tmap = T.jobs[i].tmap2 = nullptr;
        }
    }
}

xsm_status check_device_status(xsm_ctx *ctx) {
    XSM_CUDA(ctx, cudaMemcpyAsync(ctx->pinned, ctx->dev.n_active, 8, cudaMemcpyDeviceToHost, ctx->stream));
    XSM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    const int st = ctx->pinned[1];
    if (st == XSM_ERR_TIMEOUT) return fail(ctx, XSM_ERR_TIMEOUT, "a bounded device-side wait ran out of patience");
    if (st == XSM_ERR_CAPACITY) return fail(ctx, XSM_ERR_CAPACITY, "the page pool ran dry during decoding");
    if (st != 0) return fail(ctx, XSM_ERR_CUDA, "device status word is set");
    return XSM_OK;
}

// n_steps decoding steps on the stream
xsm_status run_steps(xsm_ctx *ctx, int n_steps, bool static_scratch = false) {
    const int np = ctx->n_stages;
    if (!static_scratch && ctx->static_steps) {
        // The steps since the workspace partials were last written went through the library's scratch array, so the
        // workspace copy still carries the tags of an older step; tags repeat with period three, and a stale word
        // could pass for a fresh partial.  It restarts from "never written".
        XSM_CUDA(ctx, cudaMemsetAsync(ctx->ws + ctx->lay.part, 0, ctx->lay.candx - ctx->lay.part, ctx->stream));
        if (ctx->lay.xchg_end > ctx->lay.hpart)
            XSM_CUDA(ctx, cudaMemsetAsync(ctx->ws + ctx->lay.hpart, 0, ctx->lay.xchg_end - ctx->lay.hpart, ctx->stream));
    }
    ctx->static_steps = static_scratch ? 1 : 0;
    if (!ctx->phase_launch) {
        XSM_CUDA(ctx, launch_step(ctx->dev, ctx->cfg.dtype, 0, np, n_steps, ctx->serial, ctx->grid, ctx->smem_bytes, ctx->stream));
        ctx->launches += 1;
        ctx->serial += (uint32_t)n_steps;
    } else {
        for (int t = 0; t < n_steps; ++t) {
            for (int p = 0; p < np; ++p) {
                XSM_CUDA(ctx, launch_step(ctx->dev, ctx->cfg.dtype, p, p + 1, 1, ctx->serial, ctx->grid, ctx->smem_bytes, ctx->stream));
                ctx->launches += 1;
            }
            ctx->serial += 1u;
        }
    }
    return XSM_OK;
}

}  // namespace

extern "C" {

size_t xsm_weights_bytes(const xsm_model_config *cfg) {
    if (!cfg || check_config(*cfg)) return 0;
    return weight_offsets(*cfg).total * esize(*cfg);
}

size_t xsm_workspace_bytes(const xsm_model_config *cfg) {
    if (!cfg || check_config(*cfg)) return 0;
    Layout L;
    make_layout(*cfg, 0, L);
    return L.total;
}

xsm_status xsm_create(const xsm_model_config *cfg, const void *d_weights, void *d_workspace, size_t workspace_bytes,
                      void *cuda_stream, xsm_ctx **out) {
    if (!cfg || !d_weights || !d_workspace || !out) return fail(nullptr, XSM_ERR_INVALID_ARG, "null argument");
    if (const char *m = check_config(*cfg)) return fail(nullptr, XSM_ERR_INVALID_ARG, m);
    if (((uintptr_t)d_weights & 255) || ((uintptr_t)d_workspace & 255))
        return fail(nullptr, XSM_ERR_INVALID_ARG, "weights and workspace must be 256-byte aligned");
    Layout L;
    if (!make_layout(*cfg, workspace_bytes, L))
        return fail(nullptr, XSM_ERR_CAPACITY, "workspace cannot hold the buffers plus one sequence of cache pages");
    Dev probe;
    memset(&probe, 0, sizeof(probe));
    int smem_one = 0;
    if (const char *m = plan_smem(*cfg, 1, probe, smem_one)) return fail(nullptr, XSM_ERR_INVALID_ARG, m);
    xsm_ctx *ctx = new xsm_ctx();
    ctx->cfg = *cfg;
    ctx->lay = L;
    ctx->wo = weight_offsets(*cfg);
    ctx->weights = (const char *)d_weights;
    ctx->ws = (char *)d_workspace;
    ctx->ws_bytes = workspace_bytes;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->phase_launch = 0; ctx->prefilled = 0; ctx->batch = 0; ctx->launches = 0; ctx->last_wall_ms = 0; ctx->serial = 0;
    ctx->static_steps = 0;
    ctx->pinned = nullptr; ctx->ev0 = ctx->ev1 = nullptr;
    auto bail = [&](cudaError_t e, const char *what) {
        g_create_error = std::string(what) + ": " + cudaGetErrorString(e);
        if (ctx->pinned) cudaFreeHost(ctx->pinned);
        if (ctx->ev0) cudaEventDestroy(ctx->ev0);
        if (ctx->ev1) cudaEventDestroy(ctx->ev1);
        delete ctx;
        return XSM_ERR_CUDA;
    };
    cudaError_t e;
    int grid = 0;
    {
        int dev = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return bail(e, "cudaGetDevice");
        if ((e = cudaDeviceGetAttribute(&grid, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return bail(e, "device query");
    }
    if (grid < 1) { delete ctx; return fail(nullptr, XSM_ERR_CUDA, "no multiprocessors reported"); }
    ctx->sm_count = grid;
    // every CTA must own at least one row of every projection (the exchange protocol relies on it), and the
    // buffers that are sized per CTA bound the grid from above
    if (grid > cfg->d_model) grid = cfg->d_model;
    if (grid > kSizingGrid) grid = kSizingGrid;
    ctx->grid = grid;
    if ((e = cudaHostAlloc((void **)&ctx->pinned, 64, cudaHostAllocDefault)) != cudaSuccess) return bail(e, "cudaHostAlloc");
    {   // the driver's tensor-map encoder, for the weights of the tcgen05 projections (absent: those take the mma.sync path)
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        ctx->encode_tiled = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            ctx->encode_tiled = fn;
        else
            (void)cudaGetLastError();
    }
    if ((e = cudaEventCreate(&ctx->ev0)) != cudaSuccess) return bail(e, "cudaEventCreate");
    if ((e = cudaEventCreate(&ctx->ev1)) != cudaSuccess) return bail(e, "cudaEventCreate");

    // constant tables
    // cos and sin of position * theta^(-2i/dh) for every position a window row can take
    const int half = cfg->d_head / 2, n_pos = cfg->max_seq_len + cfg->n_draft + 2;
    std::vector<float> rope((size_t)n_pos * half * 2);
    for (int i = 0; i < half; ++i) {
        const double inv_freq = pow((double)cfg->rope_theta, -2.0 * i / cfg->d_head);
        for (int p = 0; p < n_pos; ++p) {
            rope[((size_t)p * half + i) * 2] = (float)cos((double)p * inv_freq);
            rope[((size_t)p * half + i) * 2 + 1] = (float)sin((double)p * inv_freq);
        }
    }
    if ((e = cudaMemcpyAsync(ctx->ws + L.rope_cs, rope.data(), sizeof(float) * rope.size(),
                             cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess) return bail(e, "upload");
    if ((e = cudaMemcpyAsync(ctx->ws + L.wkc_off, ctx->wo.wkc.data(), sizeof(size_t) * cfg->n_layers,
                             cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess) return bail(e, "upload");
    if ((e = cudaMemcpyAsync(ctx->ws + L.wvc_off, ctx->wo.wvc.data(), sizeof(size_t) * cfg->n_layers,
                             cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess) return bail(e, "upload");
    if (cfg->head_kind == 1 && cfg->n_draft > 0) {
        if ((e = cudaMemcpyAsync(ctx->ws + L.hk_off, ctx->wo.hk.data(), sizeof(size_t) * cfg->n_draft, cudaMemcpyHostToDevice,
                                 ctx->stream)) != cudaSuccess) return bail(e, "upload");
        if ((e = cudaMemcpyAsync(ctx->ws + L.hv_off, ctx->wo.hv.data(), sizeof(size_t) * cfg->n_draft, cudaMemcpyHostToDevice,
                                 ctx->stream)) != cudaSuccess) return bail(e, "upload");
    }
    // the caches start at zero: slots that were never written are multiplied by zero weights and must be finite
    if ((e = cudaMemsetAsync(ctx->ws + L.ckv_pool, 0, L.total - L.ckv_pool, ctx->stream)) != cudaSuccess) return bail(e, "memset");
    if ((e = cudaStreamSynchronize(ctx->stream)) != cudaSuccess) return bail(e, "sync");

    Dev &D = ctx->dev;
    memset(&D, 0, sizeof(D));
    D.L = cfg->n_layers; D.d = cfg->d_model; D.H = cfg->n_heads; D.dh = cfg->d_head; D.f = cfg->d_ff;
    D.V = cfg->vocab; D.C = cfg->n_cond; D.dc = cfg->d_cond; D.K = cfg->n_draft; D.K1 = cfg->n_draft + 1;
    D.P = cfg->page_size; D.max_blocks = L.max_blocks; D.n_pages = L.n_pages; D.cpages = L.cpages;
    D.p_shift = -1;
    for (int sh = 0; sh < 30; ++sh)
        if ((1 << sh) == cfg->page_size) D.p_shift = sh;
    D.max_seq_len = cfg->max_seq_len; D.tok_ld = L.tok_ld;
    D.eps = cfg->rms_eps; D.scale = (float)(1.0 / sqrt((double)cfg->d_head)); D.bos = cfg->bos_id; D.eos = cfg->eos_id;
    D.max_new = INT_MAX;
    D.spin_limit = kSpinLimit; D.mbar_limit = kMbarSpinLimit;
    D.tables = at<Tables>(ctx, L.phases);
    D.E = wptr(ctx, ctx->wo.E);
    D.len = at<int>(ctx, L.len); D.window = at<int>(ctx, L.window); D.cand = at<int>(ctx, L.cand);
    D.acc_len = at<int>(ctx, L.acc_len); D.finished = at<int>(ctx, L.finished); D.n_gen = at<int>(ctx, L.n_gen);
    D.n_blocks = at<int>(ctx, L.n_blocks); D.block_table = at<int>(ctx, L.block_table);
    D.ingest_left = at<int>(ctx, L.ingest_left); D.step_idx = at<uint32_t>(ctx, L.step_idx);
    D.free_stack = at<int>(ctx, L.free_stack);
    int *sc = at<int>(ctx, L.scalars);
    D.n_active = sc; D.status = sc + 1; D.n_free = sc + 2;
    D.hist = at<unsigned long long>(ctx, L.hist); D.steps = at<unsigned long long>(ctx, L.steps);
    D.tok_log = at<int>(ctx, L.tok_log); D.step_tokens = at<int>(ctx, L.step_tokens);
    D.step_n_new = at<int>(ctx, L.step_n_new); D.prompt = at<int>(ctx, L.prompt);
    D.h = at<float>(ctx, L.h); D.rope_cs = at<float2>(ctx, L.rope_cs);
    D.hpub = at<float>(ctx, L.hpub); D.qkv = at<float>(ctx, L.qkv); D.attn = at<float>(ctx, L.attn);
    D.qc = at<float>(ctx, L.qc); D.cattn = at<float>(ctx, L.cattn); D.act = at<float>(ctx, L.act);
    D.y = at<float>(ctx, L.y); D.logits0 = at<float>(ctx, L.logits0); D.hlogits = at<float>(ctx, L.hlogits);
    D.part = at<float>(ctx, L.part); D.cpart = at<float>(ctx, L.cpart);
    D.candx = at<uint32_t>(ctx, L.candx); D.header = at<uint32_t>(ctx, L.header); D.done = at<uint32_t>(ctx, L.done);
    D.sspub = at<float>(ctx, L.sspub); D.gain_first = wptr(ctx, ctx->wo.g1[0]); D.grid = grid;
    D.kv_pool = ctx->ws + L.kv_pool; D.ckv_pool = ctx->ws + L.ckv_pool;
    D.head_kind = cfg->head_kind;
    D.qh = at<float>(ctx, L.qh); D.hattn = at<float>(ctx, L.hattn); D.gpub = at<float>(ctx, L.gpub); D.hpart = at<float>(ctx, L.hpart);
    D.hckv_pool = ctx->ws + L.hckv_pool;
    D.treex = at<uint32_t>(ctx, L.treex);
    *out = ctx;
    return XSM_OK;
}

xsm_status xsm_prefill(xsm_ctx *ctx, int batch, const void *d_cond, const int32_t *d_prompt, int prompt_len,
                       const xsm_decode_config *dc) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!d_cond || !d_prompt || !dc) return fail(ctx, XSM_ERR_INVALID_ARG, "null argument");
    const xsm_model_config &c = ctx->cfg;
    if (batch < 1 || batch > c.max_batch) return fail(ctx, XSM_ERR_INVALID_ARG, "batch must be in [1, max_batch]");
    if (prompt_len < 1 || prompt_len - 1 > c.max_seq_len) return fail(ctx, XSM_ERR_INVALID_ARG, "prompt_len out of range");
    if (dc->verify_mode < 0 || dc->verify_mode > 2 || dc->sample_mode < 0 || dc->sample_mode > 2)
        return fail(ctx, XSM_ERR_INVALID_ARG, "unknown verify_mode or sample_mode");
    if (dc->verify_mode == 1 && dc->k_accept < 1) return fail(ctx, XSM_ERR_INVALID_ARG, "k_accept must be >= 1");
    if (dc->sample_mode == 1 && (dc->k_sample < 1 || dc->k_sample > 64 || !(dc->temperature > 0.f)))
        return fail(ctx, XSM_ERR_INVALID_ARG, "k_sample must be in [1, 64] and temperature > 0");
    if (dc->sample_mode == 2) {
        if (dc->k_sample < 1 || dc->k_sample > 8 || !(dc->temperature > 0.f))
            return fail(ctx, XSM_ERR_INVALID_ARG, "probability-tree sampling: k_sample must be in [1, 8] and temperature > 0");
        double leaves = 1.0;
        for (int i = 0; i < c.n_draft; ++i) leaves *= dc->k_sample;
        if (leaves > 4096.0) return fail(ctx, XSM_ERR_INVALID_ARG, "probability-tree sampling: k_sample ^ n_draft must not exceed 4096 paths");
    }
    if ((long long)batch * ctx->lay.max_blocks > ctx->lay.n_pages)
        return fail(ctx, XSM_ERR_CAPACITY, "the page pool cannot hold `batch` sequences of max_seq_len positions");
    Dev &D = ctx->dev;
    int smem_bytes = 0;
    D.umma = (umma_shape(c, batch) && ctx->encode_tiled != nullptr) ? 1 : 0;
    if (const char *m = plan_smem(c, batch, D, smem_bytes, ctx->grid)) return fail(ctx, XSM_ERR_CAPACITY, m);
    {   // at most eight token rows, all activations of the widest projection staged at once with room for the warps'
        // partial products behind them, the CTAs' shares of a row readable by one warp pass: the compact instance
        const int M = batch * D.K1, kmax = c.d_model > c.d_ff ? c.d_model : c.d_ff;
        D.small = (c.dtype == 1 && M <= 8 && D.kca >= kmax && ctx->grid * M <= 1536 && (ctx->grid & 3) == 0 &&
                   D.acts_bytes - M * (kmax * 4 + 16) >= kConsumerWarps * kSmallRedBytes) ? 1 : 0;
        // (the other paths stage their partial sums of squares in the full-size area)
        if (!D.small)
            if (const char *m = plan_smem(c, batch, D, smem_bytes)) return fail(ctx, XSM_ERR_CAPACITY, m);
    }
    ctx->smem_bytes = smem_bytes;
    {   // the step kernel instance for this batch must fit one CTA per multiprocessor
        Dev probe = D;
        probe.M = batch * D.K1;
        int resident = 0;
        XSM_CUDA(ctx, step_kernel_setup(probe, c.dtype, smem_bytes, &resident));
        if (resident < ctx->grid) return fail(ctx, XSM_ERR_CUDA, "the step kernel does not fit on this device");
    }
    ctx->dc = *dc;
    ctx->batch = batch;
    D.B = batch; D.M = batch * D.K1;
    D.inv_m = ((1 << 20) + D.M - 1) / D.M;
    D.verify_mode = dc->verify_mode; D.k_accept = dc->k_accept; D.delta = dc->delta;
    D.sample_mode = dc->sample_mode; D.k_sample = dc->k_sample; D.temperature = dc->temperature;
    D.key0 = (uint32_t)dc->seed; D.key1 = (uint32_t)(dc->seed >> 32);
    D.max_new = INT_MAX; D.prompt_len = prompt_len;
    const int bh = batch * D.H;
    int s_max = ctx->grid / bh;
    D.S_max = s_max < 1 ? 1 : (s_max > 64 ? 64 : s_max);
    // the condition's keys and values of one head: one item while that is at most 96 KB, else split over CTAs
    int s_cross = 1;
    if ((long long)D.cpages * 2 * D.tile_bytes > 96 * 1024) {
        s_cross = D.S_max < D.cpages ? D.S_max : D.cpages;
        if (s_cross < 1) s_cross = 1;
    }
    D.S_cross = s_cross;
    D.B = batch; D.M = batch * D.K1;
    build_tables(ctx);
    if (!D.umma && umma_shape(c, batch)) {      // the tensor maps could not be made: plan the shared memory of the mma.sync path
        if (const char *m = plan_smem(c, batch, D, smem_bytes)) return fail(ctx, XSM_ERR_CAPACITY, m);
        ctx->smem_bytes = smem_bytes;
    }
    if (D.umma)
        XSM_CUDA(ctx, cudaMemcpyAsync(ctx->ws + ctx->lay.tmaps, ctx->h_tmaps.data(), sizeof(CUtensorMap) * ctx->h_tmaps.size(),
                                      cudaMemcpyHostToDevice, ctx->stream));
    D.n_stages = ctx->n_stages;
    XSM_CUDA(ctx, cudaMemcpyAsync(ctx->ws + ctx->lay.phases, &ctx->h_tab, sizeof(Tables), cudaMemcpyHostToDevice, ctx->stream));
    if ((const void *)d_prompt != (const void *)D.prompt)
        XSM_CUDA(ctx, cudaMemcpyAsync((void *)D.prompt, d_prompt, sizeof(int32_t) * batch * prompt_len,
                                      cudaMemcpyDeviceToDevice, ctx->stream));
    // no tag of an earlier generation may survive: the exchange buffers restart from "never written"
    XSM_CUDA(ctx, cudaMemsetAsync(ctx->ws + ctx->lay.xchg_begin, 0, ctx->lay.xchg_end - ctx->lay.xchg_begin, ctx->stream));
    ctx->serial = 0;
    ctx->static_steps = 0;
    D.script = nullptr; D.script_n = 0; D.script_acc = 0;
    // the table above is read from host memory that the next prefill rewrites
    XSM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    XSM_CUDA(ctx, launch_init(D, c.dtype, ctx->serial, ctx->stream));      // also clears the status word
    XSM_CUDA(ctx, launch_cross_kv(D, c.dtype, ctx->weights, at<size_t>(ctx, ctx->lay.wkc_off),
                                  at<size_t>(ctx, ctx->lay.wvc_off), d_cond, D.ckv_pool, D.L, ctx->stream));
    if (c.head_kind == 1 && D.K > 0) {
        XSM_CUDA(ctx, launch_cross_kv(D, c.dtype, ctx->weights, at<size_t>(ctx, ctx->lay.hk_off),
                                      at<size_t>(ctx, ctx->lay.hv_off), d_cond, D.hckv_pool, D.K, ctx->stream));
        ctx->launches += 1;
    }
    ctx->launches += 3;
    ctx->prefilled = 1;
    const int ingest_steps = (prompt_len - 1 + D.K1 - 1) / D.K1;
    if (ingest_steps > 0) {
        xsm_status st = run_steps(ctx, ingest_steps);
        if (st != XSM_OK) return st;
    }
    return XSM_OK;
}

xsm_status xsm_spec_step(xsm_ctx *ctx, int32_t *d_new_tokens, int32_t *d_n_new) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "xsm_spec_step before xsm_prefill");
    ctx->dev.max_new = INT_MAX;
    xsm_status st = run_steps(ctx, 1);
    if (st != XSM_OK) return st;
    const Dev &D = ctx->dev;
    if (d_new_tokens)
        XSM_CUDA(ctx, cudaMemcpyAsync(d_new_tokens, D.step_tokens, sizeof(int32_t) * D.M, cudaMemcpyDeviceToDevice, ctx->stream));
    if (d_n_new)
        XSM_CUDA(ctx, cudaMemcpyAsync(d_n_new, D.step_n_new, sizeof(int32_t) * D.B, cudaMemcpyDeviceToDevice, ctx->stream));
    return XSM_OK;
}

// ---- scratch owned by the library, for xsm_spec_step_static
// The name below is a device symbol: host code may not use it as an address.  Its device address is asked
// for once per device (cudaGetSymbolAddress) and kept.
constexpr size_t kStaticScratchBytes = (size_t)1 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static std::atomic<void *> g_static_scratch_addr[kMaxDevices];   // by device ordinal; null until the first call on that device

xsm_status xsm_spec_step_static(xsm_ctx *ctx, int32_t *d_new_tokens, int32_t *d_n_new) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "xsm_spec_step_static before xsm_prefill");
    Dev &D = ctx->dev;
    // the split partials of self- and cross-attention: [B * H * S_max][K + 1][d_head + 2] floats each; cross-attention
    // heads have K more such sets
    const size_t one = (size_t)D.B * D.H * D.S_max * D.K1 * (D.dh + 2) * sizeof(float);
    const size_t half = (one + 255) / 256 * 256;
    const size_t n_sets = 2 + (D.head_kind == 1 ? (size_t)D.K : 0);
    if (n_sets * half > kStaticScratchBytes)
        return fail(ctx, XSM_ERR_CAPACITY, "xsm_spec_step_static: the attention partials of this batch need " +
                                               std::to_string(n_sets * half) + " bytes, the built-in scratch holds " +
                                               std::to_string(kStaticScratchBytes));
    int dev = 0;
    XSM_CUDA(ctx, cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(ctx, XSM_ERR_INVALID_ARG, "device ordinal out of range");
    if (g_static_scratch_addr[dev].load() == nullptr) {   // set-up, once per device, with that device current
        void *p = nullptr;                                // (threads that race here all store the same address)
        XSM_CUDA(ctx, cudaGetSymbolAddress(&p, g_static_scratch));
        g_static_scratch_addr[dev].store(p);
    }
    char *scratch = static_cast<char *>(g_static_scratch_addr[dev].load());
    // the array keeps what the last call left; a stale tag would pass for a fresh partial, so it restarts from zero
    XSM_CUDA(ctx, cudaMemsetAsync(scratch, 0, n_sets * half, ctx->stream));
    float *const ws_part = D.part, *const ws_cpart = D.cpart, *const ws_hpart = D.hpart;
    D.part = reinterpret_cast<float *>(scratch);
    D.cpart = reinterpret_cast<float *>(scratch + half);
    if (D.head_kind == 1) D.hpart = reinterpret_cast<float *>(scratch + 2 * half);
    D.max_new = INT_MAX;
    const xsm_status st = run_steps(ctx, 1, true);     // the kernel arguments are copied at launch
    D.part = ws_part;
    D.cpart = ws_cpart;
    D.hpart = ws_hpart;
    if (st != XSM_OK) return st;
    if (d_new_tokens)
        XSM_CUDA(ctx, cudaMemcpyAsync(d_new_tokens, D.step_tokens, sizeof(int32_t) * D.M, cudaMemcpyDeviceToDevice, ctx->stream));
    if (d_n_new)
        XSM_CUDA(ctx, cudaMemcpyAsync(d_n_new, D.step_n_new, sizeof(int32_t) * D.B, cudaMemcpyDeviceToDevice, ctx->stream));
    return XSM_OK;
}

xsm_status xsm_generate(xsm_ctx *ctx, int max_new_tokens, int32_t *d_tokens, int32_t *d_lengths, xsm_stats *host_stats) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "xsm_generate before xsm_prefill");
    if (max_new_tokens < 1 || max_new_tokens > ctx->cfg.max_seq_len)
        return fail(ctx, XSM_ERR_INVALID_ARG, "max_new_tokens must be in [1, max_seq_len]");
    Dev &D = ctx->dev;
    D.max_new = max_new_tokens;
    XSM_CUDA(ctx, cudaEventRecord(ctx->ev0, ctx->stream));
    long long budget = (long long)max_new_tokens + 2;   // every step commits at least one token per live sequence
    while (budget > 0) {
        const int n = (int)(budget < kChunkSteps ? budget : kChunkSteps);
        xsm_status st = run_steps(ctx, n);
        if (st != XSM_OK) return st;
        budget -= n;
        st = check_device_status(ctx);
        if (st != XSM_OK) return st;
        if (ctx->pinned[0] <= 0) break;
    }
    XSM_CUDA(ctx, cudaEventRecord(ctx->ev1, ctx->stream));
    if (d_tokens || d_lengths) {
        XSM_CUDA(ctx, launch_export(D, max_new_tokens, d_tokens, d_lengths, ctx->stream));
        ctx->launches += 1;
    }
    XSM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    float ms = 0.f;
    XSM_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
    ctx->last_wall_ms = ms;
    if (host_stats) {
        std::vector<unsigned long long> hist((size_t)D.B * (kMaxDraft + 1)), steps(D.B);
        std::vector<int> ngen(D.B);
        XSM_CUDA(ctx, cudaMemcpy(hist.data(), D.hist, 8 * hist.size(), cudaMemcpyDeviceToHost));
        XSM_CUDA(ctx, cudaMemcpy(steps.data(), D.steps, 8 * steps.size(), cudaMemcpyDeviceToHost));
        XSM_CUDA(ctx, cudaMemcpy(ngen.data(), D.n_gen, 4 * ngen.size(), cudaMemcpyDeviceToHost));
        memset(host_stats, 0, sizeof(*host_stats));
        for (int b = 0; b < D.B; ++b) {
            host_stats->steps += steps[b];
            host_stats->tokens += (uint64_t)ngen[b];
            for (int a = 0; a <= kMaxDraft; ++a) host_stats->accept_hist[a] += hist[(size_t)b * (kMaxDraft + 1) + a];
        }
        host_stats->wall_ms = ms;
        host_stats->scr = host_stats->steps ? (double)host_stats->tokens / (double)host_stats->steps : 0.0;
    }
    return XSM_OK;
}

xsm_status xsm_generate_host(xsm_ctx *ctx, int batch, const void *h_cond, const int32_t *h_prompt, int prompt_len,
                             const xsm_decode_config *dc, int max_new_tokens, int32_t *h_tokens, int32_t *h_lengths,
                             xsm_stats *host_stats) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!h_cond || !h_prompt || !dc || !h_tokens || !h_lengths) return fail(ctx, XSM_ERR_INVALID_ARG, "null argument");
    const xsm_model_config &c = ctx->cfg;
    if (batch < 1 || batch > c.max_batch) return fail(ctx, XSM_ERR_INVALID_ARG, "batch must be in [1, max_batch]");
    if (prompt_len < 1 || prompt_len - 1 > c.max_seq_len) return fail(ctx, XSM_ERR_INVALID_ARG, "prompt_len out of range");
    if (max_new_tokens < 1 || max_new_tokens > c.max_seq_len)
        return fail(ctx, XSM_ERR_INVALID_ARG, "max_new_tokens must be in [1, max_seq_len]");
    void *d_cond = ctx->ws + ctx->lay.stage_cond;
    int32_t *d_prompt = at<int32_t>(ctx, ctx->lay.prompt);
    int32_t *d_tok = at<int32_t>(ctx, ctx->lay.stage_tok);
    XSM_CUDA(ctx, cudaMemcpyAsync(d_cond, h_cond, esize(c) * (size_t)batch * c.n_cond * c.d_cond, cudaMemcpyHostToDevice, ctx->stream));
    XSM_CUDA(ctx, cudaMemcpyAsync(d_prompt, h_prompt, sizeof(int32_t) * (size_t)batch * prompt_len, cudaMemcpyHostToDevice, ctx->stream));
    xsm_status st = xsm_prefill(ctx, batch, d_cond, d_prompt, prompt_len, dc);
    if (st != XSM_OK) return st;
    // lengths are staged behind the tokens
    int32_t *d_len = at<int32_t>(ctx, ctx->lay.step_n_new);
    st = xsm_generate(ctx, max_new_tokens, d_tok, d_len, host_stats);
    if (st != XSM_OK) return st;
    XSM_CUDA(ctx, cudaMemcpyAsync(h_tokens, d_tok, sizeof(int32_t) * (size_t)batch * max_new_tokens, cudaMemcpyDeviceToHost, ctx->stream));
    XSM_CUDA(ctx, cudaMemcpyAsync(h_lengths, d_len, sizeof(int32_t) * batch, cudaMemcpyDeviceToHost, ctx->stream));
    XSM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return XSM_OK;
}

xsm_status xsm_destroy(xsm_ctx *ctx) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    cudaStreamSynchronize(ctx->stream);
    if (ctx->pinned) cudaFreeHost(ctx->pinned);
    if (ctx->ev0) cudaEventDestroy(ctx->ev0);
    if (ctx->ev1) cudaEventDestroy(ctx->ev1);
    delete ctx;
    return XSM_OK;
}

const char *xsm_last_error(const xsm_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

uint64_t xsm_kernel_launches(const xsm_ctx *ctx) { return ctx ? ctx->launches : 0; }

// the exchange buffers hold fp32 words whose two lowest mantissa bits are a tag
static void strip_tags(float *p, size_t n) {
    uint32_t *u = reinterpret_cast<uint32_t *>(p);
    for (size_t i = 0; i < n; ++i) u[i] &= ~3u;
}

xsm_status xsm_debug_get_logits(xsm_ctx *ctx, float *h_logits0, float *h_head_logits) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "no step has run");
    const Dev &D = ctx->dev;
    xsm_status st = check_device_status(ctx);
    if (st != XSM_OK) return st;
    if (h_logits0) {
        XSM_CUDA(ctx, cudaMemcpy(h_logits0, D.logits0, sizeof(float) * (size_t)D.M * D.V, cudaMemcpyDeviceToHost));
        strip_tags(h_logits0, (size_t)D.M * D.V);
    }
    if (h_head_logits && D.K > 0) {
        XSM_CUDA(ctx, cudaMemcpy(h_head_logits, D.hlogits, sizeof(float) * (size_t)D.K * D.M * D.V, cudaMemcpyDeviceToHost));
        strip_tags(h_head_logits, (size_t)D.K * D.M * D.V);
    }
    return XSM_OK;
}

xsm_status xsm_debug_get_kv(xsm_ctx *ctx, int layer, int seq, int pos0, int n, float *h_k, float *h_v) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "no cache yet");
    const Dev &D = ctx->dev;
    if (layer < 0 || layer >= D.L || seq < 0 || seq >= D.B || pos0 < 0 || n < 0 || !h_k || !h_v)
        return fail(ctx, XSM_ERR_INVALID_ARG, "bad layer, sequence or range");
    xsm_status st = check_device_status(ctx);
    if (st != XSM_OK) return st;
    int held = 0;
    XSM_CUDA(ctx, cudaMemcpy(&held, D.n_blocks + seq, 4, cudaMemcpyDeviceToHost));
    if ((long long)pos0 + n > (long long)held * D.P) return fail(ctx, XSM_ERR_INVALID_ARG, "range beyond the pages held");
    float *sk = at<float>(ctx, ctx->lay.stage_kv), *sv = sk + (size_t)kKvStagePositions * D.d;
    for (int p = 0; p < n; p += kKvStagePositions) {
        const int m = n - p < kKvStagePositions ? n - p : kKvStagePositions;
        XSM_CUDA(ctx, launch_gather_kv(D, ctx->cfg.dtype, layer, seq, pos0 + p, m, sk, sv, ctx->stream));
        ctx->launches += 1;
        XSM_CUDA(ctx, cudaMemcpyAsync(h_k + (size_t)p * D.d, sk, sizeof(float) * (size_t)m * D.d, cudaMemcpyDeviceToHost, ctx->stream));
        XSM_CUDA(ctx, cudaMemcpyAsync(h_v + (size_t)p * D.d, sv, sizeof(float) * (size_t)m * D.d, cudaMemcpyDeviceToHost, ctx->stream));
        XSM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    }
    return XSM_OK;
}

xsm_status xsm_debug_set_drafts(xsm_ctx *ctx, const int32_t *h_drafts) {
    if (!ctx || !h_drafts) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "xsm_debug_set_drafts before xsm_prefill");
    const Dev &D = ctx->dev;
    if (D.K == 0) return XSM_OK;
    for (int i = 0; i < D.B * D.K; ++i)
        if (h_drafts[i] < 0 || h_drafts[i] >= D.V) return fail(ctx, XSM_ERR_INVALID_ARG, "draft token out of range");
    XSM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    XSM_CUDA(ctx, cudaMemcpy2D(D.window + 1, sizeof(int32_t) * D.K1, h_drafts, sizeof(int32_t) * D.K,
                               sizeof(int32_t) * D.K, D.B, cudaMemcpyHostToDevice));
    XSM_CUDA(ctx, launch_embed(D, ctx->cfg.dtype, ctx->serial, ctx->stream));
    ctx->launches += 1;
    return XSM_OK;
}

xsm_status xsm_debug_get_state(xsm_ctx *ctx, int32_t *h_len, int32_t *h_window, int32_t *h_finished, int32_t *h_pages,
                               int32_t *h_free_pages) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "no state before xsm_prefill");
    const Dev &D = ctx->dev;
    xsm_status st = check_device_status(ctx);
    if (st != XSM_OK) return st;
    if (h_len) XSM_CUDA(ctx, cudaMemcpy(h_len, D.len, 4 * D.B, cudaMemcpyDeviceToHost));
    if (h_window) XSM_CUDA(ctx, cudaMemcpy(h_window, D.window, 4 * D.M, cudaMemcpyDeviceToHost));
    if (h_finished) XSM_CUDA(ctx, cudaMemcpy(h_finished, D.finished, 4 * D.B, cudaMemcpyDeviceToHost));
    if (h_pages) XSM_CUDA(ctx, cudaMemcpy(h_pages, D.n_blocks, 4 * D.B, cudaMemcpyDeviceToHost));
    if (h_free_pages) XSM_CUDA(ctx, cudaMemcpy(h_free_pages, D.n_free, 4, cudaMemcpyDeviceToHost));
    return XSM_OK;
}

xsm_status xsm_debug_trace_step(xsm_ctx *ctx, uint64_t *h_times, size_t capacity, int *n_rows, int *n_ctas) {
    if (!ctx || !h_times || !n_rows || !n_ctas) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "xsm_debug_trace_step before xsm_prefill");
    if (ctx->phase_launch) return fail(ctx, XSM_ERR_STATE, "the timeline is taken from the persistent kernel");
    const int rows = 1 + 2 * ctx->n_stages;
    const size_t words = (size_t)rows * ctx->grid;
    if (capacity < words) return fail(ctx, XSM_ERR_CAPACITY, "h_times is too small");
    unsigned long long *d_trace = at<unsigned long long>(ctx, ctx->lay.trace);
    XSM_CUDA(ctx, cudaMemsetAsync(d_trace, 0, 8 * words, ctx->stream));
    ctx->dev.trace = d_trace;
    ctx->dev.max_new = INT_MAX;
    xsm_status st = run_steps(ctx, 1);
    ctx->dev.trace = nullptr;
    if (st != XSM_OK) return st;
    st = check_device_status(ctx);
    if (st != XSM_OK) return st;
    XSM_CUDA(ctx, cudaMemcpy(h_times, d_trace, 8 * words, cudaMemcpyDeviceToHost));
    *n_rows = rows;
    *n_ctas = ctx->grid;
    return XSM_OK;
}

xsm_status xsm_debug_set_script(xsm_ctx *ctx, const int32_t *h_tokens, int n, float mean_accept) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "xsm_debug_set_script before xsm_prefill");
    Dev &D = ctx->dev;
    if (h_tokens == nullptr || n <= 0) { D.script = nullptr; D.script_n = 0; D.script_acc = 0; return XSM_OK; }
    if (n > ctx->lay.tok_ld) return fail(ctx, XSM_ERR_INVALID_ARG, "script longer than max_seq_len + n_draft + 1");
    if (!(mean_accept >= 0.f) || mean_accept > (float)D.K) return fail(ctx, XSM_ERR_INVALID_ARG, "mean_accept must be in [0, n_draft]");
    for (long long i = 0; i < (long long)D.B * n; ++i)
        if (h_tokens[i] < 0 || h_tokens[i] >= D.V) return fail(ctx, XSM_ERR_INVALID_ARG, "script token out of range");
    int *d_script = at<int>(ctx, ctx->lay.script);
    XSM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    XSM_CUDA(ctx, cudaMemcpy(d_script, h_tokens, sizeof(int32_t) * (size_t)D.B * n, cudaMemcpyHostToDevice));
    D.script = d_script; D.script_n = n; D.script_acc = (int)lrintf(mean_accept * 1024.f);
    return XSM_OK;
}

xsm_status xsm_debug_set_wait_limits(xsm_ctx *ctx, uint32_t polls, uint32_t barrier_tries) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    ctx->dev.spin_limit = polls ? polls : kSpinLimit;
    ctx->dev.mbar_limit = barrier_tries ? barrier_tries : kMbarSpinLimit;
    return XSM_OK;
}

xsm_status xsm_debug_launch_stage(xsm_ctx *ctx, int stage) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    if (!ctx->prefilled) return fail(ctx, XSM_ERR_STATE, "xsm_debug_launch_stage before xsm_prefill");
    if (stage < 0 || stage >= ctx->n_stages) return fail(ctx, XSM_ERR_INVALID_ARG, "no such stage");
    XSM_CUDA(ctx, launch_step(ctx->dev, ctx->cfg.dtype, stage, stage + 1, 1, ctx->serial, ctx->grid, ctx->smem_bytes, ctx->stream));
    ctx->launches += 1;
    return XSM_OK;
}

xsm_status xsm_debug_set_phase_launch(xsm_ctx *ctx, int on) {
    if (!ctx) return XSM_ERR_INVALID_ARG;
    ctx->phase_launch = on ? 1 : 0;
    return XSM_OK;
}

}  // extern "C"
