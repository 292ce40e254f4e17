// Internal declarations shared by the host API (xsm_api.cu) and the kernels (xsm_kernels.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace xsm {

// ---- geometry of the persistent step kernel
constexpr int kConsumerWarps = 7;                    // warps that compute; with the producer warp: 8 warps, 255 registers each
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;      // + one producer warp that feeds the ring
constexpr int kMaxDraft = 16;                        // size of the histogram rows (n_draft itself is <= 15)
constexpr int kMaxTokens = 128;                      // largest M = batch * (K + 1)
constexpr int kMaxBatch = 128;
constexpr int kMaxDevices = 64;                      // device ordinals the per-device host tables cover
// Every device-side wait is bounded: polls of a tagged word (each an L2 round trip) and mbarrier try_wait calls.
constexpr unsigned kSpinLimit = 1u << 21, kMbarSpinLimit = 1u << 22;

// Ring of shared-memory slots filled by bulk copies.  A weight item is a run of consecutive weight rows at full
// width (at most kSlotBytes, one bulk copy); a cache item is one (page, head) tile of keys followed by the tile
// of values (or one of them when both do not fit).
constexpr int kSlotBytes = 16384;
constexpr int kMaxSlots = 12;
constexpr int kSmemHeader = 2048;                    // barriers and per-step scalars
constexpr int kAccumBytes = 16384;                   // accumulators of the projections that stage their activations in chunks
constexpr int kSmemMax = 227 * 1024;

// One step of Algorithm 1 is a fixed list of stages.  A stage's output is published in global memory as
// fp32 words whose two lowest mantissa bits carry a tag (1..3, cycling with the write index of the buffer);
// the next stage spins on the words it needs until they carry the expected tag.  No grid barrier exists.
enum StageKind : int { ST_GEMV = 0, ST_ATTN_SELF = 1, ST_ATTN_CROSS = 2, ST_SAMPLE = 3, ST_COMMIT = 4,
                       ST_ATTN_HEAD = 5 /* cross-attention of the decoding heads (Eq. 3) */ };
enum Epilogue : int {
    EPI_STORE = 0,    // out[m][r]  = W[r] . x[m]
    EPI_ADD = 1,      // h[m][r]   += W[r] . x[m]; out[m][r] = h[m][r]      (residual stream)
    EPI_GATEUP = 2,   // out[m][r]  = SiLU(Wgate[r] . x[m]) * (Wup[r] . x[m])
    EPI_HEADY = 3,    // out[m][r]  = x[m][r] + SiLU(W[r] . x[m])           (x = normed input)
    EPI_ADDG = 4      // out[m][r]  = res[m][r] + W[r] . x[m]               (res = the published final hidden state g)
};

// Write index of a tagged buffer = serial * wps + j (serial: decoding steps since xsm_prefill; wps: writes
// of that buffer per step; j: which write of the step).  tag = 1 + index % 3.
struct TagRef { int wps, j; };

struct GemvJob {
    const void *W, *W2;      // weight rows; W2: the up projection of EPI_GATEUP
    const float *x;          // tagged input activations [M][kdim]
    const void *gain;        // RMSNorm gain of the input (weight dtype) or nullptr: input used as is
    float *out;              // tagged output [M][out_ld]
    float *hm;               // EPI_ADD: untagged fp32 master copy of the residual stream [M][out_ld]
    int rows, kdim, out_ld, epi;
    TagRef in, outt;
    // bf16 models publish activations as bf16 hi + lo pairs (see xsm_device.cuh); then:
    const void *gain_out;    // EPI_ADD: RMSNorm gain of the stage that reads `out`, applied to the published copy
    int out_plain;           // 1: `out` is published as plain tagged fp32 (logits) even in a bf16 model
    int in_jinc, out_jinc;   // a layer job: how much in.j / outt.j grow from one layer to the next
    long long gain_out_step; // a layer job: bytes from one layer's gain_out to the next layer's
    const void *tmap, *tmap2; // tcgen05 path: tensor maps (in the workspace) of W and W2: {columns, rows, layers}, boxes of 64 x 8
    const float *res;        // EPI_ADDG: tagged fp32 residual [M][out_ld]
    int norm_out, pad_;      // norm_out (set per stage by the kernel): this job also publishes the CTA's columns of the normed input
};

struct Stage {
    int kind, layer, job0, njobs;
    TagRef in, outt, part;   // attention: q/k/v (or q) in, attention rows out, split partials
    int jinc;                // a layer stage: growth of the three j's per layer
    int norm_out;            // a projection stage whose input is normed: every CTA also publishes its columns of the normed input (D.gpub)
};

// Every layer has the same eight stages and the same weight layout, so the tables describe layer 0 (the
// weights of layer l lie l * layer_bytes further) and the tail of the step (LM head and decoding heads, their
// output projections, verify/resample, commit).  The step kernel works from a copy in shared memory.
constexpr int kLayerStages = 8, kMaxTailStages = 6, kLayerJobs = 6, kMaxTailJobs = 3 * kMaxDraft + 1;
struct Tables {
    Stage stages[kLayerStages + kMaxTailStages];
    long long layer_bytes;
    const void *gain_last;   // gain_out of the last layer's down projection (the final RMSNorm)
    int n_tail_stages, n_tail_jobs;
    GemvJob jobs[kLayerJobs + kMaxTailJobs];      // last: the copy in shared memory ends behind the jobs in use
};
// behind the tables: one record per job with this CTA's share of its rows and how they are tiled (fixed for a launch)
constexpr int kSegRecBytes = 40;
// shared memory of the tables' copy and of the plan records for a model with `tail_jobs` jobs in the tail of the step
// (Dev.tab_bytes, Dev.plan_bytes: the host sizes them, so that a model with few heads leaves more room for the ring)
constexpr int smem_tab_bytes(int tail_jobs) {
    return ((int)(sizeof(Tables) - sizeof(GemvJob) * (kMaxTailJobs - tail_jobs)) + 127) / 128 * 128;
}
constexpr int smem_plan_bytes(int tail_jobs) { return ((kLayerJobs + tail_jobs) * kSegRecBytes + 127) / 128 * 128; }

// Projections over 27 or more token rows on bf16 models run on the tensor cores of the 5th generation (tcgen05): the
// token rows (as bf16 hi and lo planes) are the M side of the product, a CTA's weight rows the N side, the fp32
// accumulator lives in tensor memory.  Weights arrive by TMA in boxes of 8 rows x 64 columns with the 128-byte swizzle;
// a ring item is one block of 64 columns for all row groups of a tile of at most kUmmaTileRows weight rows.
constexpr int kUmmaTileRows = 128, kUmmaK = 64, kUmmaTmemCols = 256;
constexpr int kUmmaMinRows = 27;                           // fewest token rows for which the path is chosen
constexpr int kUmmaPlaneBytes = 128 * kUmmaK * 2;          // one plane (hi or lo) of 128 token rows x 64 columns
constexpr int kUmmaActsBytes = 4 * kUmmaPlaneBytes;        // two buffers of two planes

constexpr int kSmallRedBytes = 512;   // at most eight token rows: partial products of one warp for one tile, [8 tokens][16 rows] floats

// Everything a kernel needs; passed by value.
struct Dev {
    // shape
    int L, d, H, dh, f, V, C, dc, K, K1, B, M, P;
    int max_blocks, n_pages, cpages, max_seq_len, tok_ld;
    int grid;                      // CTAs of the step kernel
    int inv_m;                     // ceil(2^20 / M): x / M == (x * inv_m) >> 20 for x < 8192
    int S_max, S_cross;            // most key splits of a self-attention item; splits of a cross-attention item
    float eps, scale;
    int bos, eos;
    // decoding rule
    int verify_mode, k_accept, sample_mode, k_sample;
    float delta, temperature;
    uint32_t key0, key1;
    int max_new;
    unsigned spin_limit, mbar_limit;   // bounds of the device-side waits (kSpinLimit, kMbarSpinLimit unless a test shortens them)
    // stage tables
    const Tables *tables;
    int n_stages;                  // 8 L + stages of the tail
    const void *E;                 // embedding table
    // shared-memory plan of the step kernel
    int n_slots, acts_bytes, kca, tile_bytes, kv_one_item;
    // per-sequence state (plain words, read by other CTAs only after they have seen the step header)
    int *len, *window, *cand, *acc_len, *finished, *n_gen, *n_blocks, *block_table, *ingest_left;
    uint32_t *step_idx;
    int *free_stack, *n_free, *n_active, *status;
    unsigned long long *hist, *steps;
    int *tok_log, *step_tokens, *step_n_new;
    const int *prompt;
    int prompt_len;
    // scripted drafts (load generator of the benchmark): null, or [B][script_n] tokens by absolute position; the commit
    // then drafts script tokens, of which the first floor((t+1) a) - floor(t a) are left intact at step t (a = script_acc / 1024)
    const int *script;
    int script_n, script_acc;
    // tagged exchange buffers
    float *hpub, *qkv, *attn, *qc, *cattn, *act, *y, *logits0, *hlogits, *part, *cpart;
    float *qh, *hattn, *gpub, *hpart;   // cross-attention heads: queries [K][M][d], attention rows [K][M][d], final hidden state [M][d], split partials
    void *hckv_pool;               // [K][2][B*cpages][H] tiles: keys and values of the condition under every head's own projections
    int head_kind;
    int umma;                      // projections on the tcgen05 path (bf16, kUmmaMinRows or more token rows)
    int p_shift;                   // log2 of the page size P if that is a power of two, else -1
    int tab_bytes, plan_bytes;     // shared memory of the tables' copy and of the plan records (the ring follows them)
    int small;                     // bf16, at most eight token rows, every projection's activations fit the staging area: the
                                   // kernel instance that holds nothing but that path runs the step
    uint32_t *treex;               // probability-tree sampling: [B][K][8][2] the heads' best tokens and their probabilities
    uint32_t *candx, *header;      // [B][K1 + 1] resampled tokens and accept length; [B][4] len, flags
    uint32_t *done;                // [grid] "this CTA has finished the projections of the step"
    float *sspub;                  // [grid][M] bf16 models: each CTA's share of the sum of squares of the rows of hpub
    const void *gain_first;        // RMSNorm gain that the first stage of a step applies to the embeddings
    unsigned long long *trace;     // null, or [1 + 2 * n_stages][grid] nanosecond timestamps of the launch's first step
    // untagged
    float *h;                      // master copy of the residual stream (each column range has one owner CTA)
    float2 *rope_cs;               // [max_seq_len + K + 2][dh/2] cos, sin of position * theta^(-2i/dh)
    // caches
    void *kv_pool;                 // [L][2][n_pages][H] tiles of P x dh
    void *ckv_pool;                // [L][2][B*cpages][H] tiles of P x dh
};

constexpr int kHeaderWords = 4;    // per sequence: len, flags (1 finished, 2 ingesting a prompt), 0, 0

// Host-side launchers (xsm_kernels.cu).  All return the CUDA error of the launch.
cudaError_t launch_step(const Dev &D, int dtype, int st_lo, int st_hi, int n_steps, uint32_t serial0, int grid,
                        int smem_bytes, cudaStream_t st);
cudaError_t launch_cross_kv(const Dev &D, int dtype, const void *W /*flat weights*/, const size_t *wkc_off,
                            const size_t *wvc_off, const void *cond, void *pool, int n_sets, cudaStream_t st);
cudaError_t launch_init(const Dev &D, int dtype, uint32_t serial, cudaStream_t st);
cudaError_t launch_embed(const Dev &D, int dtype, uint32_t serial, cudaStream_t st);
cudaError_t launch_gather_kv(const Dev &D, int dtype, int layer, int seq, int pos0, int n, float *out_k,
                             float *out_v, cudaStream_t st);
cudaError_t launch_export(const Dev &D, int max_new, int *d_tokens, int *d_lengths, cudaStream_t st);
cudaError_t step_kernel_setup(const Dev &D, int dtype, int smem_bytes, int *max_grid);

}  // namespace xsm
