// Internal declarations shared by the host API (xsm_api.cu) and the kernels (xsm_kernels.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace xsm {

constexpr int kThreads = 512;            // threads per CTA of the persistent step kernel
constexpr int kWarps = kThreads / 32;
constexpr int kMaxDraft = 16;
constexpr int kMaxTokens = 512;          // largest M = batch * (K + 1)
constexpr int kUnitBlock = 128;          // weight rows a CTA accumulates at a time
constexpr int kSmemBytes = 200 * 1024;   // dynamic shared memory of the step kernel

// One step of Algorithm 1 is a fixed list of phases; consecutive phases are separated by a grid barrier.
enum PhaseKind : int { PH_GEMV = 0, PH_ATTN_SELF = 1, PH_ATTN_CROSS = 2, PH_SAMPLE = 3, PH_COMMIT = 4 };
enum Epilogue : int {
    EPI_STORE = 0,    // out[m][r]  = W[r] . x[m]
    EPI_ADD = 1,      // out[m][r] += W[r] . x[m]                       (residual)
    EPI_GATEUP = 2,   // out[m][r]  = SiLU(Wgate[r] . x[m]) * (Wup[r] . x[m])
    EPI_HEADY = 3     // out[m][r]  = x[m][r] + SiLU(W[r] . x[m])       (x = normed input)
};

struct GemvJob {
    const void *W, *W2;      // weight rows; W2: the up projection of EPI_GATEUP
    const float *x;          // input activations [M][kdim]
    const void *gain;        // RMSNorm gain of the input (weight dtype) or nullptr: input used as is
    float *out;
    int rows, kdim, x_ld, out_ld, epi, pad;
};

struct Phase { int kind, layer, job0, njobs; };

// Everything a kernel needs; passed by value.
struct Dev {
    // shape
    int L, d, H, dh, f, V, C, dc, K, K1, B, M, P;
    int max_blocks, n_pages, cpages, max_seq_len, tok_ld;
    int S_self, S_cross;
    float eps, scale;
    int bos, eos;
    // decoding rule
    int verify_mode, k_accept, sample_mode, k_sample;
    float delta, temperature;
    uint32_t key0, key1;
    int max_new;
    // tables
    const Phase *phases;
    const GemvJob *jobs;
    int n_phases;
    const void *E;                 // embedding table
    const double *inv_freq;        // [dh/2] theta^(-2i/dh)
    // per-sequence state
    int *len, *window, *cand, *acc_len, *finished, *n_gen, *n_blocks, *block_table, *ingest_left;
    uint32_t *step_idx;
    int *free_stack, *n_free, *n_active, *status;
    unsigned long long *hist, *steps;
    int *tok_log, *step_tokens, *step_n_new;
    const int *prompt;
    int prompt_len;
    // activations
    float *h, *qkv, *attn, *qc, *cattn, *act, *y, *logits0, *hlogits;
    float2 *rope_cs;               // [M][dh/2] cos, sin of the window rows' positions
    float *part, *cpart;           // split partials: [B*H*S][K1][dh+2]
    unsigned *part_ctr, *cpart_ctr;
    // caches
    void *kv_pool;                 // [L][2][n_pages][H][P][dh]
    void *ckv_pool;                // [L][2][B*cpages][H][P][dh]
    unsigned *bar;
};

struct LaunchInfo { int grid; int coop; };

// Host-side launchers (xsm_kernels.cu).  All return the CUDA error of the launch.
cudaError_t launch_step(const Dev &D, int dtype, int ph_lo, int ph_hi, int n_steps, int barrier, int grid,
                        cudaStream_t st);
cudaError_t launch_cross_kv(const Dev &D, int dtype, const void *W /*flat weights*/, const size_t *wkc_off,
                            const size_t *wvc_off, const void *cond, cudaStream_t st);
cudaError_t launch_init(const Dev &D, int dtype, cudaStream_t st);
cudaError_t launch_embed(const Dev &D, int dtype, cudaStream_t st);
cudaError_t launch_gather_kv(const Dev &D, int dtype, int layer, int seq, int pos0, int n, float *out_k,
                             float *out_v, cudaStream_t st);
cudaError_t launch_export(const Dev &D, int max_new, int *d_tokens, int *d_lengths, cudaStream_t st);
cudaError_t step_kernel_setup(int dtype, int *max_grid);

}  // namespace xsm
