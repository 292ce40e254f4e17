// Host-side launchers and the kernels around the decoding step: prefill (condition keys and values, first
// window), inspection, export.  The step kernel itself is compiled in xsm_step_dh*.cu from xsm_device.cuh.
#include "xsm_device.cuh"

namespace xsm {

cudaError_t launch_step_dh32(const Dev &, int, int, int, int, uint32_t, int, int, cudaStream_t, int *);
cudaError_t launch_step_dh64(const Dev &, int, int, int, int, uint32_t, int, int, cudaStream_t, int *);
cudaError_t launch_step_dh128(const Dev &, int, int, int, int, uint32_t, int, int, cudaStream_t, int *);

static cudaError_t step_dispatch(const Dev &D, int dtype, int st_lo, int st_hi, int n_steps, uint32_t serial0, int grid,
                                 int smem_bytes, cudaStream_t st, int *max_grid) {
    if (D.dh == 32) return launch_step_dh32(D, dtype, st_lo, st_hi, n_steps, serial0, grid, smem_bytes, st, max_grid);
    if (D.dh == 64) return launch_step_dh64(D, dtype, st_lo, st_hi, n_steps, serial0, grid, smem_bytes, st, max_grid);
    return launch_step_dh128(D, dtype, st_lo, st_hi, n_steps, serial0, grid, smem_bytes, st, max_grid);
}

// resident CTAs of the instance that serves D (D.M and D.dh set)
cudaError_t step_kernel_setup(const Dev &D, int dtype, int smem_bytes, int *max_grid) {
    return step_dispatch(D, dtype, 0, 0, 0, 0u, 0, smem_bytes, nullptr, max_grid);
}

cudaError_t launch_step(const Dev &D, int dtype, int st_lo, int st_hi, int n_steps, uint32_t serial0, int grid,
                        int smem_bytes, cudaStream_t st) {
    return step_dispatch(D, dtype, st_lo, st_hi, n_steps, serial0, grid, smem_bytes, st, nullptr);
}

// ------------------------------------------------------------------------------- prefill kernels

// Cross-attention keys and values of the condition (computed once per mesh):
// out[c][r] = sum_k W[r][k] * cond[b][c][k], stored as cache tiles.
template <typename WT>
__global__ void __launch_bounds__(256) cross_kv_kernel(const Dev D, const WT *Wall, const size_t *wkc_off,
                                                       const size_t *wvc_off, const WT *cond, void *pool) {
    constexpr int T = 64, KT = 16;
    __shared__ float As[KT][T + 1], Bs[KT][T + 1];
    const int z = blockIdx.z, b = z % D.B, kv = (z / D.B) % 2, layer = z / (2 * D.B);
    const WT *W = Wall + (kv == 0 ? wkc_off[layer] : wvc_off[layer]);
    const WT *A = cond + (size_t)b * D.C * D.dc;
    const int c0 = blockIdx.x * T, r0 = blockIdx.y * T;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < D.dc; k0 += KT) {
        for (int i = threadIdx.x; i < T * KT; i += 256) {
            const int rr = i / KT, kk = i % KT;
            As[kk][rr] = (c0 + rr < D.C && k0 + kk < D.dc) ? to_f(A[(size_t)(c0 + rr) * D.dc + k0 + kk]) : 0.f;
            Bs[kk][rr] = (r0 + rr < D.d && k0 + kk < D.dc) ? to_f(W[(size_t)(r0 + rr) * D.dc + k0 + kk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < KT; ++kk) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = As[kk][ty * 4 + i]; bv[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + ty * 4 + i, r = r0 + tx * 4 + j;
            if (c < D.C && r < D.d) {
                const int page = b * D.cpages + c / D.P, head = r / D.dh, e = r % D.dh;
                typedef typename CacheT<WT>::type KVT;
                KVT *tile = kv_tile<KVT>(D, pool, D.B * D.cpages, layer, kv, page, head);
                tile[tile_off<KVT>(c % D.P, e, D.dh)] = from_f<KVT>(acc[i][j]);
            }
        }
}

// n_sets projections of the condition (the layers' Wkc / Wvc into the cross-attention cache, or the decoding heads'
// own Wk / Wv into theirs); set i of the offset tables fills set i of `pool`
cudaError_t launch_cross_kv(const Dev &D, int dtype, const void *W, const size_t *wkc_off, const size_t *wvc_off,
                            const void *cond, void *pool, int n_sets, cudaStream_t st) {
    dim3 grid((D.C + 63) / 64, (D.d + 63) / 64, n_sets * 2 * D.B);
    if (dtype == 1)
        cross_kv_kernel<bf16><<<grid, 256, 0, st>>>(D, (const bf16 *)W, wkc_off, wvc_off, (const bf16 *)cond, pool);
    else
        cross_kv_kernel<float><<<grid, 256, 0, st>>>(D, (const float *)W, wkc_off, wvc_off, (const float *)cond, pool);
    return cudaGetLastError();
}

// shared memory of prepare_window's partial sums: one float per 16 bytes of the window's embedding rows
static size_t window_scratch_bytes(const Dev &D, int elem_bytes) { return (size_t)D.K1 * (D.d / (16 / elem_bytes)) * sizeof(float); }

// Algorithm 1 line 1: pool reset, then per-sequence state, first window and its pages.
__global__ void init_pool_kernel(const Dev D) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < D.n_pages) D.free_stack[i] = D.n_pages - 1 - i;
    if (i == 0) { *D.n_free = D.n_pages; *D.n_active = D.B; *D.status = 0; }
}

template <typename WT> __global__ void __launch_bounds__(256) init_seq_kernel(const Dev D, uint32_t serial) {
    const int b = blockIdx.x, K1 = D.K1;
    extern __shared__ float s_scratch[];      // K1 * d_model / (elements per 16 bytes) floats
    __shared__ int s_win[kMaxDraft + 1];
    if (threadIdx.x == 0) {
        D.len[b] = 0; D.finished[b] = 0; D.n_gen[b] = 0; D.n_blocks[b] = 0; D.step_idx[b] = 0u;
        D.acc_len[b] = 0; D.steps[b] = 0ull; D.step_n_new[b] = 0;
        for (int a = 0; a <= kMaxDraft; ++a) D.hist[(size_t)b * (kMaxDraft + 1) + a] = 0ull;
        const int *pr = D.prompt + (size_t)b * D.prompt_len;
        D.ingest_left[b] = D.prompt_len - 1;
        if (D.prompt_len == 1) {
            s_win[0] = pr[0];
            draw_initial_drafts(D, b, s_win);
        } else {
            for (int j = 0; j < K1; ++j) s_win[j] = j < D.prompt_len ? pr[j] : 0;
        }
        for (int j = 0; j < K1; ++j) D.window[b * K1 + j] = s_win[j];
    }
    __syncthreads();
    prepare_window<WT>(D, b, serial, 0, 0, s_win, 256, s_scratch);
    __threadfence();
    __syncthreads();
    publish_header(D, b, serial, 0, D.prompt_len > 1 ? 2 : 0);
}

cudaError_t launch_init(const Dev &D, int dtype, uint32_t serial, cudaStream_t st) {
    const int n = max(D.n_pages, 1);
    init_pool_kernel<<<(n + 255) / 256, 256, 0, st>>>(D);
    if (dtype == 1) init_seq_kernel<bf16><<<D.B, 256, window_scratch_bytes(D, 2), st>>>(D, serial);
    else init_seq_kernel<float><<<D.B, 256, window_scratch_bytes(D, 4), st>>>(D, serial);
    return cudaGetLastError();
}

// re-gather the window embeddings after the drafts were replaced from outside
template <typename WT> __global__ void __launch_bounds__(256) embed_kernel(const Dev D, uint32_t serial) {
    const int b = blockIdx.x;
    extern __shared__ float s_scratch[];
    if (!D.finished[b]) prepare_window<WT>(D, b, serial, D.len[b], D.n_blocks[b], D.window + b * D.K1, 256, s_scratch);
}
cudaError_t launch_embed(const Dev &D, int dtype, uint32_t serial, cudaStream_t st) {
    if (dtype == 1) embed_kernel<bf16><<<D.B, 256, window_scratch_bytes(D, 2), st>>>(D, serial);
    else embed_kernel<float><<<D.B, 256, window_scratch_bytes(D, 4), st>>>(D, serial);
    return cudaGetLastError();
}

template <typename KVT>
__global__ void gather_kv_kernel(const Dev D, int layer, int seq, int pos0, int n, float *out_k, float *out_v) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * D.d) return;
    const int p = pos0 + i / D.d, r = i % D.d, head = r / D.dh, e = r % D.dh;
    const int page = D.block_table[(size_t)seq * D.max_blocks + p / D.P];
    const KVT *kt = kv_tile<KVT>(D, D.kv_pool, D.n_pages, layer, 0, page, head);
    const KVT *vt = kv_tile<KVT>(D, D.kv_pool, D.n_pages, layer, 1, page, head);
    out_k[i] = to_f(kt[tile_off<KVT>(p % D.P, e, D.dh)]);
    out_v[i] = to_f(vt[tile_off<KVT>(p % D.P, e, D.dh)]);
}
cudaError_t launch_gather_kv(const Dev &D, int dtype, int layer, int seq, int pos0, int n, float *out_k,
                             float *out_v, cudaStream_t st) {
    const int total = n * D.d;
    if (dtype == 1) gather_kv_kernel<__half><<<(total + 255) / 256, 256, 0, st>>>(D, layer, seq, pos0, n, out_k, out_v);
    else gather_kv_kernel<float><<<(total + 255) / 256, 256, 0, st>>>(D, layer, seq, pos0, n, out_k, out_v);
    return cudaGetLastError();
}

__global__ void export_kernel(const Dev D, int max_new, int *tokens, int *lengths) {
    const int b = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    const int n = min(D.n_gen[b], max_new);
    if (i < max_new && tokens) tokens[(size_t)b * max_new + i] = i < n ? D.tok_log[(size_t)b * D.tok_ld + i] : -1;
    if (i == 0 && lengths) lengths[b] = n;
}
cudaError_t launch_export(const Dev &D, int max_new, int *d_tokens, int *d_lengths, cudaStream_t st) {
    dim3 grid((max_new + 255) / 256, D.B);
    export_kernel<<<grid, 256, 0, st>>>(D, max_new, d_tokens, d_lengths);
    return cudaGetLastError();
}

}  // namespace xsm
