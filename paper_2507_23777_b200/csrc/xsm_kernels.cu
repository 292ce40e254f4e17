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

// ---- the same projection on the 5th-generation tensor cores (bf16 models)
// One CTA: D[128 weight rows][64 condition latents] = W[r0.., :] * cond[b][c0.., :]^T, fp32 accumulator in tensor memory.
// Both operands are staged by the threads, 64 columns at a time, into the canonical K-major layout without swizzle that
// the matrix descriptors name: a core matrix is 8 rows x 16 bytes, stored contiguously (128 bytes); core matrices that
// follow each other along K lie 128 bytes apart (leading byte offset), 8-row groups 1024 bytes apart (stride byte
// offset).  One elected thread issues the four K = 16 products of a chunk and commits them to an mbarrier; every wait
// is bounded; the accumulator is read back with tcgen05.ld (thread = weight row) and written to the cache tiles.
__device__ __forceinline__ uint64_t umma_desc_kmajor(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) | ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) |
           (1ull << 46);      // descriptor version of sm_100, no swizzle, base offset 0
}
// instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, both K-major, N and M of the tile
__device__ __forceinline__ uint32_t umma_idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                 :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0), "r"(0), "r"(0), "r"(0) : "memory");
}
constexpr int kUmmaTileM = 128, kUmmaTileN = 64, kUmmaChunk = 64, kUmmaCols = 64;

__global__ void __launch_bounds__(128) cross_kv_umma_kernel(const Dev D, const bf16 *Wall, const size_t *wk_off, const size_t *wv_off,
                                                            const bf16 *cond, void *pool, int *status) {
    __shared__ __align__(1024) char sa[kUmmaTileM * kUmmaChunk * 2];     // [16 row groups][8 k-chunks][8 rows][16 B]
    __shared__ __align__(1024) char sb[kUmmaTileN * kUmmaChunk * 2];     // [ 8 row groups][8 k-chunks][8 rows][16 B]
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int z = blockIdx.z, b = z % D.B, kv = (z / D.B) % 2, set = z / (2 * D.B);
    const bf16 *W = Wall + (kv == 0 ? wk_off[set] : wv_off[set]);
    const bf16 *A = cond + (size_t)b * D.C * D.dc;
    const int c0 = blockIdx.x * kUmmaTileN, r0 = blockIdx.y * kUmmaTileM, dc = D.dc;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(kUmmaCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        mbar_init(smem_u32(&bar), 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_slot, idesc = umma_idesc_bf16(kUmmaTileM, kUmmaTileN);
    uint32_t parity = 0;
    bool dead = false;
    for (int k0 = 0; k0 < dc; k0 += kUmmaChunk) {
        // stage 16 bytes (8 columns of one row) at a time; rows and columns past the end are zeros
        for (int i = tid; i < (kUmmaTileM + kUmmaTileN) * (kUmmaChunk / 8); i += 128) {
            const bool is_w = i < kUmmaTileM * (kUmmaChunk / 8);
            const int j = is_w ? i : i - kUmmaTileM * (kUmmaChunk / 8);
            const int r = j / (kUmmaChunk / 8), c = j % (kUmmaChunk / 8), k = k0 + c * 8;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (k < dc) {
                if (is_w) { if (r0 + r < D.d) v = __ldg(reinterpret_cast<const uint4 *>(W + (size_t)(r0 + r) * dc + k)); }
                else if (c0 + r < D.C) v = __ldg(reinterpret_cast<const uint4 *>(A + (size_t)(c0 + r) * dc + k));
            }
            *reinterpret_cast<uint4 *>((is_w ? sa : sb) + (r >> 3) * 1024 + c * 128 + (r & 7) * 16) = v;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic-proxy writes, read by the tensor core's proxy
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (tid == 0) {
#pragma unroll
            for (int ks = 0; ks < kUmmaChunk / 16; ++ks)
                umma_bf16(tmem, umma_desc_kmajor(smem_u32(sa) + ks * 256, 128, 1024), umma_desc_kmajor(smem_u32(sb) + ks * 256, 128, 1024), idesc,
                          (k0 > 0 || ks > 0) ? 1u : 0u);
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(&bar)) : "memory");
        }
        // the chunk's products must be done before the buffers are overwritten (bounded wait)
        unsigned it = 0;
        while (!mbar_try_wait(smem_u32(&bar), parity)) {
            if (++it > kMbarSpinLimit) { dead = true; break; }
        }
        parity ^= 1u;
        if (dead) { atomicExch(status, XSM_STATUS_TIMEOUT); break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    if (!dead) {
        typedef CacheT<bf16>::type KVT;
        const int r = r0 + tid, head = r / D.dh, e = r % D.dh;       // thread = weight row = lane of the accumulator
        for (int n0 = 0; n0 < kUmmaTileN; n0 += 32) {
            uint32_t v[32];
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)n0;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,"
                         "%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
                           "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
                           "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
                           "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                         : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (r < D.d) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int c = c0 + n0 + j;
                    if (c < D.C) {
                        KVT *tile = kv_tile<KVT>(D, pool, D.B * D.cpages, set, kv, b * D.cpages + c / D.P, head);
                        tile[tile_off<KVT>(c % D.P, e, D.dh)] = from_f<KVT>(__uint_as_float(v[j]));
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kUmmaCols) : "memory");
}

// n_sets projections of the condition (the layers' Wkc / Wvc into the cross-attention cache, or the decoding heads'
// own Wk / Wv into theirs); set i of the offset tables fills set i of `pool`
cudaError_t launch_cross_kv(const Dev &D, int dtype, const void *W, const size_t *wkc_off, const size_t *wvc_off,
                            const void *cond, void *pool, int n_sets, cudaStream_t st) {
    dim3 grid((D.C + 63) / 64, (D.d + 63) / 64, n_sets * 2 * D.B);
    if (dtype == 1) {
        // a dense contraction (n_cond x d_cond x d_model per projection): tcgen05 tiles, operands 16-byte aligned rows
        if (D.dc % 8 == 0) {
            dim3 g2((D.C + kUmmaTileN - 1) / kUmmaTileN, (D.d + kUmmaTileM - 1) / kUmmaTileM, n_sets * 2 * D.B);
            cross_kv_umma_kernel<<<g2, 128, 0, st>>>(D, (const bf16 *)W, wkc_off, wvc_off, (const bf16 *)cond, pool, D.status);
        } else
            cross_kv_kernel<bf16><<<grid, 256, 0, st>>>(D, (const bf16 *)W, wkc_off, wvc_off, (const bf16 *)cond, pool);
    } else
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
