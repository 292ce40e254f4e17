// Kernels of the speculative decoding step (Algorithm 1, lines 3-12) for sm_100a.
//
// One decoding step is a fixed list of phases (projection, attention, ..., verify/resample, commit).
// The step kernel is persistent: one CTA per SM walks the whole list, a grid barrier separates
// consecutive phases, and a launch may run many steps.  Every CTA owns a slice of each phase's work:
//   projection  - a contiguous range of weight rows, streamed once with 128-bit loads
//   attention   - (sequence, head, key split) items; splits are merged by the last CTA to finish
//   verify      - (sequence, candidate slot) items
// Data written by one CTA and read by another after a barrier is read with ld.global.cg (L2), never
// through the non-coherent L1.  Weights are immutable and use ld.global.nc.
#include "xsm_internal.h"

#include <cuda_bf16.h>
#include <math.h>

namespace xsm {

typedef __nv_bfloat16 bf16;

// ------------------------------------------------------------------------------------------ helpers

__device__ __forceinline__ uint4 ldnc_u4(const void *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

template <typename T> __device__ __forceinline__ float ldcg_as_f(const T *p);
template <> __device__ __forceinline__ float ldcg_as_f<float>(const float *p) { return __ldcg(p); }
template <> __device__ __forceinline__ float ldcg_as_f<bf16>(const bf16 *p) {
    unsigned short u = __ldcg(reinterpret_cast<const unsigned short *>(p));
    return __uint_as_float(((unsigned)u) << 16);
}

__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + expf(-v)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// x = hi + lo with hi, lo bf16: 16 mantissa bits of x survive, products with bf16 weights stay exact in fp32.
__device__ __forceinline__ void split_bf16(float x, unsigned short &hi, unsigned short &lo) {
    bf16 h = __float2bfloat16_rn(x);
    bf16 l = __float2bfloat16_rn(x - __bfloat162float(h));
    hi = __bfloat16_as_ushort(h);
    lo = __bfloat16_as_ushort(l);
}

// D = A(16x16, row) * B(16x8, col) + D, bf16 inputs, fp32 accumulate
__device__ __forceinline__ void mma16816(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Philox4x32-10 (Salmon et al., SC'11): returns word 0.
__device__ __forceinline__ uint32_t philox_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                 uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
        uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
        uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
        c0 = n0; c1 = l1; c2 = n2; c3 = l0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}
__device__ __forceinline__ uint32_t rand24(const Dev &D, int seq, uint32_t step, uint32_t slot, uint32_t purpose) {
    return philox_word0(step, slot, purpose, 0u, D.key0 ^ (uint32_t)seq, D.key1) >> 8;
}

constexpr int XSM_STATUS_TIMEOUT = 5, XSM_STATUS_CAPACITY = 3;
constexpr unsigned kSpinLimit = 1u << 22;

// Grid-wide barrier on a monotonic counter (zeroed by the host before the launch).  The wait is
// bounded: when it runs out, or when any CTA has raised the status word, every CTA leaves the kernel.
__device__ bool grid_barrier(const Dev &D, unsigned &epoch) {
    __shared__ int ok_s;
    __syncthreads();
    epoch += 1;
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(D.bar, 1u);
        unsigned target = epoch * gridDim.x, it = 0;
        int ok = 1;
        while (ld_acquire_u32(D.bar) < target) {
            if (++it > kSpinLimit) {
                atomicExch(D.status, XSM_STATUS_TIMEOUT);
                ok = 0;
                break;
            }
        }
        if (__ldcg(D.status) != 0) ok = 0;
        ok_s = ok;
        __threadfence();
    }
    __syncthreads();
    return ok_s != 0;
}

// ------------------------------------------------------------------------------- projection phases

struct GemvSmem {
    float *inv;      // [kMaxTokens]   1/rms of each input row
    float *accbuf;   // [kUnitBlock][n_pad]
    float *red;      // [kWarps][16][n_pad]
    char *xs;        // staged activations
    int xs_bytes;
};

__device__ __forceinline__ GemvSmem carve_gemv(char *smem) {
    GemvSmem s;
    s.inv = reinterpret_cast<float *>(smem);
    s.accbuf = s.inv + kMaxTokens;
    s.red = s.accbuf + kUnitBlock * 32;
    s.xs = reinterpret_cast<char *>(s.red + kWarps * 16 * 32);
    s.xs_bytes = kSmemBytes - (int)(s.xs - smem);
    return s;
}

// weight row of accumulator row `arow` (within the current unit block), or nullptr past the end
template <typename WT>
__device__ __forceinline__ const WT *arow_ptr(const GemvJob &J, int ub, int nu, int arow, bool clamp) {
    if (J.epi == EPI_GATEUP) {
        int tile = arow >> 4, i = arow & 15, ui = tile * 8 + (i & 7);
        if (ui >= nu) {
            if (!clamp) return nullptr;
            ui = nu - 1;
        }
        const WT *base = reinterpret_cast<const WT *>(i < 8 ? J.W : J.W2);
        return base + (size_t)(ub + ui) * J.kdim;
    }
    int ui = arow;
    if (ui >= nu) {
        if (!clamp) return nullptr;
        ui = nu - 1;
    }
    return reinterpret_cast<const WT *>(J.W) + (size_t)(ub + ui) * J.kdim;
}

// bf16 weights: tensor-core dot products.  A = 16 weight rows x 32 k per warp step (two m16n8k16),
// B = activations of 8 tokens, split into hi + lo bf16 so that fp32 activations lose nothing that matters.
// Lane (g = lane/4, t = lane%4) loads 16 bytes (8 consecutive k) of rows g and g+8; the same k
// permutation is applied to the activation fragments, so the products pair up correctly.
template <int NT>
__device__ void gemv_tiles_bf16(const GemvJob &J, int ub, int nu, int kc0, int kc, const GemvSmem &S, int ldx) {
    constexpr int NP = NT * 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const unsigned short *xs_hi = reinterpret_cast<const unsigned short *>(S.xs);
    const unsigned short *xs_lo = xs_hi + (size_t)NP * ldx;
    const int narows = J.epi == EPI_GATEUP ? ((nu + 7) / 8) * 16 : nu;
    const int ntiles = (narows + 15) / 16;
    const int nkb = kc / 32;
    for (int tile = 0; tile < ntiles; ++tile) {
        const bf16 *ra = arow_ptr<bf16>(J, ub, nu, tile * 16 + g, true) + kc0 + t * 8;
        const bf16 *rb = arow_ptr<bf16>(J, ub, nu, tile * 16 + g + 8, true) + kc0 + t * 8;
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll 2
        for (int kb = warp; kb < nkb; kb += kWarps) {
            uint4 wa = ldnc_u4(ra + kb * 32), wb = ldnc_u4(rb + kb * 32);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const size_t xo = (size_t)(nt * 8 + g) * ldx + kb * 32 + t * 8;
                uint4 bh = *reinterpret_cast<const uint4 *>(xs_hi + xo);
                uint4 bl = *reinterpret_cast<const uint4 *>(xs_lo + xo);
                mma16816(acc[nt], wa.x, wb.x, wa.y, wb.y, bh.x, bh.y);
                mma16816(acc[nt], wa.z, wb.z, wa.w, wb.w, bh.z, bh.w);
                mma16816(acc[nt], wa.x, wb.x, wa.y, wb.y, bl.x, bl.y);
                mma16816(acc[nt], wa.z, wb.z, wa.w, wb.w, bl.z, bl.w);
            }
        }
        float *r0 = S.red + ((size_t)warp * 16 + g) * NP + 2 * t, *r1 = r0 + 8 * NP;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            r0[nt * 8] = acc[nt][0]; r0[nt * 8 + 1] = acc[nt][1];
            r1[nt * 8] = acc[nt][2]; r1[nt * 8 + 1] = acc[nt][3];
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < 16 * NP; idx += kThreads) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) s += S.red[(size_t)w * 16 * NP + idx];
            S.accbuf[(size_t)tile * 16 * NP + idx] += s;
        }
        __syncthreads();
    }
}

// fp32 weights: one warp per weight row, 128-bit loads, fp32 FMA, activations of 8 tokens in shared memory.
__device__ void gemv_rows_f32(const GemvJob &J, int ub, int nu, int kc0, int kc, const GemvSmem &S, int ldx) {
    constexpr int NP = 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float *xs = reinterpret_cast<const float *>(S.xs);
    const int narows = J.epi == EPI_GATEUP ? ((nu + 7) / 8) * 16 : nu;
    for (int r = warp; r < narows; r += kWarps) {
        const float *row = arow_ptr<float>(J, ub, nu, r, false);
        if (row == nullptr) continue;
        row += kc0;
        float acc[NP];
#pragma unroll
        for (int n = 0; n < NP; ++n) acc[n] = 0.f;
        for (int k = lane * 4; k < kc; k += 128) {
            uint4 wu = ldnc_u4(row + k);
            float w0 = __uint_as_float(wu.x), w1 = __uint_as_float(wu.y), w2 = __uint_as_float(wu.z),
                  w3 = __uint_as_float(wu.w);
#pragma unroll
            for (int n = 0; n < NP; ++n) {
                float4 x = *reinterpret_cast<const float4 *>(xs + (size_t)n * ldx + k);
                acc[n] = fmaf(w0, x.x, acc[n]);
                acc[n] = fmaf(w1, x.y, acc[n]);
                acc[n] = fmaf(w2, x.z, acc[n]);
                acc[n] = fmaf(w3, x.w, acc[n]);
            }
        }
#pragma unroll
        for (int n = 0; n < NP; ++n) acc[n] = warp_sum(acc[n]);
        if (lane == 0) {
#pragma unroll
            for (int n = 0; n < NP; ++n) S.accbuf[(size_t)r * NP + n] += acc[n];
        }
    }
}

template <typename WT> struct StageFmt;
template <> struct StageFmt<bf16> {
    static __device__ int ldx(int kc) { return kc + 32; }                   // row stride = 64 (mod 128) bytes
    static __device__ int bytes_per_token(int kc) { return (kc + 32) * 4; } // hi and lo planes
};
template <> struct StageFmt<float> {
    static __device__ int ldx(int kc) { return kc + 4; }
    static __device__ int bytes_per_token(int kc) { return (kc + 4) * 4; }
};

// rows [lo, hi) of one job
template <typename WT>
__device__ void gemv_job(const Dev &D, const GemvJob &J, int lo, int hi, char *smem) {
    const GemvSmem S = carve_gemv(smem);
    const int M = D.M, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool is_bf16 = sizeof(WT) == 2;
    const int NP = !is_bf16 ? 8 : (M <= 8 ? 8 : (M <= 16 ? 16 : 32));
    const WT *gain = reinterpret_cast<const WT *>(J.gain);

    __syncthreads();
    if (gain != nullptr) {   // 1 / rms of every input row (each CTA computes it for itself)
        for (int m = warp; m < M; m += kWarps) {
            float ss = 0.f;
            for (int k = lane * 4; k < J.kdim; k += 128) {
                float4 v = __ldcg(reinterpret_cast<const float4 *>(J.x + (size_t)m * J.x_ld + k));
                ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
            }
            ss = warp_sum(ss);
            if (lane == 0) S.inv[m] = 1.0f / sqrtf(ss / (float)J.kdim + D.eps);
        }
    }
    // k chunk that fits the staging area
    int KC = S.xs_bytes / (NP * 4) - (is_bf16 ? 32 : 4);
    KC = KC >= 512 ? (KC / 512) * 512 : (KC / 32) * 32;
    const int upb = J.epi == EPI_GATEUP ? kUnitBlock / 2 : kUnitBlock;   // units per accumulator block
    __syncthreads();

    for (int ub = lo; ub < hi; ub += upb) {
        const int nu = min(upb, hi - ub);
        const int narows = J.epi == EPI_GATEUP ? ((nu + 7) / 8) * 16 : nu;
        for (int tok0 = 0; tok0 < M; tok0 += NP) {
            const int ntok = min(NP, M - tok0);
            for (int i = threadIdx.x; i < ((narows + 15) / 16) * 16 * NP; i += kThreads) S.accbuf[i] = 0.f;
            for (int kc0 = 0; kc0 < J.kdim; kc0 += KC) {
                const int kc = min(KC, J.kdim - kc0), ldx = StageFmt<WT>::ldx(kc);
                __syncthreads();
                // stage activations tok0.., columns kc0..kc0+kc (normalised when the job has a gain)
                for (int i = threadIdx.x; i < NP * (kc / 4); i += kThreads) {
                    const int n = i / (kc / 4), k = (i % (kc / 4)) * 4;
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (n < ntok) {
                        const int m = tok0 + n;
                        v = __ldcg(reinterpret_cast<const float4 *>(J.x + (size_t)m * J.x_ld + kc0 + k));
                        if (gain != nullptr) {
                            const float s = S.inv[m];
                            v.x = v.x * s * to_f(gain[kc0 + k]);
                            v.y = v.y * s * to_f(gain[kc0 + k + 1]);
                            v.z = v.z * s * to_f(gain[kc0 + k + 2]);
                            v.w = v.w * s * to_f(gain[kc0 + k + 3]);
                        }
                    }
                    if (is_bf16) {
                        unsigned short h[4], l[4];
                        split_bf16(v.x, h[0], l[0]); split_bf16(v.y, h[1], l[1]);
                        split_bf16(v.z, h[2], l[2]); split_bf16(v.w, h[3], l[3]);
                        unsigned short *xh = reinterpret_cast<unsigned short *>(S.xs) + (size_t)n * ldx + k;
                        unsigned short *xl = xh + (size_t)NP * ldx;
                        *reinterpret_cast<uint2 *>(xh) =
                            make_uint2((unsigned)h[0] | ((unsigned)h[1] << 16), (unsigned)h[2] | ((unsigned)h[3] << 16));
                        *reinterpret_cast<uint2 *>(xl) =
                            make_uint2((unsigned)l[0] | ((unsigned)l[1] << 16), (unsigned)l[2] | ((unsigned)l[3] << 16));
                    } else {
                        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(S.xs) + (size_t)n * ldx + k) = v;
                    }
                }
                __syncthreads();
                if (is_bf16) {
                    if (NP == 8) gemv_tiles_bf16<1>(J, ub, nu, kc0, kc, S, ldx);
                    else if (NP == 16) gemv_tiles_bf16<2>(J, ub, nu, kc0, kc, S, ldx);
                    else gemv_tiles_bf16<4>(J, ub, nu, kc0, kc, S, ldx);
                } else {
                    gemv_rows_f32(J, ub, nu, kc0, kc, S, ldx);
                }
            }
            __syncthreads();
            // epilogue
            for (int i = threadIdx.x; i < nu * ntok; i += kThreads) {
                const int ui = i / ntok, n = i % ntok, m = tok0 + n, u = ub + ui;
                float *o = J.out + (size_t)m * J.out_ld + u;
                if (J.epi == EPI_GATEUP) {
                    const int tile = ui >> 3, r = ui & 7;
                    const float vg = S.accbuf[(size_t)(tile * 16 + r) * NP + n];
                    const float vu = S.accbuf[(size_t)(tile * 16 + 8 + r) * NP + n];
                    __stcg(o, silu_f(vg) * vu);
                } else {
                    const float v = S.accbuf[(size_t)ui * NP + n];
                    if (J.epi == EPI_STORE) __stcg(o, v);
                    else if (J.epi == EPI_ADD) __stcg(o, __ldcg(o) + v);
                    else {   // EPI_HEADY: residual on the normalised input
                        const float xg = __ldcg(J.x + (size_t)m * J.x_ld + u) * S.inv[m] * to_f(gain[u]);
                        __stcg(o, xg + silu_f(v));
                    }
                }
            }
            __syncthreads();
        }
    }
}

template <typename WT> __device__ void gemv_phase(const Dev &D, const Phase &ph, char *smem) {
    long long total = 0;
    for (int j = 0; j < ph.njobs; ++j) total += D.jobs[ph.job0 + j].rows;
    const long long u_lo = total * blockIdx.x / gridDim.x, u_hi = total * (blockIdx.x + 1) / gridDim.x;
    long long base = 0;
    for (int j = 0; j < ph.njobs; ++j) {
        const GemvJob &J = D.jobs[ph.job0 + j];
        const long long lo = max(u_lo - base, 0LL), hi = min(u_hi - base, (long long)J.rows);
        if (lo < hi) gemv_job<WT>(D, J, (int)lo, (int)hi, smem);
        base += J.rows;
    }
}

// -------------------------------------------------------------------------------- attention phases

constexpr int kQChunk = 8;   // query rows handled per pass over the keys

template <typename KVT>
__device__ __forceinline__ const KVT *kv_tile(const Dev &D, const void *pool, int pool_pages, int layer, int kv,
                                              int page, int head) {
    return reinterpret_cast<const KVT *>(pool) +
           ((((size_t)layer * 2 + kv) * pool_pages + page) * D.H + head) * (size_t)D.P * D.dh;
}

// One (sequence b, head h, split s of S) item.  Self-attention: K+1 window rows (positions len+j) against
// the cached keys 0..len-1 of this split's pages; the last split also takes the window's own keys
// (row j sees window keys 0..j) and appends them to the cache.  Cross-attention: the same rows against
// the n_cond cached condition keys, no mask, no rotation.  EPL = elements of a head row per lane.
template <typename KVT, int EPL>
__device__ void attn_item(const Dev &D, int layer, bool cross, int b, int h, int s, int S, char *smem_raw) {
    const int K1 = D.K1, dh = D.dh, P = D.P, d = D.d, half = dh / 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
    const int n = cross ? D.C : __ldcg(D.len + b);
    const int np = (n + P - 1) / P, pp = (np + S - 1) / S;
    const int key_lo = min(n, s * pp * P), key_hi = min(n, (s + 1) * pp * P);
    const bool win = !cross && s == S - 1;
    const float *qsrc = cross ? D.qc : D.qkv;
    const int q_ld = cross ? d : 3 * d;
    const void *pool = cross ? D.ckv_pool : D.kv_pool;
    const int pool_pages = cross ? D.B * D.cpages : D.n_pages;
    float *part = cross ? D.cpart : D.part;
    unsigned *ctr = cross ? D.cpart_ctr : D.part_ctr;
    float *out = cross ? D.cattn : D.attn;

    float *qs = reinterpret_cast<float *>(smem_raw);      // [K1][dh]  rotated, scaled queries
    float *kw = qs + K1 * dh;                             // [K1][dh]  window keys (rotated)
    float *vw = kw + K1 * dh;                             // [K1][dh]  window values
    float *st = vw + K1 * dh;                             // [kWarps][kQChunk][dh + 2]
    __shared__ int last_s;

    __syncthreads();
    for (int i = tid; i < K1 * dh; i += kThreads) {
        const int j = i / dh, e = i % dh, row = b * K1 + j;
        const float *qr = qsrc + (size_t)row * q_ld + h * dh;
        float v = __ldcg(qr + e);
        if (!cross) {
            const float2 cs = __ldcg(D.rope_cs + (size_t)row * half + (e % half));
            const float o = __ldcg(qr + (e < half ? e + half : e - half));
            v = e < half ? v * cs.x - o * cs.y : o * cs.y + v * cs.x;
        }
        qs[i] = v * D.scale;
        if (win) {
            const float *kr = qr + d, *vr = qr + 2 * d;
            float kv = __ldcg(kr + e);
            const float2 cs = __ldcg(D.rope_cs + (size_t)row * half + (e % half));
            const float ko = __ldcg(kr + (e < half ? e + half : e - half));
            kv = e < half ? kv * cs.x - ko * cs.y : ko * cs.y + kv * cs.x;
            const float vv = __ldcg(vr + e);
            kw[i] = kv;
            vw[i] = vv;
            // append to the cache at position len + j
            const int pos = n + j, page = __ldcg(D.block_table + (size_t)b * D.max_blocks + pos / P);
            KVT *kt = const_cast<KVT *>(kv_tile<KVT>(D, pool, pool_pages, layer, 0, page, h)) + (size_t)(pos % P) * dh;
            KVT *vt = const_cast<KVT *>(kv_tile<KVT>(D, pool, pool_pages, layer, 1, page, h)) + (size_t)(pos % P) * dh;
            kt[e] = from_f<KVT>(kv);
            vt[e] = from_f<KVT>(vv);
        }
    }
    __syncthreads();

    const int e0 = lane * EPL;
    const bool lane_on = e0 < dh;
    for (int j0 = 0; j0 < K1; j0 += kQChunk) {
        const int nq = min(kQChunk, K1 - j0);
        float q[kQChunk][EPL], acc[kQChunk][EPL], mx[kQChunk], l[kQChunk];
#pragma unroll
        for (int j = 0; j < kQChunk; ++j) {
            mx[j] = -INFINITY;
            l[j] = 0.f;
#pragma unroll
            for (int i = 0; i < EPL; ++i) {
                acc[j][i] = 0.f;
                q[j][i] = (j < nq && lane_on) ? qs[(j0 + j) * dh + e0 + i] : 0.f;
            }
        }
        // cached keys of this split, one key per warp at a time
        for (int key = key_lo + warp; key < key_hi; key += kWarps) {
            const int page = cross ? b * D.cpages + key / P : __ldcg(D.block_table + (size_t)b * D.max_blocks + key / P);
            const KVT *kt = kv_tile<KVT>(D, pool, pool_pages, layer, 0, page, h) + (size_t)(key % P) * dh + e0;
            const KVT *vt = kv_tile<KVT>(D, pool, pool_pages, layer, 1, page, h) + (size_t)(key % P) * dh + e0;
            float kf[EPL], vf[EPL];
#pragma unroll
            for (int i = 0; i < EPL; ++i) {
                kf[i] = lane_on ? ldcg_as_f<KVT>(kt + i) : 0.f;
                vf[i] = lane_on ? ldcg_as_f<KVT>(vt + i) : 0.f;
            }
#pragma unroll
            for (int j = 0; j < kQChunk; ++j) {
                if (j < nq) {
                    float dsum = 0.f;
#pragma unroll
                    for (int i = 0; i < EPL; ++i) dsum = fmaf(q[j][i], kf[i], dsum);
                    dsum = warp_sum(dsum);
                    const float mn = fmaxf(mx[j], dsum), corr = expf(mx[j] - mn), p = expf(dsum - mn);
                    l[j] = l[j] * corr + p;
#pragma unroll
                    for (int i = 0; i < EPL; ++i) acc[j][i] = acc[j][i] * corr + p * vf[i];
                    mx[j] = mn;
                }
            }
        }
        // the window's own keys, under the causal mask
        if (win) {
            for (int wk = warp; wk < K1; wk += kWarps) {
                float kf[EPL], vf[EPL];
#pragma unroll
                for (int i = 0; i < EPL; ++i) {
                    kf[i] = lane_on ? kw[wk * dh + e0 + i] : 0.f;
                    vf[i] = lane_on ? vw[wk * dh + e0 + i] : 0.f;
                }
#pragma unroll
                for (int j = 0; j < kQChunk; ++j) {
                    if (j < nq && wk <= j0 + j) {
                        float dsum = 0.f;
#pragma unroll
                        for (int i = 0; i < EPL; ++i) dsum = fmaf(q[j][i], kf[i], dsum);
                        dsum = warp_sum(dsum);
                        const float mn = fmaxf(mx[j], dsum), corr = expf(mx[j] - mn), p = expf(dsum - mn);
                        l[j] = l[j] * corr + p;
#pragma unroll
                        for (int i = 0; i < EPL; ++i) acc[j][i] = acc[j][i] * corr + p * vf[i];
                        mx[j] = mn;
                    }
                }
            }
        }
        // per-warp states -> shared memory
#pragma unroll
        for (int j = 0; j < kQChunk; ++j) {
            float *sw = st + ((size_t)warp * kQChunk + j) * (dh + 2);
            if (lane_on) {
#pragma unroll
                for (int i = 0; i < EPL; ++i) sw[e0 + i] = acc[j][i];
            }
            if (lane == 0) { sw[dh] = mx[j]; sw[dh + 1] = l[j]; }
        }
        __syncthreads();
        // merge the warps: one thread per (query, element)
        for (int i = tid; i < nq * (dh + 1); i += kThreads) {
            const int j = i / (dh + 1), e = i % (dh + 1);   // e == dh: the denominator
            float m = -INFINITY;
            for (int w = 0; w < kWarps; ++w) m = fmaxf(m, st[((size_t)w * kQChunk + j) * (dh + 2) + dh]);
            float o = 0.f;
            for (int w = 0; w < kWarps; ++w) {
                const float *sw = st + ((size_t)w * kQChunk + j) * (dh + 2);
                const float wgt = sw[dh] == -INFINITY ? 0.f : expf(sw[dh] - m);
                o += wgt * (e < dh ? sw[e] : sw[dh + 1]);
            }
            const int row = b * K1 + j0 + j;
            if (S == 1) {
                // denominators are summed by the e == dh thread; normalise after the sync below
                st[(size_t)kWarps * kQChunk * (dh + 2) + j * (dh + 2) + e] = o;
            } else {
                float *pr = part + (((size_t)(b * D.H + h) * S + s) * K1 + (j0 + j)) * (dh + 2);
                __stcg(pr + (e < dh ? e : dh + 1), o);
                if (e == dh) __stcg(pr + dh, m);
            }
            (void)row;
        }
        __syncthreads();
        if (S == 1) {
            const float *mg = st + (size_t)kWarps * kQChunk * (dh + 2);
            for (int i = tid; i < nq * dh; i += kThreads) {
                const int j = i / dh, e = i % dh;
                __stcg(out + (size_t)(b * K1 + j0 + j) * d + h * dh + e, mg[j * (dh + 2) + e] / mg[j * (dh + 2) + dh]);
            }
            __syncthreads();
        }
    }
    if (S > 1) {
        // the last split to arrive merges all of them
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned old = atomicAdd(ctr + b * D.H + h, 1u);
            last_s = old == (unsigned)(S - 1);
            if (last_s) atomicExch(ctr + b * D.H + h, 0u);
            __threadfence();
        }
        __syncthreads();
        if (last_s) {
            for (int i = tid; i < K1 * dh; i += kThreads) {
                const int j = i / dh, e = i % dh;
                const float *pb = part + (((size_t)(b * D.H + h) * S) * K1 + j) * (dh + 2);
                const size_t sstride = (size_t)K1 * (dh + 2);
                float m = -INFINITY;
                for (int ss = 0; ss < S; ++ss) m = fmaxf(m, __ldcg(pb + ss * sstride + dh));
                float o = 0.f, den = 0.f;
                for (int ss = 0; ss < S; ++ss) {
                    const float ms = __ldcg(pb + ss * sstride + dh);
                    const float wgt = ms == -INFINITY ? 0.f : expf(ms - m);
                    o += wgt * __ldcg(pb + ss * sstride + e);
                    den += wgt * __ldcg(pb + ss * sstride + dh + 1);
                }
                __stcg(out + (size_t)(b * K1 + j) * d + h * dh + e, o / den);
            }
        }
        __syncthreads();
    }
}

template <typename KVT> __device__ void attn_phase(const Dev &D, const Phase &ph, char *smem) {
    const bool cross = ph.kind == PH_ATTN_CROSS;
    const int S = cross ? D.S_cross : D.S_self;
    const int items = D.B * D.H * S;
    for (int it = blockIdx.x; it < items; it += gridDim.x) {
        const int s = it % S, h = (it / S) % D.H, b = it / (S * D.H);
        if (__ldcg(D.finished + b)) continue;
        if (D.dh <= 32) attn_item<KVT, 1>(D, ph.layer, cross, b, h, s, S, smem);
        else if (D.dh <= 64) attn_item<KVT, 2>(D, ph.layer, cross, b, h, s, S, smem);
        else attn_item<KVT, 4>(D, ph.layer, cross, b, h, s, S, smem);
    }
}

// ----------------------------------------------------------------- verify / accept length / resample

// is (va, ia) ranked before (vb, ib): larger logit first, then smaller index
__device__ __forceinline__ bool ranked_before(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

__device__ float block_sum(float v, float *sh) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    float s = 0.f;
    for (int w = 0; w < kWarps; ++w) s += sh[w];
    return s;
}
__device__ float block_max(float v, float *sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    float s = -INFINITY;
    for (int w = 0; w < kWarps; ++w) s = fmaxf(s, sh[w]);
    return s;
}
// best (value, index) over the block under ranked_before; threads without a candidate pass idx = INT_MAX
__device__ void block_best(float &v, int &idx, float *shv, int *shi) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, v, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (oi != 0x7fffffff && (idx == 0x7fffffff || ranked_before(ov, oi, v, idx))) { v = ov; idx = oi; }
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { shv[threadIdx.x >> 5] = v; shi[threadIdx.x >> 5] = idx; }
    __syncthreads();
    v = shv[0]; idx = shi[0];
    for (int w = 1; w < kWarps; ++w)
        if (shi[w] != 0x7fffffff && (idx == 0x7fffffff || ranked_before(shv[w], shi[w], v, idx))) { v = shv[w]; idx = shi[w]; }
}

// acceptance of token x under backbone logits z (global), block-wide; every thread returns the same answer
__device__ bool accept_token(const Dev &D, const float *z, int x, float *sh) {
    const int V = D.V;
    if (x < 0 || x >= V) return false;
    if (D.verify_mode == 2) {     // p0(x) > delta
        float m = -INFINITY;
        for (int v = threadIdx.x; v < V; v += kThreads) m = fmaxf(m, __ldcg(z + v));
        m = block_max(m, sh);
        float sum = 0.f;
        for (int v = threadIdx.x; v < V; v += kThreads) sum += expf(__ldcg(z + v) - m);
        sum = block_sum(sum, sh);
        return expf(__ldcg(z + x) - m) / sum > D.delta;
    }
    const int ka = D.verify_mode == 0 ? 1 : D.k_accept;
    const float zx = __ldcg(z + x);
    float cnt = 0.f;
    for (int v = threadIdx.x; v < V; v += kThreads)
        if (v != x && ranked_before(__ldcg(z + v), v, zx, x)) cnt += 1.f;
    cnt = block_sum(cnt, sh);
    return (int)cnt < ka;
}

__device__ int sample_token(const Dev &D, const float *z, uint32_t r24, float *sh, char *smem) {
    const int V = D.V;
    float *shv = sh;
    int *shi = reinterpret_cast<int *>(sh + kWarps);
    float *cv = sh + 2 * kWarps;                       // candidates (value, index), up to 64
    int *ci = reinterpret_cast<int *>(cv + 64);
    __shared__ int pick_s;
    const int k = D.sample_mode == 0 ? 1 : min(max(D.k_sample, 1), min(V, 64));
    float pv = INFINITY;
    int pi = -1;
    (void)smem;
    for (int j = 0; j < k; ++j) {      // j-th candidate: best among those ranked after the previous one
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int v = threadIdx.x; v < V; v += kThreads) {
            const float zv = __ldcg(z + v);
            if (j > 0 && !ranked_before(pv, pi, zv, v)) continue;
            if (bi == 0x7fffffff || ranked_before(zv, v, bv, bi)) { bv = zv; bi = v; }
        }
        block_best(bv, bi, shv, shi);
        if (threadIdx.x == 0) { cv[j] = bv; ci[j] = bi; }
        pv = bv; pi = bi;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int pick = ci[0];
        if (D.sample_mode != 0) {
            float total = 0.f, w[64];
            for (int j = 0; j < k; ++j) { w[j] = expf((cv[j] - cv[0]) / D.temperature); total += w[j]; }
            const float u = (float)r24 * (1.0f / 16777216.0f);
            float cum = 0.f;
            pick = ci[k - 1];
            for (int j = 0; j < k; ++j) {
                cum += w[j];
                if (cum > u * total) { pick = ci[j]; break; }
            }
        }
        pick_s = pick;
    }
    __syncthreads();
    return pick_s;
}

// item (sequence b, slot): slot 0 resamples x_{s*} from the backbone row of the first rejection, slot i
// from head i's logits of the same row (independent sampling).  Every item recomputes the accept length.
__device__ void sample_phase(const Dev &D, char *smem) {
    float *sh = reinterpret_cast<float *>(smem);
    const int K1 = D.K1, K = D.K, V = D.V;
    for (int it = blockIdx.x; it < D.B * K1; it += gridDim.x) {
        const int b = it / K1, slot = it % K1;
        if (__ldcg(D.finished + b) || __ldcg(D.ingest_left + b) > 0) continue;
        int a = 0;
        while (a < K) {
            const int x = __ldcg(D.window + b * K1 + a + 1);
            if (!accept_token(D, D.logits0 + (size_t)(b * K1 + a) * V, x, sh)) break;
            ++a;
        }
        const float *z = slot == 0 ? D.logits0 + (size_t)(b * K1 + a) * V
                                   : D.hlogits + ((size_t)(slot - 1) * D.M + b * K1 + a) * V;
        const uint32_t r = rand24(D, b, __ldcg(D.step_idx + b), (uint32_t)slot, 0u);
        const int tok = sample_token(D, z, r, sh, smem);
        if (threadIdx.x == 0) {
            __stcg(D.cand + b * K1 + slot, tok);
            if (slot == 0) __stcg(D.acc_len + b, a);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------- commit / next window

// After len[b] and window[b][*] are final: reserve cache pages for positions < len + K + 1, gather the
// embeddings of the window into h, and tabulate cos/sin of the window rows' positions.
template <typename WT> __device__ void prepare_window(const Dev &D, int b) {
    const int K1 = D.K1, d = D.d, half = D.dh / 2;
    __shared__ int s_len;
    if (threadIdx.x == 0) {
        const int len = __ldcg(D.len + b);
        s_len = len;
        const int need = (len + K1 + D.P - 1) / D.P;
        int nb = __ldcg(D.n_blocks + b);
        while (nb < need) {
            const int idx = atomicSub(D.n_free, 1) - 1;
            if (idx < 0 || nb >= D.max_blocks) {
                atomicAdd(D.n_free, 1);
                atomicExch(D.status, XSM_STATUS_CAPACITY);
                break;
            }
            __stcg(D.block_table + (size_t)b * D.max_blocks + nb, __ldcg(D.free_stack + idx));
            ++nb;
        }
        __stcg(D.n_blocks + b, nb);
    }
    __syncthreads();
    const WT *E = reinterpret_cast<const WT *>(D.E);
    for (int i = threadIdx.x; i < K1 * d; i += kThreads) {
        const int j = i / d, e = i % d;
        int tok = __ldcg(D.window + b * K1 + j);
        tok = min(max(tok, 0), D.V - 1);
        __stcg(D.h + (size_t)(b * K1 + j) * d + e, to_f(E[(size_t)tok * d + e]));
    }
    for (int i = threadIdx.x; i < K1 * half; i += kThreads) {
        const int j = i / half, f = i % half;
        double sn, cs;
        sincos((double)(s_len + j) * D.inv_freq[f], &sn, &cs);
        __stcg(D.rope_cs + (size_t)(b * K1 + j) * half + f, make_float2((float)cs, (float)sn));
    }
    __syncthreads();
}

__device__ void draw_initial_drafts(const Dev &D, int b) {
    for (int i = 1; i <= D.K; ++i) {
        const unsigned long long m = rand24(D, b, 0u, (uint32_t)i, 1u);
        __stcg(D.window + b * D.K1 + i, (int)((m * (unsigned long long)D.V) >> 24));
    }
}

// Algorithm 1 line 12 and the loop guard: commit x_{s+1..s*}, s <- s*, next window <- candidates.
template <typename WT> __device__ void commit_phase(const Dev &D) {
    const int K1 = D.K1;
    for (int b = blockIdx.x; b < D.B; b += gridDim.x) {
        if (__ldcg(D.finished + b)) {
            if (threadIdx.x == 0) __stcg(D.step_n_new + b, 0);
            continue;
        }
        if (threadIdx.x == 0) {
            int len = __ldcg(D.len + b);
            const int left = __ldcg(D.ingest_left + b);
            if (left > 0) {
                // prompt ingestion: the window held prompt tokens; all of them that are prompt enter the cache
                const int n = min(K1, left);
                len += n;
                __stcg(D.len + b, len);
                __stcg(D.ingest_left + b, left - n);
                __stcg(D.step_n_new + b, 0);
                const int *pr = D.prompt + (size_t)b * D.prompt_len;
                if (left - n > 0) {
                    for (int j = 0; j < K1; ++j) __stcg(D.window + b * K1 + j, len + j < D.prompt_len ? pr[len + j] : 0);
                } else {
                    __stcg(D.window + b * K1, pr[D.prompt_len - 1]);
                    draw_initial_drafts(D, b);
                }
            } else {
                const int a = __ldcg(D.acc_len + b);
                int n_gen = __ldcg(D.n_gen + b), fin = 0, n_out = 0;
                for (int j = 0; j <= a; ++j) {
                    const int tok = j < a ? __ldcg(D.window + b * K1 + j + 1) : __ldcg(D.cand + b * K1);
                    if (n_gen >= D.max_new) break;
                    __stcg(D.tok_log + (size_t)b * D.tok_ld + n_gen, tok);
                    __stcg(D.step_tokens + b * K1 + n_out, tok);
                    ++n_gen; ++n_out;
                    if (D.eos >= 0 && tok == D.eos) { fin = 1; break; }
                }
                for (int j = n_out; j < K1; ++j) __stcg(D.step_tokens + b * K1 + j, -1);
                __stcg(D.step_n_new + b, n_out);
                len += a + 1;
                if (n_gen >= D.max_new || len > D.max_seq_len) fin = 1;
                __stcg(D.len + b, len);
                __stcg(D.n_gen + b, n_gen);
                for (int j = 0; j < K1; ++j) __stcg(D.window + b * K1 + j, __ldcg(D.cand + b * K1 + j));
                __stcg(D.step_idx + b, __ldcg(D.step_idx + b) + 1u);
                D.hist[(size_t)b * (kMaxDraft + 1) + a] += 1ull;
                D.steps[b] += 1ull;
                if (fin) {
                    __stcg(D.finished + b, 1);
                    atomicSub(D.n_active, 1);
                }
            }
            __threadfence();
        }
        __syncthreads();
        if (!__ldcg(D.finished + b)) prepare_window<WT>(D, b);
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------ step kernel

template <typename WT>
__global__ void __launch_bounds__(kThreads, 1)
step_kernel(const __grid_constant__ Dev D, int ph_lo, int ph_hi, int n_steps, int use_barrier) {
    extern __shared__ __align__(128) char smem[];
    unsigned epoch = 0;
    for (int t = 0; t < n_steps; ++t) {
        if (__ldcg(D.n_active) <= 0) break;
        for (int p = ph_lo; p < ph_hi; ++p) {
            const Phase ph = D.phases[p];
            switch (ph.kind) {
                case PH_GEMV: gemv_phase<WT>(D, ph, smem); break;
                case PH_ATTN_SELF:
                case PH_ATTN_CROSS: attn_phase<WT>(D, ph, smem); break;
                case PH_SAMPLE: sample_phase(D, smem); break;
                case PH_COMMIT: commit_phase<WT>(D); break;
            }
            if (use_barrier && !grid_barrier(D, epoch)) return;
        }
    }
}

cudaError_t step_kernel_setup(int dtype, int *max_grid) {
    cudaError_t e;
    const void *fn = dtype == 1 ? (const void *)step_kernel<bf16> : (const void *)step_kernel<float>;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0, per_sm = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, kSmemBytes);
    if (e != cudaSuccess) return e;
    *max_grid = per_sm >= 1 ? sms : 0;
    return cudaSuccess;
}

cudaError_t launch_step(const Dev &D, int dtype, int ph_lo, int ph_hi, int n_steps, int barrier, int grid,
                        cudaStream_t st) {
    const void *fn = dtype == 1 ? (const void *)step_kernel<bf16> : (const void *)step_kernel<float>;
    void *args[] = {(void *)&D, &ph_lo, &ph_hi, &n_steps, &barrier};
    if (barrier) {
        cudaError_t e = cudaMemsetAsync(D.bar, 0, sizeof(unsigned), st);
        if (e != cudaSuccess) return e;
        return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kThreads), args, kSmemBytes, st);
    }
    return cudaLaunchKernel(fn, dim3(grid), dim3(kThreads), args, kSmemBytes, st);
}

// ------------------------------------------------------------------------------- prefill kernels

// Cross-attention keys and values of the condition (computed once per mesh):
// out[c][r] = sum_k W[r][k] * cond[b][c][k], stored as cache tiles [page][head][slot][dh].
template <typename WT>
__global__ void __launch_bounds__(256) cross_kv_kernel(const Dev D, const WT *Wall, const size_t *wkc_off,
                                                       const size_t *wvc_off, const WT *cond) {
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
    WT *pool = reinterpret_cast<WT *>(D.ckv_pool);
    for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + ty * 4 + i, r = r0 + tx * 4 + j;
            if (c < D.C && r < D.d) {
                const int page = b * D.cpages + c / D.P, head = r / D.dh, e = r % D.dh;
                const size_t o = (((((size_t)layer * 2 + kv) * (D.B * D.cpages) + page) * D.H + head) * D.P + c % D.P) * D.dh + e;
                pool[o] = from_f<WT>(acc[i][j]);
            }
        }
}

cudaError_t launch_cross_kv(const Dev &D, int dtype, const void *W, const size_t *wkc_off, const size_t *wvc_off,
                            const void *cond, cudaStream_t st) {
    dim3 grid((D.C + 63) / 64, (D.d + 63) / 64, D.L * 2 * D.B);
    if (dtype == 1)
        cross_kv_kernel<bf16><<<grid, 256, 0, st>>>(D, (const bf16 *)W, wkc_off, wvc_off, (const bf16 *)cond);
    else
        cross_kv_kernel<float><<<grid, 256, 0, st>>>(D, (const float *)W, wkc_off, wvc_off, (const float *)cond);
    return cudaGetLastError();
}

// Algorithm 1 line 1: pool reset, then per-sequence state, first window and its pages.
__global__ void init_pool_kernel(const Dev D) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < D.n_pages) D.free_stack[i] = D.n_pages - 1 - i;
    if (i < D.B * D.H) { D.part_ctr[i] = 0u; D.cpart_ctr[i] = 0u; }
    if (i == 0) { *D.n_free = D.n_pages; *D.n_active = D.B; *D.status = 0; *D.bar = 0u; }
}

template <typename WT> __global__ void __launch_bounds__(kThreads) init_seq_kernel(const Dev D) {
    const int b = blockIdx.x, K1 = D.K1;
    if (threadIdx.x == 0) {
        D.len[b] = 0; D.finished[b] = 0; D.n_gen[b] = 0; D.n_blocks[b] = 0; D.step_idx[b] = 0u;
        D.acc_len[b] = 0; D.steps[b] = 0ull; D.step_n_new[b] = 0;
        for (int a = 0; a <= kMaxDraft; ++a) D.hist[(size_t)b * (kMaxDraft + 1) + a] = 0ull;
        const int *pr = D.prompt + (size_t)b * D.prompt_len;
        D.ingest_left[b] = D.prompt_len - 1;
        if (D.prompt_len == 1) {
            D.window[b * K1] = pr[0];
            draw_initial_drafts(D, b);
        } else {
            for (int j = 0; j < K1; ++j) D.window[b * K1 + j] = j < D.prompt_len ? pr[j] : 0;
        }
        __threadfence();
    }
    __syncthreads();
    prepare_window<WT>(D, b);
}

cudaError_t launch_init(const Dev &D, int dtype, cudaStream_t st) {
    const int n = max(D.n_pages, max(D.B * D.H, 1));
    init_pool_kernel<<<(n + 255) / 256, 256, 0, st>>>(D);
    if (dtype == 1) init_seq_kernel<bf16><<<D.B, kThreads, 0, st>>>(D);
    else init_seq_kernel<float><<<D.B, kThreads, 0, st>>>(D);
    return cudaGetLastError();
}

// re-gather the window embeddings after the drafts were replaced from outside
template <typename WT> __global__ void __launch_bounds__(kThreads) embed_kernel(const Dev D) {
    if (!D.finished[blockIdx.x]) prepare_window<WT>(D, blockIdx.x);
}
cudaError_t launch_embed(const Dev &D, int dtype, cudaStream_t st) {
    if (dtype == 1) embed_kernel<bf16><<<D.B, kThreads, 0, st>>>(D);
    else embed_kernel<float><<<D.B, kThreads, 0, st>>>(D);
    return cudaGetLastError();
}

template <typename KVT>
__global__ void gather_kv_kernel(const Dev D, int layer, int seq, int pos0, int n, float *out_k, float *out_v) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * D.d) return;
    const int p = pos0 + i / D.d, r = i % D.d, head = r / D.dh, e = r % D.dh;
    const int page = D.block_table[(size_t)seq * D.max_blocks + p / D.P];
    const KVT *kt = kv_tile<KVT>(D, D.kv_pool, D.n_pages, layer, 0, page, head) + (size_t)(p % D.P) * D.dh + e;
    const KVT *vt = kv_tile<KVT>(D, D.kv_pool, D.n_pages, layer, 1, page, head) + (size_t)(p % D.P) * D.dh + e;
    out_k[i] = to_f(*kt);
    out_v[i] = to_f(*vt);
}
cudaError_t launch_gather_kv(const Dev &D, int dtype, int layer, int seq, int pos0, int n, float *out_k,
                             float *out_v, cudaStream_t st) {
    const int total = n * D.d;
    if (dtype == 1) gather_kv_kernel<bf16><<<(total + 255) / 256, 256, 0, st>>>(D, layer, seq, pos0, n, out_k, out_v);
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
