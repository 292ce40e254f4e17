// Kernels of the speculative decoding step (Algorithm 1, lines 3-12) for sm_100a.
//
// One decoding step is a fixed list of stages (projection, attention, ..., verify/resample, commit).  The
// step kernel is persistent: one CTA per SM walks the whole list, and a launch may run many steps.
//
//  * Streaming.  Every byte that must come from HBM in a step (weight rows, cached keys and values, the
//    condition's keys and values) has an address that is known when the step starts.  A producer warp walks
//    the CTA's share of the step in order and pulls it into a ring of shared-memory slots with bulk copies
//    (cp.async.bulk, completion on an mbarrier); seven consumer warps compute out of the ring.  HBM stays
//    busy while the consumers wait for activations of the previous stage.
//  * Exchange.  Activations travel between CTAs as fp32 words in global memory whose two lowest mantissa
//    bits carry a tag that cycles with the write index of the buffer.  A consumer spins on the words it
//    needs until they carry the expected tag: data and flag arrive in one L2 round trip, and no grid
//    barrier exists.  A word is reused only after every reader of its previous content has produced data
//    that the next writer has itself consumed (every CTA owns rows of every projection), so one copy of
//    each buffer is enough.
//  * Arithmetic.  bf16 weights: mma.sync.m16n8k16 with weight rows on M and the token rows on N, the
//    fp32 activations split into bf16 hi + lo so that nothing that matters is lost; fp32 accumulation.
//    fp32 weights: FMA.  Attention over the 16-bit cache (fp16 elements): flash-decoding with mma.sync,
//    queries as fp16 hi + lo pairs, base-2 online softmax, splits over keys merged by the last split.
//  * Every wait is bounded.  When one runs out the CTA raises the status word; every CTA that sees it stops
//    waiting on global memory, still drains its ring, and leaves at the end of the step.
#pragma once
#include "xsm_internal.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math.h>

#include <atomic>

namespace xsm {

typedef __nv_bfloat16 bf16;

constexpr int XSM_STATUS_TIMEOUT = 5, XSM_STATUS_CAPACITY = 3;
constexpr float kNegBig = -1.0e30f;            // "no key seen yet" (finite: tags must not turn it into a NaN)
constexpr float kLog2e = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------ helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint4 ld_relaxed_u4(const void *p) {
    uint4 r;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const void *p) {
    uint32_t r;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(r) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ void st_relaxed_u32(void *p, uint32_t v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint4 lds_u4(uint32_t a) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(a));
    return r;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// global -> shared bulk copy; bytes and both addresses are multiples of 16
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Timeline of the first step of a launch, when the host asked for one: row 0 = the step's start, rows
// 1 + 2p and 2 + 2p = stage p has its inputs / has published its outputs; one column per CTA.
__device__ __forceinline__ void trace_mark(const Dev &D, int row) {
    if (D.trace != nullptr && threadIdx.x == 0) D.trace[(size_t)row * gridDim.x + blockIdx.x] = global_ns();
}

// barrier among the consumer warps only (the producer warp never joins it)
__device__ __forceinline__ void csync() { asm volatile("bar.sync 1, %0;" :: "n"(kConsumerThreads) : "memory"); }

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f(__half v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f<__half>(float v) { return __float2half_rn(fminf(fmaxf(v, -65504.f), 65504.f)); }

// Element type of the key/value caches.  bf16 models keep them in fp16: the same two bytes, eleven bits of
// mantissa instead of eight (cached keys and values are normalised activations times small weights, far
// inside the fp16 range; stores saturate).  Rounding of the cache is the largest error of the whole path.
template <typename WT> struct CacheT { typedef WT type; };
template <> struct CacheT<bf16> { typedef __half type; };

__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + expf(-v)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// x = hi + lo with hi, lo bf16: 16 mantissa bits of x survive, products with bf16 weights stay exact in fp32.
__device__ __forceinline__ void split_bf16(float x, unsigned &hi, unsigned &lo) {
    bf16 h = __float2bfloat16_rn(x);
    bf16 l = __float2bfloat16_rn(x - __bfloat162float(h));
    hi = __bfloat16_as_ushort(h);
    lo = __bfloat16_as_ushort(l);
}
// 2^x for the online softmax (x <= 0 or -inf): the hardware approximation, 2 ulp
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// two values rounded to fp16, first in the low half
__device__ __forceinline__ unsigned pack_f16x2(float a, float b) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const unsigned *>(&h);
}
// x = hi + lo with hi, lo fp16 (operands of the attention products)
__device__ __forceinline__ void split_f16(float x, unsigned &hi, unsigned &lo) {
    const __half h = __float2half_rn(x);
    const __half l = __float2half_rn(x - __half2float(h));
    hi = __half_as_ushort(h);
    lo = __half_as_ushort(l);
}
// four values -> {hi01, hi23, lo01, lo23}
__device__ __forceinline__ uint4 split4(float a, float b, float c, float d) {
    unsigned h0, l0, h1, l1, h2, l2, h3, l3;
    split_bf16(a, h0, l0); split_bf16(b, h1, l1); split_bf16(c, h2, l2); split_bf16(d, h3, l3);
    return make_uint4(h0 | (h1 << 16), h2 | (h3 << 16), l0 | (l1 << 16), l2 | (l3 << 16));
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
__device__ __forceinline__ void mma16816_f16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                             unsigned b0, unsigned b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(unsigned (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
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

// ------------------------------------------------------------------------------------------- tags

__device__ __forceinline__ uint32_t tag_of(uint32_t serial, TagRef r) { return 1u + (serial * (uint32_t)r.wps + (uint32_t)r.j) % 3u; }
// the mantissa is rounded to 22 bits (to nearest, in magnitude) before the tag takes the two lowest bits
__device__ __forceinline__ uint32_t tagged(float v, uint32_t tag) { return ((__float_as_uint(v) + 2u) & ~3u) | tag; }
__device__ __forceinline__ float untag(uint32_t w) { return __uint_as_float(w & ~3u); }
__device__ __forceinline__ bool tags_ok(const uint4 &v, uint32_t tag) {
    return (((v.x ^ tag) | (v.y ^ tag) | (v.z ^ tag) | (v.w ^ tag)) & 3u) == 0u;
}
// integers travel as (value << 2) | tag
__device__ __forceinline__ uint32_t tagged_int(int v, uint32_t tag) { return ((uint32_t)v << 2) | tag; }
__device__ __forceinline__ int untag_int(uint32_t w) { return (int)(w >> 2); }

// bf16 models: an activation travels as one word, bits 31..16 = hi = bf16(x), bits 15..2 = the leading bits of
// lo = bf16(x - hi), bits 1..0 = tag (14 bits of mantissa survive; weights and cache have 8).  The reader gets
// the two MMA operands by byte permutation, without arithmetic.  fp32 models publish tagged fp32 words.
__device__ __forceinline__ uint32_t pack_act(float v, uint32_t tag) {
    const bf16 h = __float2bfloat16_rn(v);
    const bf16 l = __float2bfloat16_rn(v - __bfloat162float(h));
    return ((uint32_t)__bfloat16_as_ushort(h) << 16) | ((uint32_t)__bfloat16_as_ushort(l) & 0xFFFCu) | tag;
}
__device__ __forceinline__ float unpack_act(uint32_t w) {
    return __uint_as_float(w & 0xFFFF0000u) + __uint_as_float((w & 0xFFFCu) << 16);
}
template <typename WT> __device__ __forceinline__ uint32_t publish_word(float v, uint32_t tag, bool plain) {
    return (sizeof(WT) == 2 && !plain) ? pack_act(v, tag) : tagged(v, tag);
}
template <typename WT> __device__ __forceinline__ float read_word(uint32_t w) {
    return sizeof(WT) == 2 ? unpack_act(w) : untag(w);
}

// Per-CTA control block in shared memory (after the barriers).
struct Ctl {
    volatile int dead;          // a wait ran out somewhere: stop waiting on global memory
    volatile int dead_allowance;   // tries that the barrier waits of a dead CTA may still spend, all together
    int go;                     // written by the consumers before they release the producer for a step
    int trace_row;              // row of the timeline that the running stage fills when its inputs are in (0: off)
    int any_dead;               // some sequence of the batch has finished: row_dead has entries set
    volatile unsigned char landed[16];   // attention: number (modulo 4) of the latest fill of each ring slot that is known to have landed
    uint32_t tmem;              // tcgen05 path: base address of the CTA's accumulator columns in tensor memory
    volatile uint32_t umma_chunks, umma_tiles;   // tcgen05 path: column blocks and tiles multiplied since the launch (phases of abar, dbar)
    int len[kMaxBatch];
    int flags[kMaxBatch];       // 1 finished, 2 ingesting
    unsigned char row_dead[kMaxTokens];   // token rows of finished sequences (not fetched, read as zeros)
};

struct Smem {
    uint32_t full0, empty0, go_bar;   // shared-space addresses of full[0], empty[0], go
    uint32_t abar0, dbar, sbar0;      // tcgen05 path: "products that read activation buffer i are done" (two barriers), "the tile's accumulator is
                                      // complete", "activation buffer i is staged" (two barriers, one arrival per staging warp)
    Ctl *ctl;
    const Tables *tab;                // shared-memory copy of the stage and job tables
    struct SegRec *seg;               // per job: this CTA's rows and their tiling
    char *ring;
    char *acts;
    float *ss;                        // [kMaxTokens] sum of squares / 1 / rms
    float *sspart;                    // warp partial sums of squares of the chunk being staged
    int n_slots;
};


__device__ __forceinline__ Smem carve(char *smem, const Dev &D) {
    Smem s;
    s.full0 = smem_u32(smem);
    s.empty0 = s.full0 + 8u * kMaxSlots;
    s.go_bar = s.empty0 + 8u * kMaxSlots;
    s.abar0 = s.go_bar + 8u;
    s.dbar = s.abar0 + 16u;
    s.sbar0 = s.dbar + 8u;
    s.ctl = reinterpret_cast<Ctl *>(smem + 256);   // 2 * 12 * 8 + 8 + 40 = 240 bytes of barriers before it
    s.tab = reinterpret_cast<const Tables *>(smem + kSmemHeader);
    s.seg = reinterpret_cast<struct SegRec *>(smem + kSmemHeader + D.tab_bytes);
    s.ring = smem + kSmemHeader + D.tab_bytes + D.plan_bytes;
    s.n_slots = D.n_slots;
    s.acts = s.ring + (size_t)D.n_slots * kSlotBytes;
    s.ss = reinterpret_cast<float *>(s.acts + D.acts_bytes);
    s.sspart = s.ss + kMaxTokens;
    return s;
}
static_assert(256 + sizeof(Ctl) <= kSmemHeader, "control block overflows the header");

__device__ __forceinline__ void raise_timeout(const Dev &D, Ctl *ctl) {
    atomicExch(D.status, XSM_STATUS_TIMEOUT);
    ctl->dead = 1;
}

// A CTA's share of the sum of squares of row m of the published residual stream: [row][CTA]
__device__ __forceinline__ float *ss_word(const Dev &D, int cta, int m) { return D.sspub + (size_t)m * D.grid + cta; }

// Spins until the four words at p carry `tag`.  Gives up when the CTA is dead or the status word is raised.
__device__ __forceinline__ uint4 poll_u4(const Dev &D, Ctl *ctl, const void *p, uint32_t tag) {
    uint4 v = ld_relaxed_u4(p);
    unsigned it = 0;
    while (!tags_ok(v, tag)) {
        if (ctl->dead) break;
        if (++it > D.spin_limit) { raise_timeout(D, ctl); break; }
        if ((it & 1023u) == 0u && ld_relaxed_u32(D.status) != 0u) { ctl->dead = 1; break; }
        v = ld_relaxed_u4(p);
    }
    return v;
}
__device__ __forceinline__ uint32_t poll_u32(const Dev &D, Ctl *ctl, const void *p, uint32_t tag) {
    uint32_t v = ld_relaxed_u32(p);
    unsigned it = 0;
    while ((v & 3u) != tag) {
        if (ctl->dead) break;
        if (++it > D.spin_limit) { raise_timeout(D, ctl); break; }
        if ((it & 1023u) == 0u && ld_relaxed_u32(D.status) != 0u) { ctl->dead = 1; break; }
        v = ld_relaxed_u32(p);
    }
    return v;
}

// the same waits as calls, for places where the wait is rare and the code around it is unrolled many times (the code of a
// loop body should stay inside the instruction cache)
static __device__ __noinline__ uint4 poll_u4_cold(const Dev &D, Ctl *ctl, const void *p, uint32_t tag) { return poll_u4(D, ctl, p, tag); }
static __device__ __noinline__ uint32_t poll_u32_cold(const Dev &D, Ctl *ctl, const void *p, uint32_t tag) { return poll_u32(D, ctl, p, tag); }

// ------------------------------------------------------------------------------------------- ring

// A ring position is the slot (low byte) and the parity of the number of trips round the ring (bit 8): items passed so
// far, modulo twice the ring, kept in a form that needs no division.  Same sequence on the producer and on every
// consumer warp.
struct Ring {
    uint32_t pos;
};
__device__ __forceinline__ uint32_t ring_slot(const Smem &S, uint32_t pos) { return pos & 0xFFu; }
__device__ __forceinline__ uint32_t ring_parity(const Smem &S, uint32_t pos) { return (pos >> 8) & 1u; }
// the position k items further (k is at most a few rings)
__device__ __forceinline__ uint32_t ring_add(const Smem &S, uint32_t pos, int k) {
    uint32_t slot = (pos & 0xFFu) + (uint32_t)k, par = pos >> 8;
    while (slot >= (uint32_t)S.n_slots) { slot -= (uint32_t)S.n_slots; par ^= 1u; }
    return slot | (par << 8);
}

// A wait on a shared-memory barrier, bounded.  Once a wait has run out somewhere (ctl->dead) the CTA still tries to
// complete its ring protocol, but all its later waits together get one more allowance of tries, not one each.
__device__ __forceinline__ void mbar_wait(const Dev &D, Ctl *ctl, uint32_t bar, uint32_t parity) {
    for (unsigned it = 0; it < D.mbar_limit; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if ((it & 255u) == 255u && ctl->dead && atomicSub(const_cast<int *>(&ctl->dead_allowance), 256) <= 0) return;
    }
    raise_timeout(D, ctl);
}

// consumer: wait until the item at ring position r.pos has landed; returns its slot
__device__ __forceinline__ char *ring_wait(const Dev &D, const Smem &S, const Ring &r) {
    const uint32_t slot = ring_slot(S, r.pos);
    mbar_wait(D, S.ctl, S.full0 + 8u * slot, ring_parity(S, r.pos));
    return S.ring + (size_t)slot * kSlotBytes;
}
// consumer (whole warp): done with the item
__device__ __forceinline__ void ring_release(const Smem &S, Ring &r) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(S.empty0 + 8u * ring_slot(S, r.pos));
    r.pos = ring_add(S, r.pos, 1);
}
// producer (lane 0 decides, the warp follows): claim the next slot, announce `bytes`
__device__ __forceinline__ void ring_claim(const Dev &D, const Smem &S, const Ring &r, uint32_t bytes, uint32_t &dst,
                                           uint32_t &bar) {
    const uint32_t slot = ring_slot(S, r.pos);
    bar = S.full0 + 8u * slot;
    dst = smem_u32(S.ring + (size_t)slot * kSlotBytes);
    if ((threadIdx.x & 31) == 0) {
        mbar_wait(D, S.ctl, S.empty0 + 8u * slot, ring_parity(S, r.pos) ^ 1u);
        mbar_arrive_expect_tx(bar, bytes);
    }
    __syncwarp();
}

// ------------------------------------------------------------------------------------ tables

// stage p of the step: layers first (eight stages each), then the tail
__device__ __forceinline__ Stage stage_at(const Dev &D, const Smem &S, int p) {
    const int n_layer = kLayerStages * D.L;
    if (p < n_layer) {
        const int l = p / kLayerStages;
        Stage st = S.tab->stages[p - l * kLayerStages];
        st.layer = l;
        st.in.j += l * st.jinc; st.outt.j += l * st.jinc; st.part.j += l * st.jinc;
        return st;
    }
    Stage st = S.tab->stages[kLayerStages + p - n_layer];
    st.layer = -1;
    return st;
}
// job `idx` of a stage of layer `layer` (< 0: a job of the tail), by value: its fields then live in registers
__device__ __forceinline__ GemvJob job_at(const Dev &D, const Smem &S, int idx, int layer) {
    GemvJob J = S.tab->jobs[idx];
    if (layer > 0) {
        const long long off = S.tab->layer_bytes * layer;
        J.W = reinterpret_cast<const char *>(J.W) + off;
        if (J.W2 != nullptr) J.W2 = reinterpret_cast<const char *>(J.W2) + off;
        if (J.gain != nullptr) J.gain = reinterpret_cast<const char *>(J.gain) + off;
        if (J.gain_out != nullptr) J.gain_out = reinterpret_cast<const char *>(J.gain_out) + off;
        J.in.j += layer * J.in_jinc;
        J.outt.j += layer * J.out_jinc;
    }
    // the down projection's published copy carries the gain of the next layer's first RMSNorm, or the final one
    if (layer >= 0 && J.gain_out_step != 0) {
        if (layer == D.L - 1) J.gain_out = S.tab->gain_last;
        else J.gain_out = reinterpret_cast<const char *>(J.gain_out) + J.gain_out_step;
    }
    return J;
}

// ------------------------------------------------------------------------------ projection: plan

// The rows of a stage's jobs form one range that is cut evenly over the CTAs; a CTA's piece of one job is a
// segment.  A segment is processed as groups of tiles, the activations in chunks of D.kca columns.
// A tile has up to 16 layout rows (16 weight rows, or 8 gate rows then 8 up rows; 8 or 4 rows where a row is
// longer than 4 KB, so that a tile never exceeds four slots).  An item is `rpi` consecutive layout rows at full
// width: consecutive weight rows are contiguous in memory, so one bulk copy brings an item.  A tile group
// (`tpg` tiles at most) has all its items in the ring at once.
constexpr int kItemBytes = kSlotBytes;
struct SegPlan {
    int tile_units;   // units (output rows) per tile: 16, 8 or 4; 8 for gate/up
    int tu_shift;     // log2(tile_units)
    int tile_rows;    // layout rows per tile: tile_units, or 16 for gate/up
    int n_tiles;
    int rpi_shift;    // log2 of the layout rows per item (rows per item: 1, 2, 4 or 8)
    int ipt;          // items per tile
    int tpg;          // tiles per group = min(consumer warps, slots / ipt), at least 1
    int row_bytes;
};
struct SegRec { int lo, hi; SegPlan p; };    // rows [lo, hi) of the job belong to this CTA
static_assert(sizeof(SegRec) == kSegRecBytes, "size of a plan record");
// Projections of at most eight token rows whose activations fit the staging area at once (batch 1) take the path of
// consume_small: every warp multiplies all tiles of a group over its share of the columns.
constexpr int kSmallTiles = 4;        // tiles of a group on that path (their accumulators live in registers)
template <typename WT> __device__ __forceinline__ bool small_mode(const Dev &D, int kdim) {
    return sizeof(WT) == 2 && D.small;      // (decided by the host for all projections of the model at once)
}
template <typename WT> __device__ __forceinline__ SegPlan seg_plan(const Dev &D, const Smem &S, const GemvJob &J, int lo, int hi) {
    SegPlan p;
    p.row_bytes = J.kdim * (int)sizeof(WT);            // the host refuses rows beyond kItemBytes
    const int fit = kItemBytes / p.row_bytes;          // whole rows per item
    p.rpi_shift = fit >= 8 ? 3 : fit >= 4 ? 2 : fit >= 2 ? 1 : 0;
    if (J.epi == EPI_GATEUP) { p.tile_units = 8; p.tu_shift = 3; p.tile_rows = 16; }      // rows are d_model long: <= 4 KB
    else {
        p.tu_shift = p.row_bytes <= 4096 ? 4 : p.row_bytes <= 8192 ? 3 : 2;
        p.tile_units = p.tile_rows = 1 << p.tu_shift;
    }
    p.n_tiles = (hi - lo + p.tile_units - 1) / p.tile_units;
    p.ipt = max(1, p.tile_rows >> p.rpi_shift);
    p.tpg = max(1, min(kConsumerWarps, S.n_slots / p.ipt));
    if (small_mode<WT>(D, J.kdim)) {
        // the warps' partial products of a group sit behind the staged activations
        const int room = D.acts_bytes - D.M * (J.kdim * 4 + 16);
        p.tpg = max(1, min(min(kSmallTiles, p.tpg), room / (kConsumerWarps * kSmallRedBytes)));
    }
    return p;
}
// valid weight rows of item `it` of a tile that starts at unit u0 and has nu units, and where they come from
template <typename WT>
__device__ __forceinline__ int item_rows(const GemvJob &J, const SegPlan &p, int u0, int nu, int it, const WT *&src) {
    const int r0 = it << p.rpi_shift, rpi = 1 << p.rpi_shift;      // first layout row
    if (J.epi == EPI_GATEUP) {
        const int ui = r0 & 7;                                      // unit of the first row
        src = reinterpret_cast<const WT *>(r0 < 8 ? J.W : J.W2) + (size_t)(u0 + ui) * J.kdim;
        return min(max(nu - ui, 0), rpi);
    }
    src = reinterpret_cast<const WT *>(J.W) + (size_t)(u0 + r0) * J.kdim;
    return min(max(nu - r0, 0), rpi);
}

// ---------------------------------------------------------------------------- projection: producer

template <typename WT>
static __device__ void produce_segment(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R) {
    const SegPlan p = R.p;
    const int lo = R.lo, hi = R.hi;
    const int lane = threadIdx.x & 31;
    for (int tg0 = 0; tg0 < p.n_tiles; tg0 += p.tpg) {
        const int tg = min(p.tpg, p.n_tiles - tg0);
        for (int t = 0; t < tg; ++t) {
            const int u0 = lo + (tg0 + t) * p.tile_units, nu = min(p.tile_units, hi - u0);
            for (int it = 0; it < p.ipt; ++it) {
                const WT *src;
                const int nrows = item_rows<WT>(J, p, u0, nu, it, src);
                const uint32_t bytes = (uint32_t)(nrows * p.row_bytes);
                uint32_t dst, bar;
                ring_claim(D, S, ring, bytes, dst, bar);        // an item without valid rows is only announced
                if (lane == 0 && bytes != 0u) bulk_g2s(dst, src, bytes, bar);
                ring.pos = ring_add(S, ring.pos, 1);
            }
        }
    }
}

// ---- projections whose activations do not fit the staging area at once (many token rows, or very long rows).
// The activations are staged in chunks of D.kca columns, each chunk once per round of tiles, and the weights follow
// the same order: an item holds the columns of one chunk for `rpi` rows of one tile (one bulk copy per row).  A
// round is as many tiles as have their accumulators ([tile][token][16] floats) in kAccumBytes of shared memory.
__device__ __forceinline__ int chunk_tiles_per_round(const SegPlan &p, int M) {
    return max(1, min(p.n_tiles, kAccumBytes / (M * 64)));
}
// log2 of the rows of a tile that share one item when a row contributes seg_bytes (<= 4096) to it
__device__ __forceinline__ int chunk_rpi_shift(const SegPlan &p, int seg_bytes) {
    const int fit = min(kSlotBytes / seg_bytes, p.tile_rows);
    return fit >= 16 ? 4 : fit >= 8 ? 3 : fit >= 4 ? 2 : fit >= 2 ? 1 : 0;
}

template <typename WT>
static __device__ void produce_segment_chunked(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R) {
    const SegPlan p = R.p;
    const int lo = R.lo, hi = R.hi, lane = threadIdx.x & 31;
    const int tr = chunk_tiles_per_round(p, D.M);
    for (int r0 = 0; r0 < p.n_tiles; r0 += tr) {
        const int nr = min(tr, p.n_tiles - r0);
        for (int ac0 = 0; ac0 < J.kdim; ac0 += D.kca) {
            const int acw = min(D.kca, J.kdim - ac0), seg = acw * (int)sizeof(WT);
            const int sh = chunk_rpi_shift(p, seg), ipt = p.tile_rows >> sh;
            for (int tl = 0; tl < nr; ++tl) {
                const int u0 = lo + (r0 + tl) * p.tile_units, nu = min(p.tile_units, hi - u0);
                for (int it = 0; it < ipt; ++it) {
                    const int row = (it << sh) + lane;          // layout row of the tile that this lane copies
                    bool valid = lane < (1 << sh);
                    const WT *src;
                    if (J.epi == EPI_GATEUP) {
                        const int unit = row & 7;
                        valid = valid && unit < nu;
                        src = reinterpret_cast<const WT *>(row < 8 ? J.W : J.W2) + (size_t)(u0 + unit) * J.kdim + ac0;
                    } else {
                        valid = valid && row < nu;
                        src = reinterpret_cast<const WT *>(J.W) + (size_t)(u0 + row) * J.kdim + ac0;
                    }
                    const uint32_t bytes = (uint32_t)(__popc(__ballot_sync(0xffffffffu, valid)) * seg);
                    uint32_t dst, bar;
                    ring_claim(D, S, ring, bytes, dst, bar);
                    if (valid) bulk_g2s(dst + (uint32_t)(lane * seg), src, (uint32_t)seg, bar);
                    ring.pos = ring_add(S, ring.pos, 1);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------- projection: consumer

// Stages columns [ac0, ac0+acw) of the tagged input of job J into shared memory: polls the words, strips the
// tags, accumulates the sum of squares of every row, applies the RMSNorm gain, and stores bf16 hi+lo pairs
// (bf16 weights) or fp32 (fp32 weights), 16 bytes per 4 columns, rows (acw*4 + 16) bytes apart.  Rows of
// finished sequences are filled with zeros without waiting.
template <typename WT> __device__ __forceinline__ float4 load_gain4(const WT *gain, int k);
template <> __device__ __forceinline__ float4 load_gain4<float>(const float *gain, int k) {
    return __ldg(reinterpret_cast<const float4 *>(gain + k));
}
template <> __device__ __forceinline__ float4 load_gain4<bf16>(const bf16 *gain, int k) {
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(gain + k));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xffff0000u));
}

constexpr int kPollBatch = 6;   // tagged 16-byte loads a thread keeps in flight (20 KB of activations over 224 threads: one batch)

// walks the (row, 16-byte word) pairs of a staging pass without dividing: thread t starts at word t of row 0
struct RowWalk {
    int m, c4;
    __device__ __forceinline__ RowWalk(int tid, int v4_per_row) {
        m = 0; c4 = tid;
        while (c4 >= v4_per_row) { c4 -= v4_per_row; ++m; }      // v4_per_row >= 32: seven rounds at most
    }
    __device__ __forceinline__ void next(int v4_per_row) {
        c4 += kConsumerThreads;
        while (c4 >= v4_per_row) { c4 -= v4_per_row; ++m; }
    }
};

template <typename WT>
static __device__ void stage_acts(const Dev &D, const Smem &S, const GemvJob &J, int ac0, int acw, uint32_t tag);

// fp32 models: tagged fp32 words in, fp32 out; the reader applies the gain and sums the squares.
template <>
__device__ void stage_acts<float>(const Dev &D, const Smem &S, const GemvJob &J, int ac0, int acw, uint32_t tag) {
    const int M = D.M, tid = threadIdx.x;
    const int v4_per_row = acw >> 2, total = M * v4_per_row;
    const int pitch = acw * 4 + 16;
    const float *gain = reinterpret_cast<const float *>(J.gain);
    const float *x = J.x;
    const int kdim = J.kdim;
    const bool first = ac0 == 0;
    RowWalk rd(tid, v4_per_row), wr(tid, v4_per_row);
    for (int i0 = 0; i0 < total; i0 += kConsumerThreads * kPollBatch) {
        uint4 w[kPollBatch];
        float4 gn[kPollBatch];
        // issue every load of the batch before looking at any of them
#pragma unroll
        for (int u = 0; u < kPollBatch; ++u) {
            w[u] = make_uint4(tag, tag, tag, tag);          // rows that are not fetched read as zeros
            gn[u] = make_float4(1.f, 1.f, 1.f, 1.f);
            if (rd.m < M) {
                const int k = ac0 + (rd.c4 << 2);
                if (!S.ctl->row_dead[rd.m]) w[u] = ld_relaxed_u4(x + (size_t)rd.m * kdim + k);
                if (gain != nullptr) gn[u] = load_gain4<float>(gain, k);
            }
            rd.next(v4_per_row);
        }
#pragma unroll
        for (int u = 0; u < kPollBatch; ++u) {
            const int i = i0 + u * kConsumerThreads + tid;
            float ssq = 0.f;
            if (wr.m < M) {
                if (!tags_ok(w[u], tag)) w[u] = poll_u4(D, S.ctl, x + (size_t)wr.m * kdim + ac0 + (wr.c4 << 2), tag);
                float4 v = make_float4(untag(w[u].x), untag(w[u].y), untag(w[u].z), untag(w[u].w));
                if (gain != nullptr) {
                    ssq = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
                    v.x *= gn[u].x; v.y *= gn[u].y; v.z *= gn[u].z; v.w *= gn[u].w;
                }
                *reinterpret_cast<float4 *>(S.acts + (size_t)wr.m * pitch + ((size_t)wr.c4 << 4)) = v;
            }
            if (gain != nullptr && i0 + u * kConsumerThreads < total) {
                // acw is a multiple of 128: the 32 lanes of a warp hold words of one row
                ssq = warp_sum(ssq);
                if ((tid & 31) == 0 && i < total) S.sspart[i >> 5] = ssq;
            }
            wr.next(v4_per_row);
        }
    }
    csync();
    if (gain != nullptr && tid < M) {   // deterministic: fixed slots, fixed order
        const int per_row = v4_per_row >> 5;
        float s = first ? 0.f : S.ss[tid];
        for (int q = 0; q < per_row; ++q) s += S.sspart[tid * per_row + q];
        S.ss[tid] = s;
    }
    // the next csync() of the caller orders ss before its readers
}

// bf16 models: packed hi + lo words in (gain already applied by the writer), {hi01, hi23, lo01, lo23} out.
template <>
__device__ void stage_acts<bf16>(const Dev &D, const Smem &S, const GemvJob &J, int ac0, int acw, uint32_t tag) {
    const int M = D.M, tid = threadIdx.x;
    const int v4_per_row = acw >> 2, total = M * v4_per_row;
    const int pitch = acw * 4 + 16;
    const float *x = J.x;
    const int kdim = J.kdim;
    const bool dead_rows = S.ctl->any_dead != 0;
    RowWalk rd(tid, v4_per_row), wr(tid, v4_per_row);
    for (int i0 = 0; i0 < total; i0 += kConsumerThreads * kPollBatch) {
        uint4 w[kPollBatch];
        const float *src[kPollBatch];      // nullptr: nothing to fetch (past the end, or a finished sequence's row)
#pragma unroll
        for (int u = 0; u < kPollBatch; ++u) {
            src[u] = (rd.m < M && !(dead_rows && S.ctl->row_dead[rd.m])) ? x + (size_t)rd.m * kdim + ac0 + (rd.c4 << 2) : nullptr;
            rd.next(v4_per_row);
        }
        // The whole batch is requested at once.  Where a word has not arrived, the thread waits for the first such
        // word alone (one spin loop in the code, one word of polling traffic) and then requests the batch again.
        for (;;) {
            const float *stale = nullptr;
#pragma unroll
            for (int u = 0; u < kPollBatch; ++u) w[u] = src[u] != nullptr ? ld_relaxed_u4(src[u]) : make_uint4(tag, tag, tag, tag);
#pragma unroll
            for (int u = kPollBatch - 1; u >= 0; --u)
                if (!tags_ok(w[u], tag)) stale = src[u];
            if (stale == nullptr) break;
            poll_u4(D, S.ctl, stale, tag);
            if (S.ctl->dead) break;
        }
#pragma unroll
        for (int u = 0; u < kPollBatch; ++u) {
            if (wr.m < M) {
                uint4 o;
                o.x = __byte_perm(w[u].x, w[u].y, 0x7632);
                o.y = __byte_perm(w[u].z, w[u].w, 0x7632);
                o.z = __byte_perm(w[u].x, w[u].y, 0x5410) & 0xFFFCFFFCu;
                o.w = __byte_perm(w[u].z, w[u].w, 0x5410) & 0xFFFCFFFCu;
                *reinterpret_cast<uint4 *>(S.acts + (size_t)wr.m * pitch + ((size_t)wr.c4 << 4)) = o;
            }
            wr.next(v4_per_row);
        }
    }
    csync();
}

// bf16 models: the sum of squares of row m of a normed input = sum of the writer CTAs' shares, one warp per row,
// fixed order; left in S.ss (the caller synchronises).  Only the epilogue needs it, so it is gathered after the
// products, when the shares have long been published.
static __device__ void gather_ss(const Dev &D, const Smem &S, uint32_t tag) {
    const int M = D.M, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = (int)gridDim.x;
    for (int m = warp; m < M; m += kConsumerWarps) {
        float s = 0.f;
        if (!S.ctl->row_dead[m]) {
            uint32_t v[8];            // G <= 256: at most 8 shares per lane, all requested at once, and again
                                      // after a wait for the first one that was missing
            for (;;) {
                const float *stale = nullptr;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int c = lane + 32 * q;
                    v[q] = c < G ? ld_relaxed_u32(ss_word(D, c, m)) : tag;
                }
#pragma unroll
                for (int q = 7; q >= 0; --q)
                    if ((v[q] & 3u) != tag) stale = ss_word(D, lane + 32 * q, m);
                if (stale == nullptr) break;
                poll_u32(D, S.ctl, stale, tag);
                if (S.ctl->dead) break;
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) s += untag(v[q]);
        }
        s = warp_sum(s);
        if (lane == 0) S.ss[m] = s;
    }
}

// shared-memory address of layout row `row` of the tile whose first item sits at ring position pos_tile
__device__ __forceinline__ uint32_t tile_row_addr(const Smem &S, const SegPlan &p, uint32_t pos_tile, int row) {
    const int ns = S.n_slots;
    row = min(row, p.tile_rows - 1);     // rows past a short tile read its last row; their products are never used
    int slot = (int)ring_slot(S, pos_tile) + (row >> p.rpi_shift);
    if (slot >= ns) slot -= ns;
    return smem_u32(S.ring) + (uint32_t)slot * kSlotBytes + (uint32_t)((row & ((1 << p.rpi_shift) - 1)) * p.row_bytes);
}

// bf16 weights.  Warp (tile, part): A = 16 weight rows x 32 columns per step out of the ring (lane g = lane/4,
// t = lane%4 loads 16 bytes = 8 consecutive columns of rows g and g+8; the same column permutation is applied
// to the activation fragments, so the products pair up), B = activations of 8 tokens.  The warp takes the
// column blocks part, part + parts, ... of columns [k0, k0 + 32 * n_kb); U blocks are in flight together, each
// with accumulators of its own.
template <int NT, int U>
__device__ __forceinline__ void mma_tile_bf16(uint32_t row_a, uint32_t row_b, const char *acts, int pitch, int k0, int n_kb, int part,
                                              int parts, int M, float (&acc)[NT][2][4]) {
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const uint32_t wa0 = row_a + (uint32_t)(k0 * 2 + t * 16), wb0 = row_b + (uint32_t)(k0 * 2 + t * 16);
    const uint32_t x_base = smem_u32(acts) + (uint32_t)t * 32u;
    float au[U][NT][2][4];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int q = 0; q < 4; ++q) au[u][nt][0][q] = au[u][nt][1][q] = 0.f;
    for (int q0 = part; q0 < n_kb; q0 += parts * U) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kb = q0 + u * parts;
            if (kb < n_kb) {
                const uint4 wa = lds_u4(wa0 + (uint32_t)kb * 64u), wb = lds_u4(wb0 + (uint32_t)kb * 64u);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int m = nt * 8 + g;
                    uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = xa;
                    if (m < M) {
                        const uint32_t a = x_base + (uint32_t)m * (uint32_t)pitch + (uint32_t)kb * 128u;
                        xa = lds_u4(a);
                        xb = lds_u4(a + 16u);
                    }
                    mma16816(au[u][nt][0], wa.x, wb.x, wa.y, wb.y, xa.x, xa.y);
                    mma16816(au[u][nt][1], wa.x, wb.x, wa.y, wb.y, xa.z, xa.w);
                    mma16816(au[u][nt][0], wa.z, wb.z, wa.w, wb.w, xb.x, xb.y);
                    mma16816(au[u][nt][1], wa.z, wb.z, wa.w, wb.w, xb.z, xb.w);
                }
            }
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int q = 0; q < 4; ++q) { acc[nt][0][q] += au[u][nt][0][q]; acc[nt][1][q] += au[u][nt][1][q]; }
}

// A word of the published final hidden state (plain tagged fp32, written once per step by some CTA of an earlier
// stage of the same step: it carries the step's tag by now, except when that CTA is late; bounded wait).
__device__ __forceinline__ float residual_word(const float *p, uint32_t tag) {
    uint32_t w = ld_relaxed_u32(p);
    for (unsigned it = 0; (w & 3u) != tag && it < kSpinLimit; ++it) w = ld_relaxed_u32(p);
    return untag(w);
}

// Every CTA's part of the side output of a projection stage with a normed input: columns [c d / G, (c + 1) d / G) of
// g[m] = x[m] / rms(x[m]) (times the gain where the input is published without it), as plain tagged fp32 in D.gpub.
// inv[m] = 1 / rms(x[m]) in shared memory.  Called by all consumer threads after the inputs have arrived.
template <typename WT>
__device__ __forceinline__ void publish_normed_slice(const Dev &D, const float *x, int kdim, const void *gain, const float *inv, uint32_t tag) {
    const int G = (int)gridDim.x, c = (int)blockIdx.x;
    const int u0 = (int)((long long)kdim * c / G), u1 = (int)((long long)kdim * (c + 1) / G), nu = u1 - u0;
    for (int i = threadIdx.x; i < D.M * nu; i += kConsumerThreads) {
        const int m = i / nu, u = u0 + i - m * nu;
        float v = read_word<WT>(ld_relaxed_u32(x + (size_t)m * kdim + u)) * inv[m];
        if (sizeof(WT) == 4) v *= reinterpret_cast<const float *>(gain)[u];
        st_relaxed_u32(D.gpub + (size_t)m * kdim + u, tagged(v, tag));
    }
}

// What one output element becomes (after the dot product v, already scaled by 1/rms when the job has a gain).
// hprev: the residual stream's value when the caller has fetched it ahead (have_prev), EPI_ADD only.
// Returns the value before any gain of the next stage is applied (the residual stream's new value for EPI_ADD).
template <typename WT>
__device__ __forceinline__ float epilogue_store(const GemvJob &J, int m, int u, float v, float v2, float inv, uint32_t tag_out,
                                                bool have_prev = false, float hprev = 0.f, float gprev = 1.f) {
    float *o = J.out + (size_t)m * J.out_ld + u;
    float r, pub;
    if (J.epi == EPI_STORE) pub = r = v;
    else if (J.epi == EPI_GATEUP) pub = r = silu_f(v) * v2;
    else if (J.epi == EPI_ADD) {
        float *hm = J.hm + (size_t)m * J.out_ld + u;
        pub = r = (have_prev ? hprev : __ldcg(hm)) + v;
        __stcg(hm, r);
        // bf16 models: the reader's RMSNorm gain is applied here, once, instead of by every reader
        if (sizeof(WT) == 2 && J.gain_out != nullptr) pub = r * (have_prev ? gprev : to_f(reinterpret_cast<const WT *>(J.gain_out)[u]));
    } else if (J.epi == EPI_ADDG) {   // the final hidden state g (published by the stage before the heads' attention) + v
        pub = r = residual_word(J.res + (size_t)m * J.out_ld + u, tag_out) + v;
    } else {   // EPI_HEADY: residual on the normalised input (this CTA has already waited for that word);
               // inv = 1 / rms(x[m]), times gain[u] where the input is published without its gain (fp32 models)
        pub = r = read_word<WT>(ld_relaxed_u32(J.x + (size_t)m * J.kdim + u)) * inv + silu_f(v);
    }
    st_relaxed_u32(o, publish_word<WT>(pub, tag_out, J.out_plain != 0));
    return r;
}

template <typename WT, int NT>
static __device__ void consume_segment_bf16(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R,
                                     uint32_t serial) {
    const SegPlan p = R.p;
    const int lo = R.lo, hi = R.hi;
    const int M = D.M, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int kca = J.kdim;               // the whole input fits the staging area (else: consume_segment_chunked)
    constexpr bool one_chunk = true;
    const uint32_t tag_in = tag_of(serial, J.in), tag_out = tag_of(serial, J.outt);
    const WT *gain = reinterpret_cast<const WT *>(J.gain);
    constexpr int NP = NT * 8;
    bool staged = false, ss_raw = false;     // ss_raw: S.ss holds sums of squares that still await 1/sqrt
    float ss_share = 0.f;
    for (int tg0 = 0; tg0 < p.n_tiles; tg0 += p.tpg) {
        const int tg = min(p.tpg, p.n_tiles - tg0);
        // parts = 7 / tg and my_tile = warp / parts without dividing (tg in 1..7, warp in 0..6)
        static_assert(kConsumerWarps == 7, "the two lookups below are for seven consumer warps");
        const int parts = (0x11112370 >> (4 * tg)) & 15;
        const int my_tile = (warp * (parts == 7 ? 5 : parts == 3 ? 11 : parts == 2 ? 16 : 32)) >> 5;
        const int my_part = warp - my_tile * parts;                            // my_tile >= tg: idle warp
        const uint32_t pos0 = ring.pos;      // the group's items: tile tl at positions pos0 + tl * ipt ...
        bool landed = false;
        float acc[NT][2][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[nt][0][q] = acc[nt][1][q] = 0.f;
        // The static part of the epilogue is done now, while the inputs are still on their way: where this
        // thread's first four outputs go (output i = (tile, token, unit), unit fastest), and what they need from
        // global memory (the residual stream's old value, the gain applied to the published copy).
        const int outs = tg * p.tile_units * M;
        const int tu_shift = p.tu_shift, tu_mask = p.tile_units - 1;
        const int n_out_iter = (outs + kConsumerThreads - 1) / kConsumerThreads;
        int o_n[4], o_u[4], o_red[4];
        float hpre[4], gpre[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = tid + q * kConsumerThreads;
            o_n[q] = 0; o_u[q] = -1; o_red[q] = 0; hpre[q] = 0.f; gpre[q] = 1.f;
            if (i < outs) {
                const int ui = i & tu_mask, rest = i >> tu_shift, tl = (rest * D.inv_m) >> 20, n = rest - tl * M;
                const int u = lo + (tg0 + tl) * p.tile_units + ui;
                o_n[q] = n;
                o_red[q] = tl * parts * NP * 16 + n * 16 + ui;
                if (u < hi) {
                    o_u[q] = u;
                    if (J.epi == EPI_ADD) {
                        hpre[q] = __ldcg(J.hm + (size_t)n * J.out_ld + u);
                        if (J.gain_out != nullptr) gpre[q] = to_f(reinterpret_cast<const WT *>(J.gain_out)[u]);
                    }
                }
            }
        }
        for (int ac0 = 0; ac0 < J.kdim; ac0 += kca) {
            const int acw = min(kca, J.kdim - ac0), pitch = acw * 4 + 16;
            if (!(one_chunk && staged)) {
                csync();                       // everyone is done with the previous content of the area
                stage_acts<WT>(D, S, J, ac0, acw, tag_in);
                csync();
                staged = true;
                if (ac0 == 0) ss_raw = true;
                if (S.ctl->trace_row) trace_mark(D, S.ctl->trace_row);
            }
            // All items of the group are in the ring at once, each in a slot of its own.  A warp waits only for
            // the items of its tile (once, before the first chunk of activations is multiplied).
            if (my_tile < tg) {
                if (!landed) {
                    Ring r;
                    for (int i = 0; i < p.ipt; ++i) { r.pos = ring_add(S, pos0, my_tile * p.ipt + i); ring_wait(D, S, r); }
                    landed = true;
                }
                constexpr int U = NT == 1 ? 4 : (NT == 2 ? 2 : 1);
                const uint32_t pos_tile = ring_add(S, pos0, my_tile * p.ipt);
                mma_tile_bf16<NT, U>(tile_row_addr(S, p, pos_tile, g), tile_row_addr(S, p, pos_tile, g + 8), S.acts, pitch, ac0,
                                     acw >> 5, my_part, parts, M, acc);
            }
        }
        // Every warp frees every item of the group; a warp that did not read an item does so without waiting
        // for it: the previous item of that slot was freed by all warps before the barrier that opened this
        // group's staging, so no arrival can fall into the wrong phase.
        __syncwarp();
        if (lane == 0)
            for (int i = 0; i < tg * p.ipt; ++i) mbar_arrive(S.empty0 + 8u * ring_slot(S, ring_add(S, pos0, i)));
        ring.pos = ring_add(S, pos0, tg * p.ipt);
        if (gain != nullptr && ss_raw) gather_ss(D, S, tag_in);
        // cross-warp reduction through the activation area, then the epilogue
        csync();
        // [warp][NP][16] partial products: behind the staged activations when both fit (then a following tile
        // group finds the activations still in place), else over them
        const int red_bytes = (kConsumerWarps * NP * 16 + kConsumerWarps * M) * 4;
        const bool red_apart = one_chunk && M * (J.kdim * 4 + 16) + red_bytes <= D.acts_bytes;
        float *red = reinterpret_cast<float *>(S.acts + (red_apart ? M * (J.kdim * 4 + 16) : 0));
        if (!red_apart) staged = false;
        if (my_tile < tg) {
            float *r = red + (size_t)warp * NP * 16;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int n0 = nt * 8 + 2 * t;
                r[n0 * 16 + g] = acc[nt][0][0] + acc[nt][1][0];
                r[(n0 + 1) * 16 + g] = acc[nt][0][1] + acc[nt][1][1];
                r[n0 * 16 + g + 8] = acc[nt][0][2] + acc[nt][1][2];
                r[(n0 + 1) * 16 + g + 8] = acc[nt][0][3] + acc[nt][1][3];
            }
        }
        // a tile group that found the activations still staged also finds the inverse norms of the group before
        if (gain != nullptr && ss_raw && tid < M) S.ss[tid] = 1.0f / sqrtf(S.ss[tid] / (float)J.kdim + D.eps);
        ss_raw = false;
        csync();
        if (J.norm_out && gain != nullptr && tg0 == 0) publish_normed_slice<WT>(D, J.x, J.kdim, J.gain, S.ss, tag_out);
        float *ssg = red + (size_t)kConsumerWarps * NP * 16;   // [tile][token] sums of squares of the new residual values
        const bool want_ss = J.epi == EPI_ADD && J.gain_out != nullptr;
        for (int q = 0; q < n_out_iter; ++q) {
            const int i = tid + q * kConsumerThreads;
            int n, u, ro;
            if (q < 4) {
                n = q == 0 ? o_n[0] : q == 1 ? o_n[1] : q == 2 ? o_n[2] : o_n[3];
                u = q == 0 ? o_u[0] : q == 1 ? o_u[1] : q == 2 ? o_u[2] : o_u[3];
                ro = q == 0 ? o_red[0] : q == 1 ? o_red[1] : q == 2 ? o_red[2] : o_red[3];
            } else {
                const int ui = i & tu_mask, rest = i >> tu_shift, tl = (rest * D.inv_m) >> 20;
                n = rest - tl * M;
                u = lo + (tg0 + tl) * p.tile_units + ui;
                ro = tl * parts * NP * 16 + n * 16 + ui;
                if (i >= outs || u >= hi) u = -1;
            }
            float r = 0.f;
            if (u >= 0) {
                float v = 0.f, v2 = 0.f;
                for (int pq = 0; pq < parts; ++pq) {
                    const float *rr = red + ro + pq * NP * 16;
                    v += rr[0];
                    if (J.epi == EPI_GATEUP) v2 += rr[8];
                }
                float inv = 1.f;
                if (gain != nullptr) { inv = S.ss[n]; v *= inv; v2 *= inv; }
                r = epilogue_store<WT>(J, n, u, v, v2, inv, tag_out, q < 4,
                                       q == 0 ? hpre[0] : q == 1 ? hpre[1] : q == 2 ? hpre[2] : hpre[3],
                                       q == 0 ? gpre[0] : q == 1 ? gpre[1] : q == 2 ? gpre[2] : gpre[3]);
            }
            if (want_ss) {
                // the units of one (tile, token) sit in adjacent lanes: a fixed tree adds their squares
                float sq = r * r;
                sq += __shfl_xor_sync(0xffffffffu, sq, 1);
                sq += __shfl_xor_sync(0xffffffffu, sq, 2);
                if (p.tile_units >= 8) sq += __shfl_xor_sync(0xffffffffu, sq, 4);
                if (p.tile_units == 16) sq += __shfl_xor_sync(0xffffffffu, sq, 8);
                if ((i & tu_mask) == 0 && i < outs) ssg[i >> tu_shift] = sq;
            }
        }
        if (want_ss) {
            // this CTA's share of the sum of squares of every row, in a fixed order
            csync();
            if (tid < M) {
                for (int tl = 0; tl < tg; ++tl) ss_share += ssg[tl * M + tid];
                if (tg0 + p.tpg >= p.n_tiles) st_relaxed_u32(ss_word(D, blockIdx.x, tid), tagged(ss_share, tag_out));
            }
        }
    }
}

// Consumer side of produce_segment_chunked.  Every warp waits for every item (so every warp frees every item it has
// seen land); a warp multiplies the token tiles warp, warp + 7, ... of each tile and adds its products to the
// accumulators in shared memory, which it alone touches for those tokens.
template <typename WT>
static __device__ void consume_segment_chunked(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R,
                                               uint32_t serial) {
    const SegPlan p = R.p;
    const int lo = R.lo, hi = R.hi;
    const int M = D.M, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const uint32_t tag_in = tag_of(serial, J.in), tag_out = tag_of(serial, J.outt);
    const WT *gain = reinterpret_cast<const WT *>(J.gain);
    const int tr = chunk_tiles_per_round(p, M);
    float *accum = reinterpret_cast<float *>(S.acts + (size_t)M * (D.kca * 4 + 16));   // [tile][token][16]
    float *ssg = accum + kAccumBytes / 4;                                              // [tile][token]
    const int tu_shift = p.tu_shift, tu_mask = p.tile_units - 1;
    const bool want_ss = J.epi == EPI_ADD && J.gain_out != nullptr;
    float ss_share = 0.f;
    for (int r0 = 0; r0 < p.n_tiles; r0 += tr) {
        const int nr = min(tr, p.n_tiles - r0);
        csync();                               // the previous round's epilogue has read the accumulators
        for (int i = tid; i < nr * M * 16; i += kConsumerThreads) accum[i] = 0.f;
        for (int ac0 = 0; ac0 < J.kdim; ac0 += D.kca) {
            const int acw = min(D.kca, J.kdim - ac0), seg = acw * (int)sizeof(WT), pitch = acw * 4 + 16;
            const int sh = chunk_rpi_shift(p, seg), ipt = p.tile_rows >> sh;
            csync();                           // everyone is done with the previous chunk
            stage_acts<WT>(D, S, J, ac0, acw, tag_in);
            if (ac0 == 0 && S.ctl->trace_row) trace_mark(D, S.ctl->trace_row);
            for (int tl = 0; tl < nr; ++tl) {
                const uint32_t pos_tile = ring.pos;
                Ring r;
                for (int i = 0; i < ipt; ++i) { r.pos = ring_add(S, pos_tile, i); ring_wait(D, S, r); }
                // rows g and g + 8 of the tile (rows past a short tile read its last row; their products are not used)
                const int ra = min(g, p.tile_rows - 1), rb = min(g + 8, p.tile_rows - 1);
                const uint32_t base = smem_u32(S.ring);
                const uint32_t row_a = base + ring_slot(S, ring_add(S, pos_tile, ra >> sh)) * kSlotBytes + (uint32_t)((ra & ((1 << sh) - 1)) * seg);
                const uint32_t row_b = base + ring_slot(S, ring_add(S, pos_tile, rb >> sh)) * kSlotBytes + (uint32_t)((rb & ((1 << sh) - 1)) * seg);
                for (int nt = warp; nt * 8 < M; nt += kConsumerWarps) {
                    float acc[1][2][4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) acc[0][0][q] = acc[0][1][q] = 0.f;
                    mma_tile_bf16<1, 4>(row_a, row_b, S.acts + (size_t)nt * 8 * pitch, pitch, 0, acw >> 5, 0, 1, M - nt * 8, acc);
                    const int n0 = nt * 8 + 2 * t;
                    float *a = accum + ((size_t)tl * M + n0) * 16;
                    if (n0 < M) { a[g] += acc[0][0][0] + acc[0][1][0]; a[g + 8] += acc[0][0][2] + acc[0][1][2]; }
                    if (n0 + 1 < M) { a[16 + g] += acc[0][0][1] + acc[0][1][1]; a[16 + g + 8] += acc[0][0][3] + acc[0][1][3]; }
                }
                __syncwarp();
                if (lane == 0)
                    for (int i = 0; i < ipt; ++i) mbar_arrive(S.empty0 + 8u * ring_slot(S, ring_add(S, pos_tile, i)));
                ring.pos = ring_add(S, pos_tile, ipt);
            }
        }
        if (gain != nullptr && r0 == 0) gather_ss(D, S, tag_in);
        csync();
        if (gain != nullptr && r0 == 0 && tid < M) S.ss[tid] = 1.0f / sqrtf(S.ss[tid] / (float)J.kdim + D.eps);
        csync();
        if (J.norm_out && gain != nullptr && r0 == 0) publish_normed_slice<WT>(D, J.x, J.kdim, J.gain, S.ss, tag_out);
        const int outs = nr * p.tile_units * M;
        for (int i0 = 0; i0 < outs; i0 += kConsumerThreads) {
            const int i = i0 + tid;
            const int ui = i & tu_mask, rest = i >> tu_shift, tl = (rest * D.inv_m) >> 20, n = rest - tl * M;
            const int u = lo + (r0 + tl) * p.tile_units + ui;
            float r = 0.f;
            if (i < outs && u < hi) {
                const float *a = accum + ((size_t)tl * M + n) * 16;
                float v = a[ui], v2 = J.epi == EPI_GATEUP ? a[ui + 8] : 0.f, inv = 1.f;
                if (gain != nullptr) { inv = S.ss[n]; v *= inv; v2 *= inv; }
                r = epilogue_store<WT>(J, n, u, v, v2, inv, tag_out);
            }
            if (want_ss) {
                // the units of one (tile, token) sit in adjacent lanes: a fixed tree adds their squares
                float sq = r * r;
                sq += __shfl_xor_sync(0xffffffffu, sq, 1);
                sq += __shfl_xor_sync(0xffffffffu, sq, 2);
                if (p.tile_units >= 8) sq += __shfl_xor_sync(0xffffffffu, sq, 4);
                if (p.tile_units == 16) sq += __shfl_xor_sync(0xffffffffu, sq, 8);
                if ((i & tu_mask) == 0 && i < outs) ssg[i >> tu_shift] = sq;
            }
        }
        if (want_ss) {
            csync();
            if (tid < M) {
                for (int tl = 0; tl < nr; ++tl) ss_share += ssg[tl * M + tid];
                if (r0 + tr >= p.n_tiles) st_relaxed_u32(ss_word(D, blockIdx.x, tid), tagged(ss_share, tag_out));
            }
        }
    }
}

// fp32 weights: the 16 rows of a tile form 8 pairs (q, q+8) (for gate/up: the gate and the up row of unit q);
// warp w owns pairs w, w + kConsumerWarps, ...; lanes stride over the columns; the activations of all tokens
// must fit the staging area in one chunk.
template <int MT>
__device__ void consume_segment_f32(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R,
                                    uint32_t serial) {
    constexpr int PPW = (8 + kConsumerWarps - 1) / kConsumerWarps;   // pairs per warp
    const SegPlan p = R.p;
    const int lo = R.lo, hi = R.hi;
    const int M = D.M, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t tag_in = tag_of(serial, J.in), tag_out = tag_of(serial, J.outt);
    const float *gain = reinterpret_cast<const float *>(J.gain);
    const int pitch = J.kdim * 4 + 16;
    csync();
    stage_acts<float>(D, S, J, 0, J.kdim, tag_in);
    csync();
    if (gain != nullptr && tid < M) S.ss[tid] = 1.0f / sqrtf(S.ss[tid] / (float)J.kdim + D.eps);
    csync();
    if (J.norm_out && gain != nullptr) publish_normed_slice<float>(D, J.x, J.kdim, J.gain, S.ss, tag_out);
    if (S.ctl->trace_row) trace_mark(D, S.ctl->trace_row);
    for (int tg0 = 0; tg0 < p.n_tiles; tg0 += p.tpg) {
        const int tg = min(p.tpg, p.n_tiles - tg0);
        const uint32_t pos0 = ring.pos;
        for (int tl = 0; tl < tg; ++tl) {
            const uint32_t pos_tile = ring_add(S, pos0, tl * p.ipt);
            Ring r;
            for (int i = 0; i < p.ipt; ++i) { r.pos = ring_add(S, pos_tile, i); ring_wait(D, S, r); }
            float acc[PPW][2][MT];
#pragma unroll
            for (int s2 = 0; s2 < PPW; ++s2)
#pragma unroll
                for (int n = 0; n < MT; ++n) acc[s2][0][n] = acc[s2][1][n] = 0.f;
#pragma unroll
            for (int s2 = 0; s2 < PPW; ++s2) {
                const int q = warp + s2 * kConsumerWarps;
                if (q < 8) {
                    const uint32_t ra = tile_row_addr(S, p, pos_tile, q), rb = tile_row_addr(S, p, pos_tile, q + 8);
                    for (int k = lane * 4; k < J.kdim; k += 128) {
                        const uint4 ua = lds_u4(ra + (uint32_t)k * 4u), ub = lds_u4(rb + (uint32_t)k * 4u);
                        const float4 wa = make_float4(__uint_as_float(ua.x), __uint_as_float(ua.y), __uint_as_float(ua.z), __uint_as_float(ua.w));
                        const float4 wb = make_float4(__uint_as_float(ub.x), __uint_as_float(ub.y), __uint_as_float(ub.z), __uint_as_float(ub.w));
#pragma unroll
                        for (int n = 0; n < MT; ++n) {
                            if (n < M) {
                                const float4 x = *reinterpret_cast<const float4 *>(S.acts + (size_t)n * pitch + (size_t)k * 4);
                                acc[s2][0][n] = fmaf(wa.x, x.x, acc[s2][0][n]); acc[s2][0][n] = fmaf(wa.y, x.y, acc[s2][0][n]);
                                acc[s2][0][n] = fmaf(wa.z, x.z, acc[s2][0][n]); acc[s2][0][n] = fmaf(wa.w, x.w, acc[s2][0][n]);
                                acc[s2][1][n] = fmaf(wb.x, x.x, acc[s2][1][n]); acc[s2][1][n] = fmaf(wb.y, x.y, acc[s2][1][n]);
                                acc[s2][1][n] = fmaf(wb.z, x.z, acc[s2][1][n]); acc[s2][1][n] = fmaf(wb.w, x.w, acc[s2][1][n]);
                            }
                        }
                    }
                }
            }
            const int u0 = lo + (tg0 + tl) * p.tile_units;
#pragma unroll
            for (int s2 = 0; s2 < PPW; ++s2) {
                const int q = warp + s2 * kConsumerWarps;
                if (q >= 8) continue;
#pragma unroll
                for (int n = 0; n < MT; ++n) {
                    if (n < M) {
                        float va = warp_sum(acc[s2][0][n]), vb = warp_sum(acc[s2][1][n]);
                        if (lane == 0) {
                            const float inv = gain != nullptr ? S.ss[n] : 1.f;
                            va *= inv; vb *= inv;
                            if (J.epi == EPI_GATEUP) {
                                if (u0 + q < hi) epilogue_store<float>(J, n, u0 + q, va, vb, inv, tag_out);
                            } else {
                                if (q < p.tile_units && u0 + q < hi)
                                    epilogue_store<float>(J, n, u0 + q, va, 0.f, J.epi == EPI_HEADY ? inv * gain[u0 + q] : inv, tag_out);
                                if (q + 8 < p.tile_units && u0 + q + 8 < hi)
                                    epilogue_store<float>(J, n, u0 + q + 8, vb, 0.f, J.epi == EPI_HEADY ? inv * gain[u0 + q + 8] : inv, tag_out);
                            }
                        }
                    }
                }
            }
        }
        // every warp has read every item of the group
        __syncwarp();
        if (lane == 0)
            for (int i = 0; i < tg * p.ipt; ++i) mbar_arrive(S.empty0 + 8u * ring_slot(S, ring_add(S, pos0, i)));
        ring.pos = ring_add(S, pos0, tg * p.ipt);
    }
}

// ------------------------------------------------------------- projection: consumer, few token rows (batch 1)

// the same product as mma16816, left to the compiler's scheduler (no ordering against other statements)
__device__ __forceinline__ void mma16816_free(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0,
                                              unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Staging of the whole tagged input x[M][kdim] of a job (at most eight rows) as {hi01, hi23, lo01, lo23} words, NB
// 16-byte loads per thread in flight.  The loads of the first batch are issued as soon as the stage begins (plan,
// issue); the caller then does everything that does not need them, and finish() waits for the words, stores them and
// works through the remaining batches.  With want_ss the CTAs' shares of the rows' sums of squares travel in the first
// batch and are left, tags stripped and added four by four, in S.sspart as [row][CTA / 4].  finish() ends with a barrier of the consumer warps.
template <int NB>
struct ActLoads {
    int src[NB];               // element offset into x, -1: nothing to fetch (past the end, or a finished sequence's row)
    int dst[NB];               // byte offset in the staging area, -1: past the end
    int sh[2];                 // the shares: 16-byte words tid and tid + 224 of [row][CTA] (at most 1536 floats), -1: none
    uint4 w[NB], sw[2];

    __device__ __forceinline__ void plan(const Dev &D, const Smem &S, int kdim, int i0, bool want_ss) {
        const int M = D.M, tid = threadIdx.x;
        const int v4 = kdim >> 2, total = M * v4, pitch = kdim * 4 + 16;
        const uint32_t inv = 0xFFFFFFFFu / (uint32_t)v4 + 1u;       // i / v4 == umulhi(i, inv) for i, v4 < 2^16
        const bool dead_rows = S.ctl->any_dead != 0;
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int i = i0 + u * kConsumerThreads + tid;
            src[u] = -1; dst[u] = -1;
            if (i < total) {
                const int m = (int)__umulhi((uint32_t)i, inv), c4 = i - m * v4;
                dst[u] = m * pitch + (c4 << 4);
                if (!(dead_rows && S.ctl->row_dead[m])) src[u] = m * kdim + (c4 << 2);
            }
        }
        const int n_sh = (want_ss && i0 == 0) ? ((int)gridDim.x * M) >> 2 : 0;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int wi = tid + q * kConsumerThreads;
            sh[q] = wi < n_sh ? wi : -1;
            // nobody publishes the shares of a finished sequence's rows ([row][CTA]: a word lies in one row)
            if (dead_rows && wi < n_sh && S.ctl->row_dead[(4 * wi) / (int)gridDim.x]) sh[q] = -1;
        }
    }
    __device__ __forceinline__ void issue(const Dev &D, const float *x, uint32_t tag) {
#pragma unroll
        for (int u = 0; u < NB; ++u) w[u] = src[u] >= 0 ? ld_relaxed_u4(x + src[u]) : make_uint4(tag, tag, tag, tag);
#pragma unroll
        for (int q = 0; q < 2; ++q) sw[q] = sh[q] >= 0 ? ld_relaxed_u4(D.sspub + 4 * sh[q]) : make_uint4(tag, tag, tag, tag);
    }
    // the first word that does not carry the tag yet (nullptr: all have arrived)
    __device__ __forceinline__ const float *stale(const Dev &D, const float *x, uint32_t tag) const {
        const float *st = nullptr;
#pragma unroll
        for (int q = 1; q >= 0; --q)
            if (!tags_ok(sw[q], tag)) st = D.sspub + 4 * sh[q];
#pragma unroll
        for (int u = NB - 1; u >= 0; --u)
            if (!tags_ok(w[u], tag)) st = x + src[u];
        return st;
    }
    __device__ __forceinline__ void store(const Smem &S) const {
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            if (dst[u] >= 0) {
                uint4 o;
                o.x = __byte_perm(w[u].x, w[u].y, 0x7632);
                o.y = __byte_perm(w[u].z, w[u].w, 0x7632);
                o.z = __byte_perm(w[u].x, w[u].y, 0x5410) & 0xFFFCFFFCu;
                o.w = __byte_perm(w[u].z, w[u].w, 0x5410) & 0xFFFCFFFCu;
                *reinterpret_cast<uint4 *>(S.acts + dst[u]) = o;
            }
        }
#pragma unroll
        for (int q = 0; q < 2; ++q)
            if (sh[q] >= 0)      // four shares of one row, added here already: [row][CTA / 4]
                S.sspart[sh[q]] = (untag(sw[q].x) + untag(sw[q].y)) + (untag(sw[q].z) + untag(sw[q].w));
    }
    // Where a word has not arrived, the thread waits for the first such word alone and then requests the batch again.
    __device__ __forceinline__ void finish(const Dev &D, const Smem &S, const float *x, int kdim, uint32_t tag) {
        const int total = D.M * (kdim >> 2);
        for (int i0 = 0;;) {
            for (;;) {
                const float *st = stale(D, x, tag);
                if (st == nullptr) break;
                poll_u4(D, S.ctl, st, tag);
                if (S.ctl->dead) break;
                issue(D, x, tag);
            }
            store(S);
            i0 += kConsumerThreads * NB;
            if (i0 >= total) break;
            plan(D, S, kdim, i0, false);
            issue(D, x, tag);
        }
        csync();
    }
};

constexpr int kSmallLoads = 6;   // 16-byte loads of activations a thread keeps in flight on this path

// The consumer of produce_segment for at most eight token rows.  ONE code path serves every shape (the code of a stage
// runs about once per stage, so what counts is how much of it the layers share: variants per shape would stream
// through the instruction cache).  Two barriers per tile group: after the staging of the activations (once per job),
// and after every warp has parked its partial products.  Between them warp w multiplies every tile of the group (at
// most four, accumulators in registers) over the column blocks w, w + 7, ... and (w < M) adds up the sums of squares
// of token row w; after them warp w finishes the outputs of token row w (unit = lane), so the row's share of the new
// sum of squares is a shuffle reduction and no further barrier is needed.
// J0, R: the job's entry in the table (layer 0, or the tail when layer < 0) and this CTA's plan record, both in shared
// memory: a field is read when it is needed.
template <typename WT>
static __device__ void consume_small(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J0, int layer, const SegRec &R, uint32_t serial,
                                     bool norm_out) {
    static_assert(kConsumerWarps == 7, "the sum of the warps' partial products is written out for seven warps");
    const int M = D.M, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int kdim = J0.kdim, pitch = kdim * 4 + 16, n_kb = kdim >> 5;
    const int lay = max(layer, 0);
    const float *x = J0.x;
    const bool normed = J0.gain != nullptr;
    const uint32_t tag_in = tag_of(serial, TagRef{J0.in.wps, J0.in.j + lay * J0.in_jinc});
    // the activations are requested before anything else: their round trip through the L2 is the longest wait of the stage
    ActLoads<kSmallLoads> A;
    A.plan(D, S, kdim, 0, normed);
    A.issue(D, x, tag_in);
    const float inv_kdim = 1.0f / (float)kdim;
    const SegPlan p = R.p;
    const int lo = R.lo, hi = R.hi;
    const int epi = J0.epi, out_ld = J0.out_ld;
    const bool out_plain = J0.out_plain != 0;
    float *const out = J0.out, *const hmaster = J0.hm;
    const uint32_t tag_out = tag_of(serial, TagRef{J0.outt.wps, J0.outt.j + lay * J0.out_jinc});
    // the gain that the published copy of the residual stream carries: that of the RMSNorm which reads it next
    const WT *gain_out = reinterpret_cast<const WT *>(J0.gain_out);
    if (gain_out != nullptr) {
        if (layer > 0) gain_out = reinterpret_cast<const WT *>(reinterpret_cast<const char *>(gain_out) + S.tab->layer_bytes * layer);
        if (layer >= 0 && J0.gain_out_step != 0)
            gain_out = layer == D.L - 1 ? reinterpret_cast<const WT *>(S.tab->gain_last)
                                        : reinterpret_cast<const WT *>(reinterpret_cast<const char *>(gain_out) + J0.gain_out_step);
    }
    const bool want_ss = epi == EPI_ADD && gain_out != nullptr;
    const int tu_shift = p.tu_shift, tu_mask = p.tile_units - 1;
    // tiles of at most eight rows: rows 8..15 of the products are never used and not read
    const bool lower = p.tile_rows <= 8 || (epi != EPI_GATEUP && p.n_tiles == 1 && hi - lo <= 8);
    // EPI_ADD: the residual stream's old values and the gains of the published copy for the first group, fetched while
    // the inputs are on their way (token row = warp, unit = lane and lane + 32)
    float hpre[2] = {0.f, 0.f}, gpre[2] = {1.f, 1.f};
    if (epi == EPI_ADD && warp < M) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int u = lo + lane + 32 * q;
            if (u < hi && lane + 32 * q < p.tpg * p.tile_units) {
                hpre[q] = __ldcg(hmaster + (size_t)warp * out_ld + u);
                if (gain_out != nullptr) gpre[q] = to_f(gain_out[u]);
            }
        }
    }
    float *red = reinterpret_cast<float *>(S.acts + M * pitch);      // [warp][tile of the group: p.tpg][token 8][row 16]
    float ss_acc[2] = {0.f, 0.f}, inv_rms[2] = {1.f, 1.f};
    const uint32_t x_addr = smem_u32(S.acts) + (uint32_t)(min(g, M - 1) * pitch) + (uint32_t)t * 32u;
    const bool has_x = g < M;
    for (int tg0 = 0; tg0 < p.n_tiles; tg0 += p.tpg) {
        const int tg = min(p.tpg, p.n_tiles - tg0), n_items = tg * p.ipt;
        const uint32_t pos0 = ring.pos;
        // every warp reads every tile of the group: lane i waits for item i (and will free it)
        uint32_t my_empty = 0u;
        if (lane < n_items) {
            Ring r;
            r.pos = ring_add(S, pos0, lane);
            ring_wait(D, S, r);
            my_empty = S.empty0 + 8u * ring_slot(S, r.pos);
        }
        __syncwarp();
        uint32_t row_a[kSmallTiles], row_b[kSmallTiles];
#pragma unroll
        for (int tl = 0; tl < kSmallTiles; ++tl) {
            const uint32_t pos_tile = ring_add(S, pos0, min(tl, tg - 1) * p.ipt);
            row_a[tl] = tile_row_addr(S, p, pos_tile, g) + (uint32_t)t * 16u;
            row_b[tl] = tile_row_addr(S, p, pos_tile, g + 8) + (uint32_t)t * 16u;
        }
        if (tg0 == 0) {
            A.finish(D, S, x, kdim, tag_in);
            if (S.ctl->trace_row) trace_mark(D, S.ctl->trace_row);
            // 1 / rms of token row `warp` (and of row warp + 7): the shares [row][CTA] are added in a fixed order
            if (normed) {
                const int G4 = (int)gridDim.x >> 2;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int m = warp + q * kConsumerWarps;
                    if (m < M) {
                        float sum = 0.f;
                        for (int c4 = lane; c4 < G4; c4 += 32) sum += S.sspart[m * G4 + c4];
                        sum = warp_sum(sum);
                        inv_rms[q] = S.ctl->row_dead[m] ? 1.f : rsqrtf(fmaf(sum, inv_kdim, D.eps));
                        if (norm_out && lane == 0) S.ss[m] = inv_rms[q];
                    }
                }
                if (norm_out) {      // the side output of the stage: this CTA's columns of the normed input (rare: once per step)
                    csync();
                    publish_normed_slice<WT>(D, x, kdim, J0.gain, S.ss, tag_out);
                }
            }
        }
        // products: per column block the activations once, then every tile of the group (hi and lo chains of a tile
        // are independent, tiles are independent)
        float acc[kSmallTiles][2][4];
#pragma unroll
        for (int tl = 0; tl < kSmallTiles; ++tl)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[tl][0][q] = acc[tl][1][q] = 0.f;
        for (int kb = warp; kb < n_kb; kb += kConsumerWarps) {
            uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = xa;
            if (has_x) {
                xa = lds_u4(x_addr + (uint32_t)kb * 128u);
                xb = lds_u4(x_addr + (uint32_t)kb * 128u + 16u);
            }
#pragma unroll
            for (int tl = 0; tl < kSmallTiles; ++tl) {
                if (tl < tg) {
                    const uint4 wa = lds_u4(row_a[tl] + (uint32_t)kb * 64u);
                    uint4 wb = make_uint4(0u, 0u, 0u, 0u);
                    if (!lower) wb = lds_u4(row_b[tl] + (uint32_t)kb * 64u);
                    mma16816_free(acc[tl][0], wa.x, wb.x, wa.y, wb.y, xa.x, xa.y);
                    mma16816_free(acc[tl][1], wa.x, wb.x, wa.y, wb.y, xa.z, xa.w);
                    mma16816_free(acc[tl][0], wa.z, wb.z, wa.w, wb.w, xb.x, xb.y);
                    mma16816_free(acc[tl][1], wa.z, wb.z, wa.w, wb.w, xb.z, xb.w);
                }
            }
        }
        __syncwarp();
        if (lane < n_items) mbar_arrive(my_empty);
        ring.pos = ring_add(S, pos0, n_items);
        if (tg0 != 0) csync();        // the previous group's partial products have been read
#pragma unroll
        for (int tl = 0; tl < kSmallTiles; ++tl) {
            if (tl < tg) {
                float *r = red + ((size_t)(warp * p.tpg + tl) * 8) * 16;
                r[(2 * t) * 16 + g] = acc[tl][0][0] + acc[tl][1][0];
                r[(2 * t + 1) * 16 + g] = acc[tl][0][1] + acc[tl][1][1];
                r[(2 * t) * 16 + g + 8] = acc[tl][0][2] + acc[tl][1][2];
                r[(2 * t + 1) * 16 + g + 8] = acc[tl][0][3] + acc[tl][1][3];
            }
        }
        // EPI_HEADY adds the normalised input itself: taken from the staged copy before anyone may overwrite it
        const int u_first = lo + tg0 * p.tile_units, ug = min(tg * p.tile_units, hi - u_first);
        float xin[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
        if (epi == EPI_HEADY) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int m = warp + q * kConsumerWarps;
#pragma unroll
                for (int jq = 0; jq < 2; ++jq) {
                    const int j = lane + 32 * jq;
                    if (m < M && j < ug) {
                        const int u = u_first + j;
                        const uint4 o = *reinterpret_cast<const uint4 *>(S.acts + (size_t)m * pitch + ((u >> 2) << 4));
                        const uint32_t hw = (u & 2) ? o.y : o.x, lw = (u & 2) ? o.w : o.z;
                        const uint32_t hb = (u & 1) ? (hw & 0xFFFF0000u) : (hw << 16), lb = (u & 1) ? (lw & 0xFFFF0000u) : (lw << 16);
                        xin[q][jq] = __uint_as_float(hb) + __uint_as_float(lb);
                    }
                }
            }
        }
        csync();
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int m = warp + q * kConsumerWarps;
            if (m >= M) break;
            const float inv = inv_rms[q];
#pragma unroll
            for (int jq = 0; jq < 2; ++jq) {
                const int j = lane + 32 * jq;
                if (j >= ug) break;
                const int tl = j >> tu_shift, ui = j & tu_mask, u = u_first + j;
                const float *rr = red + ((size_t)tl * 8 + m) * 16 + ui;
                float pv[kConsumerWarps], pv2[kConsumerWarps];
#pragma unroll
                for (int w2 = 0; w2 < kConsumerWarps; ++w2) {
                    pv[w2] = rr[(size_t)w2 * p.tpg * 128];
                    pv2[w2] = epi == EPI_GATEUP ? rr[(size_t)w2 * p.tpg * 128 + 8] : 0.f;
                }
                float v = ((pv[0] + pv[1]) + (pv[2] + pv[3])) + ((pv[4] + pv[5]) + pv[6]);
                float v2 = ((pv2[0] + pv2[1]) + (pv2[2] + pv2[3])) + ((pv2[4] + pv2[5]) + pv2[6]);
                v *= inv; v2 *= inv;
                float *o = out + (size_t)m * out_ld + u;
                float pub;
                if (epi == EPI_STORE) pub = v;
                else if (epi == EPI_GATEUP) pub = silu_f(v) * v2;
                else if (epi == EPI_ADD) {
                    float *hm = hmaster + (size_t)m * out_ld + u;
                    const bool pre = tg0 == 0 && q == 0;
                    const float r = (pre ? hpre[jq] : __ldcg(hm)) + v;
                    __stcg(hm, r);
                    pub = r;
                    if (gain_out != nullptr) pub = r * (pre ? gpre[jq] : to_f(gain_out[u]));
                    ss_acc[q] += r * r;
                } else if (epi == EPI_ADDG) pub = residual_word(J0.res + (size_t)m * out_ld + u, tag_out) + v;
                else pub = xin[q][jq] * inv + silu_f(v);
                st_relaxed_u32(o, publish_word<WT>(pub, tag_out, out_plain));
            }
        }
    }
    if (want_ss) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int m = warp + q * kConsumerWarps;
            if (m < M) {
                const float sh = warp_sum(ss_acc[q]);
                if (lane == 0) st_relaxed_u32(ss_word(D, blockIdx.x, m), tagged(sh, tag_out));
            }
        }
    }
}

// ------------------------------------------------- projection on the tcgen05 path (27 or more token rows, bf16)

// K-major operand tile with the 128-byte swizzle: rows of 64 bf16 (128 bytes), 8-row groups 1024 bytes apart (stride byte
// offset), leading byte offset unused (1), descriptor version of sm_100, layout type 2.  The tile starts on a 1024-byte
// boundary; a K = 16 step inside the 64 columns is 32 bytes further.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, both K-major, N and M of the tile
__device__ __forceinline__ uint32_t umma_idesc(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                 :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0), "r"(0), "r"(0), "r"(0) : "memory");
}
// one arrival at the barrier when every product issued by this thread so far has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
// box {64 columns, 8 rows, 1 layer} of a weight matrix -> shared memory (swizzled), completion on an mbarrier; every CTA fetches its own boxes
__device__ __forceinline__ void tma_box(uint32_t dst, const void *tmap, int x, int y, int z, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 :: "r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// A tile of the CTA's segment: up to 128 weight rows (64 units of gate + up rows), 8-row groups in the order the
// accumulator's columns take: plain jobs [rows 0-7][8-15]..., gate/up jobs [gate units 0-7][up units 0-7][gate 8-15]...
struct UmmaTile { int u0, nu, groups; };
__device__ __forceinline__ UmmaTile umma_tile(int epi, int u0, int hi) {
    UmmaTile t;
    t.u0 = u0;
    t.nu = min(epi == EPI_GATEUP ? kUmmaTileRows / 2 : kUmmaTileRows, hi - u0);
    t.groups = ((t.nu + 7) >> 3) * (epi == EPI_GATEUP ? 2 : 1);
    return t;
}

// Producer: for every tile, for every block of 64 columns, one ring item with a box per row group.
template <typename WT>
static __device__ void produce_segment_umma(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R, int layer) {
    const int lane = threadIdx.x & 31, lay = max(layer, 0);
    for (int u0 = R.lo; u0 < R.hi;) {
        const UmmaTile t = umma_tile(J.epi, u0, R.hi);
        for (int kc = 0; kc < J.kdim; kc += kUmmaK) {
            uint32_t dst, bar;
            ring_claim(D, S, ring, (uint32_t)t.groups * 1024u, dst, bar);
            if (lane < t.groups) {
                const bool up = J.epi == EPI_GATEUP && (lane & 1);
                const int row = J.epi == EPI_GATEUP ? t.u0 + 8 * (lane >> 1) : t.u0 + 8 * lane;
                tma_box(dst + (uint32_t)lane * 1024u, up ? J.tmap2 : J.tmap, kc, row, lay, bar);
            }
            ring.pos = ring_add(S, ring.pos, 1);
        }
        u0 += t.nu;
    }
}

// One consumer warp issues the products; with at most 32 token rows (little to stage, the issuing thread is the limit) two
// do, one per activation buffer, each into an accumulator of its own.  The other consumer warps stage activations.
__host__ __device__ constexpr int umma_issuers(int m) { return m <= 32 ? 2 : 1; }
// 16-byte loads of one column block per staging thread: NTM * 8 token rows x 16 quads over the staging threads
__host__ __device__ constexpr int umma_loads(int ntm) {
    return (ntm * 8 * 16 + (kConsumerWarps - umma_issuers(ntm * 8)) * 32 - 1) / ((kConsumerWarps - umma_issuers(ntm * 8)) * 32);
}

// Consumer.  Per tile and block of 64 columns: the staging warps (0..5) store the activations of the block (all token
// rows) as two planes of bf16 (hi, lo) in the swizzled K-major layout, double buffered, the loads of the next block in
// flight while this one is stored, and arrive at the buffer's "staged" barrier; the issuing warp (6) waits for that
// barrier and for the block's weights, issues the eight products (four K = 16 steps, hi and lo planes into one
// accumulator) and commits them to the buffer's "done" barrier.  Nobody waits for the issuing thread: staging runs
// ahead until it needs a buffer back.  A ring slot is freed (one arrival per consumer warp) when the products that read
// it are known to be done: two blocks later, or after the tile's last commit.  After the last block the accumulator
// D[token][weight row] is read back by the thread of the token (warps 0..3), which finishes all outputs of its token
// row: the row's share of the new sum of squares needs no reduction.  The shares of the input rows are added up on the
// way, a few rows per staging warp and column block.
template <typename WT, int NTM>
static __device__ void consume_segment_umma(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R, uint32_t serial) {
    constexpr int kUmmaLoads = umma_loads(NTM);
    const int M = D.M, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kdim = J.kdim, n_kc = kdim / kUmmaK;
    const uint32_t tag_in = tag_of(serial, J.in), tag_out = tag_of(serial, J.outt);
    const bool normed = J.gain != nullptr;
    const bool want_ss = J.epi == EPI_ADD && J.gain_out != nullptr;
    const bool dead_rows = S.ctl->any_dead != 0;
    const int n_iss = umma_issuers(M), stage_warps = kConsumerWarps - n_iss, stage_threads = stage_warps * 32;
    const bool issuer = warp >= stage_warps;
    const float *x = J.x;
    char *const planes = S.acts;                     // [buffer][hi | lo][128 rows x 128 bytes]
    const int G = (int)gridDim.x;
    // rows whose shares a staging warp adds up per column block, so that all M rows are done by the last block
    const int rows_per = (M + stage_warps * n_kc - 1) / (stage_warps * n_kc);
    csync();                                         // the previous user of the activation area and of S.ss is done
    uint32_t chunk = S.ctl->umma_chunks, tiles = S.ctl->umma_tiles;
    float ss_acc = 0.f;
    // a staging thread's quads of a column block: i = tid + u * 192 -> token row i / 16, quad i % 16 (four columns);
    // where a quad comes from (block 0; nullptr: a finished sequence's row, read as zeros) and where it goes inside a
    // plane (-1: past the last token row) is the same for every block of the job
    const float *q_src[kUmmaLoads];
    int q_off[kUmmaLoads];
#pragma unroll
    for (int u = 0; u < kUmmaLoads; ++u) {
        const int i = tid + u * stage_threads, r = i >> 4, q = i & 15;
        q_src[u] = (r < M && !(dead_rows && S.ctl->row_dead[r])) ? x + (size_t)r * kdim + q * 4 : nullptr;
        q_off[u] = r < M ? (r >> 3) * 1024 + (r & 7) * 128 + (((q >> 1) ^ (r & 7)) << 4) + ((q & 1) << 3) : -1;
    }
    auto issue = [&](uint4 (&w)[kUmmaLoads], int kc) {
#pragma unroll
        for (int u = 0; u < kUmmaLoads; ++u)
            w[u] = q_src[u] != nullptr ? ld_relaxed_u4(q_src[u] + kc * kUmmaK) : make_uint4(tag_in, tag_in, tag_in, tag_in);
    };
    // one arrival of this warp at the "empty" barrier of the ring slot that held block kc of the tile
    auto free_slot = [&](uint32_t pos0, int kc) {
        if (lane == 0) mbar_arrive(S.empty0 + 8u * ring_slot(S, ring_add(S, pos0, kc)));
    };
    for (int u0 = R.lo; u0 < R.hi;) {
        const UmmaTile t = umma_tile(J.epi, u0, R.hi);
        const int n_cols = t.groups * 8, mma_n = (n_cols + 15) & ~15;
        const uint32_t idesc = umma_idesc(128, mma_n);      // M = 128: row i of the accumulator is lane i of tensor memory
        const uint32_t pos0 = ring.pos, chunk0 = chunk;
        const bool first_tile = u0 == R.lo;
        if (issuer) {
            // ---- an issuing warp.  It passes every block of the tile: once a block's weights have landed the warp gives its
            // arrival for the slot (the slot is refilled only after the staging warps' arrivals, which follow the completion
            // of the products that read it); the blocks of its own buffer it multiplies.
            const int me = warp - stage_warps;
            for (int kc = 0; kc < n_kc; ++kc) {
                const uint32_t c = chunk0 + (uint32_t)kc;
                const int buf = (int)(c & 1u);
                Ring r;
                r.pos = ring_add(S, pos0, kc);
                const uint32_t wts = smem_u32(ring_wait(D, S, r));
                free_slot(pos0, kc);
                if (n_iss == 2 && buf != me) continue;
                mbar_wait(D, S.ctl, S.sbar0 + 8u * (uint32_t)buf, (c >> 1) & 1u);       // the block's activations are staged
                tcgen05_after_sync();
                if (lane == 0) {
                    const uint32_t a_hi = smem_u32(planes + buf * 2 * kUmmaPlaneBytes), a_lo = a_hi + (uint32_t)kUmmaPlaneBytes;
                    const uint32_t acc = S.ctl->tmem + (n_iss == 2 ? (uint32_t)(buf * kUmmaTileRows) : 0u);
                    const bool fresh = kc < n_iss;                       // the accumulator's first block of the tile
#pragma unroll
                    for (int ks = 0; ks < kUmmaK / 16; ++ks) {
                        const uint64_t db = umma_desc_sw128(wts + (uint32_t)ks * 32u);
                        umma_mma(acc, umma_desc_sw128(a_hi + (uint32_t)ks * 32u), db, idesc, (!fresh || ks > 0) ? 1u : 0u);
                        umma_mma(acc, umma_desc_sw128(a_lo + (uint32_t)ks * 32u), db, idesc, 1u);
                    }
                    umma_commit(S.abar0 + 8u * (uint32_t)buf);
                }
                __syncwarp();
            }
            if (lane == 0) umma_commit(S.dbar);          // one arrival per issuing warp when all its products are done
            __syncwarp();
        } else {
            // ---- the staging warps
            uint4 wa[kUmmaLoads], wb[kUmmaLoads];
            issue(wa, 0);
            // one column block: w holds its words, wn receives those of the next block
            auto block = [&](uint4 (&w)[kUmmaLoads], uint4 (&wn)[kUmmaLoads], int kc) {
                const uint32_t c = chunk0 + (uint32_t)kc;
                const int buf = (int)(c & 1u);
                char *p_hi = planes + buf * 2 * kUmmaPlaneBytes, *p_lo = p_hi + kUmmaPlaneBytes;
                if (kc + 1 < n_kc) issue(wn, kc + 1);          // the loads of the next block go out before this one is looked at
                // the shares of a few input rows per warp (normed jobs, first tile only): all loads first, then the tags
                if (normed && first_tile) {
                    for (int q = 0; q < rows_per; ++q) {
                        const int m = (kc * rows_per + q) * stage_warps + warp;
                        if (m < M) {
                            float sum = 0.f;
                            if (!S.ctl->row_dead[m]) {
                                uint32_t sw[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) sw[e] = lane + 32 * e < G ? ld_relaxed_u32(ss_word(D, lane + 32 * e, m)) : tag_in;
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    if ((sw[e] & 3u) != tag_in) sw[e] = poll_u32_cold(D, S.ctl, ss_word(D, lane + 32 * e, m), tag_in);
                                    if (lane + 32 * e < G) sum += untag(sw[e]);
                                }
                                sum = warp_sum(sum);
                            }
                            if (lane == 0) S.ss[m] = sum;
                        }
                    }
                }
                // the products that read this buffer two blocks ago must be done; their ring slot is free then
                if (kc >= 2) {
                    mbar_wait(D, S.ctl, S.abar0 + 8u * (uint32_t)buf, ((c >> 1) - 1u) & 1u);
                    free_slot(pos0, kc - 2);
                }
#pragma unroll
                for (int u = 0; u < kUmmaLoads; ++u) {
                    if (q_off[u] >= 0) {
                        if (!tags_ok(w[u], tag_in) && q_src[u] != nullptr) w[u] = poll_u4_cold(D, S.ctl, q_src[u] + kc * kUmmaK, tag_in);
                        uint2 hi, lo;
                        hi.x = __byte_perm(w[u].x, w[u].y, 0x7632);
                        hi.y = __byte_perm(w[u].z, w[u].w, 0x7632);
                        lo.x = __byte_perm(w[u].x, w[u].y, 0x5410) & 0xFFFCFFFCu;
                        lo.y = __byte_perm(w[u].z, w[u].w, 0x5410) & 0xFFFCFFFCu;
                        *reinterpret_cast<uint2 *>(p_hi + q_off[u]) = hi;
                        *reinterpret_cast<uint2 *>(p_lo + q_off[u]) = lo;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic-proxy stores to shared memory, read by the tensor core's proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(S.sbar0 + 8u * (uint32_t)buf);
                if (kc == 0 && first_tile && S.ctl->trace_row) trace_mark(D, S.ctl->trace_row);
            };
            for (int kc = 0; kc < n_kc; kc += 2) {
                block(wa, wb, kc);
                if (kc + 1 < n_kc) block(wb, wa, kc + 1);
            }
        }
        ring.pos = ring_add(S, pos0, n_kc);
        chunk = chunk0 + (uint32_t)n_kc;
        // ---- every product of the tile is done: the last slots are freed, the accumulator is read
        mbar_wait(D, S.ctl, S.dbar, tiles & 1u);
        ++tiles;
        tcgen05_after_sync();
        if (!issuer)       // (an issuing warp gave its arrival for every slot when the slot's weights landed)
            for (int kc = max(n_kc - 2, 0); kc < n_kc; ++kc) free_slot(pos0, kc);
        if (normed && first_tile) {
            csync();
            if (tid < M) S.ss[tid] = S.ctl->row_dead[tid] ? 1.f : 1.0f / sqrtf(S.ss[tid] / (float)kdim + D.eps);
            csync();
            if (J.norm_out) publish_normed_slice<WT>(D, J.x, J.kdim, J.gain, S.ss, tag_out);
        }
        // Jobs without a residual add (wide tiles, no row sums): the accumulator is copied to shared memory (the
        // activation planes are idle now) and its elements are finished by all consumer warps, a warp per token row
        // and a lane per weight row, so that the stores of a row are coalesced.  Residual adds (few weight rows per
        // CTA, a sum of squares per token row) stay with the thread of the token row.
        const bool spread = J.epi != EPI_ADD;
        float *const acc_copy = reinterpret_cast<float *>(planes);
        const int pitch = (M * (n_cols + 4) * 4 <= kUmmaActsBytes) ? n_cols + 4 : n_cols;      // (multiples of four floats)
        if (warp < 4) {      // thread = token row (warps 0..3 own the accumulator's lanes 0..127)
            const int m = tid;
            const float inv = (normed && m < M) ? S.ss[m] : 1.f;
            for (int c0 = 0; c0 < n_cols; c0 += 16) {
                uint32_t v[16];
                // (a tile of one block has used the accumulator of that block's buffer only)
                const uint32_t taddr = S.ctl->tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0 +
                                       ((n_iss == 2 && (chunk0 & 1u)) ? (uint32_t)kUmmaTileRows : 0u);
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                             : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                               "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                             : "r"(taddr) : "memory");
                if (n_iss == 2 && n_kc >= 2) {       // two accumulators (one per activation buffer): their sum
                    uint32_t v2[16];
                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                                 : "=r"(v2[0]), "=r"(v2[1]), "=r"(v2[2]), "=r"(v2[3]), "=r"(v2[4]), "=r"(v2[5]), "=r"(v2[6]), "=r"(v2[7]), "=r"(v2[8]),
                                   "=r"(v2[9]), "=r"(v2[10]), "=r"(v2[11]), "=r"(v2[12]), "=r"(v2[13]), "=r"(v2[14]), "=r"(v2[15])
                                 : "r"(taddr ^ (uint32_t)kUmmaTileRows) : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(v2[j]));
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (spread) {
                    if (m < M) {
#pragma unroll
                        for (int j = 0; j < 16; j += 4)
                            if (c0 + j < n_cols) *reinterpret_cast<uint4 *>(acc_copy + (size_t)m * pitch + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    }
                } else if (m < M) {
                    // sixteen columns = two row groups: plain jobs sixteen units, gate/up jobs eight units (gate, up)
                    const int units = J.epi == EPI_GATEUP ? 8 : 16;
                    const int ub = t.u0 + (J.epi == EPI_GATEUP ? (c0 >> 1) : c0);
                    // residual add: the old values of the residual stream (and the gains of the published copy) are all
                    // requested before the first is used
                    const bool pre = J.epi == EPI_ADD;
                    float hprev[16], gprev[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        hprev[j] = 0.f; gprev[j] = 1.f;
                        if (pre && ub + j < t.u0 + t.nu) {
                            hprev[j] = __ldcg(J.hm + (size_t)m * J.out_ld + ub + j);
                            if (J.gain_out != nullptr) gprev[j] = to_f(reinterpret_cast<const WT *>(J.gain_out)[ub + j]);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (j < units && ub + j < t.u0 + t.nu) {
                            const float a = __uint_as_float(v[j]) * inv;
                            const float b2 = J.epi == EPI_GATEUP ? __uint_as_float(v[(j + 8) & 15]) * inv : 0.f;
                            const float r = epilogue_store<WT>(J, m, ub + j, a, b2, inv, tag_out, pre, hprev[j], gprev[j]);
                            ss_acc += r * r;
                        }
                    }
                }
            }
        }
        tcgen05_before_sync();
        csync();                 // the accumulator has been read: the next tile (or job) may overwrite it
        tcgen05_after_sync();
        if (spread) {
            const bool gateup = J.epi == EPI_GATEUP;
            for (int m = warp; m < M; m += kConsumerWarps) {
                const float inv = normed ? S.ss[m] : 1.f;
                for (int j = lane; j < t.nu; j += 32) {
                    const int ca = gateup ? ((j >> 3) * 16 + (j & 7)) : j;      // gate/up: [gate units 0-7][up units 0-7][gate 8-15]...
                    const float a = acc_copy[(size_t)m * pitch + ca] * inv;
                    const float b2 = gateup ? acc_copy[(size_t)m * pitch + ca + 8] * inv : 0.f;
                    epilogue_store<WT>(J, m, t.u0 + j, a, b2, inv, tag_out);
                }
            }
            csync();             // the copy has been read: the next tile's activations may overwrite it
        }
        u0 += t.nu;
    }
    if (want_ss && tid < M) st_relaxed_u32(ss_word(D, blockIdx.x, tid), tagged(ss_acc, tag_out));
    if (tid == 0) { S.ctl->umma_chunks = chunk; S.ctl->umma_tiles = tiles; }
}

// NTM: token tiles of 8 (bf16 weights) or token rows (fp32 weights) the kernel is compiled for
template <typename WT, int NTM> struct ConsumeSegment;
template <int NTM> struct ConsumeSegment<bf16, NTM> {
    static __device__ __forceinline__ void run(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R, uint32_t serial) {
        if constexpr (NTM > 1) {     // (the instance for at most eight token rows holds consume_small only)
            if constexpr (NTM * 8 >= kUmmaMinRows) {     // (the instance for 9..16 token rows never takes the tcgen05 path)
                if (D.umma) { consume_segment_umma<bf16, NTM>(D, S, ring, J, R, serial); return; }
            }
            if (D.kca < J.kdim) { consume_segment_chunked<bf16>(D, S, ring, J, R, serial); return; }
            consume_segment_bf16<bf16, NTM>(D, S, ring, J, R, serial);
        }
    }
};
template <int NTM> struct ConsumeSegment<float, NTM> {
    static __device__ __forceinline__ void run(const Dev &D, const Smem &S, Ring &ring, const GemvJob &J, const SegRec &R, uint32_t serial) {
        consume_segment_f32<NTM>(D, S, ring, J, R, serial);
    }
};

// This CTA's share of every job, worked out once per launch: the rows of a stage's jobs form one range that is cut
// evenly over the CTAs.  Thread i fills the record of job i.
template <typename WT> static __device__ void plan_segments(const Dev &D, const Smem &S) {
    const Tables &T = *S.tab;
    const int n_jobs = kLayerJobs + T.n_tail_jobs, n_st = kLayerStages + T.n_tail_stages;
    for (int i = threadIdx.x; i < n_jobs; i += blockDim.x) {
        SegRec r;
        r.lo = r.hi = 0;
        r.p = seg_plan<WT>(D, S, T.jobs[i], 0, 0);
        for (int s = 0; s < n_st; ++s) {
            const Stage &st = T.stages[s];
            if (st.kind != ST_GEMV || i < st.job0 || i >= st.job0 + st.njobs) continue;
            unsigned total = 0;      // rows of all jobs of the stage (a few tens of thousands at most)
            int base = 0;
            for (int j = 0; j < st.njobs; ++j) {
                if (st.job0 + j == i) base = (int)total;
                total += (unsigned)T.jobs[st.job0 + j].rows;
            }
            const int u_lo = (int)(total * blockIdx.x / gridDim.x), u_hi = (int)(total * (blockIdx.x + 1) / gridDim.x);
            r.lo = max(u_lo - base, 0);
            r.hi = max(min(u_hi - base, T.jobs[i].rows), r.lo);
            r.p = seg_plan<WT>(D, S, T.jobs[i], r.lo, r.hi);
        }
        S.seg[i] = r;
    }
}

// A projection stage, seen by the producer warp (PRODUCER) or by the consumer warps.
template <typename WT, int NTM, bool PRODUCER>
static __device__ void gemv_stage(const Dev &D, const Smem &S, Ring &ring, const Stage &st, uint32_t serial) {
    bool norm_out = st.norm_out != 0;      // the first job this CTA has rows of carries the stage's side output
    for (int j = 0; j < st.njobs; ++j) {
        if (!PRODUCER && sizeof(WT) == 2 && NTM == 1 && small_mode<WT>(D, S.tab->jobs[st.job0 + j].kdim)) {
            if (S.seg[st.job0 + j].lo < S.seg[st.job0 + j].hi) {
                consume_small<bf16>(D, S, ring, S.tab->jobs[st.job0 + j], st.layer, S.seg[st.job0 + j], serial, norm_out);
                norm_out = false;
            }
            continue;
        }
        const SegRec R = S.seg[st.job0 + j];
        if (R.lo < R.hi) {
            GemvJob J = job_at(D, S, st.job0 + j, st.layer);
            J.norm_out = norm_out ? 1 : 0;
            norm_out = false;
            if (PRODUCER) {
                if (sizeof(WT) == 2 && NTM * 8 >= kUmmaMinRows && D.umma) produce_segment_umma<WT>(D, S, ring, J, R, st.layer);
                else if (sizeof(WT) == 2 && D.kca < J.kdim) produce_segment_chunked<WT>(D, S, ring, J, R);
                else produce_segment<WT>(D, S, ring, J, R);
            }
            else ConsumeSegment<WT, NTM>::run(D, S, ring, J, R, serial);
        }
    }
}

// -------------------------------------------------------------------------------- attention: plan

// Cache tiles.  One (page, head) tile holds P rows (positions) of dh elements.  16-bit tiles are stored with
// their 16-byte chunks permuted so that ldmatrix over 8 consecutive rows touches every bank once; fp32
// tiles are stored plain.
template <typename KVT>
__device__ __forceinline__ KVT *kv_tile(const Dev &D, void *pool, int pool_pages, int layer, int kv, int page, int head) {
    return reinterpret_cast<KVT *>(pool) + ((((size_t)layer * 2 + kv) * pool_pages + page) * D.H + head) * (size_t)D.P * D.dh;
}
// physical 16-byte chunk of logical chunk c of row r, rows of row_bytes
__device__ __forceinline__ int swz(int r, int c, int row_bytes) {
    return row_bytes >= 128 ? (c ^ (r & 7)) : (c ^ ((r >> 1) & 3));
}
// element offset of (row r, element e) inside a tile
template <typename KVT> __device__ __forceinline__ size_t tile_off(int r, int e, int dh);
template <> __device__ __forceinline__ size_t tile_off<float>(int r, int e, int dh) { return (size_t)r * dh + e; }
template <> __device__ __forceinline__ size_t tile_off<__half>(int r, int e, int dh) {
    return (size_t)r * dh + (size_t)swz(r, e >> 3, dh * 2) * 8 + (e & 7);
}

struct AttnItem { int b, h, s, S, hd; };     // hd: decoding head (stage ST_ATTN_HEAD), else 0

// page and row inside the page of a position (pages of a power of two of positions need no division: an integer
// division by a run-time value costs a hundred cycles, and these sit at the head of every attention item)
__device__ __forceinline__ int page_of(const Dev &D, int pos) { return D.p_shift >= 0 ? pos >> D.p_shift : pos / D.P; }
__device__ __forceinline__ int row_in_page(const Dev &D, int pos) { return D.p_shift >= 0 ? pos & (D.P - 1) : pos % D.P; }
// number of key splits of sequence b's self-attention this step
__device__ __forceinline__ int self_splits(const Dev &D, int len) {
    const int np = page_of(D, len + D.P - 1);
    return min(max((np + 3) / 4, 1), D.S_max);
}
// the idx-th live item of the stage (sequences that are finished have none); false when idx is past the end
__device__ __forceinline__ bool attn_item_at(const Dev &D, const Ctl *ctl, int kind, int idx, AttnItem &it) {
    const int sets = kind == ST_ATTN_HEAD ? D.K : 1;      // the decoding heads attend one after the other
    for (int hd = 0; hd < sets; ++hd)
        for (int b = 0; b < D.B; ++b) {
            if (ctl->flags[b] & 1) continue;
            const int S = kind != ST_ATTN_SELF ? D.S_cross : self_splits(D, ctl->len[b]);
            const int n = D.H * S;
            if (idx < n) {
                it.b = b; it.S = S; it.hd = hd;
                it.h = S == 1 ? idx : idx / S;
                it.s = idx - it.h * S;
                return true;
            }
            idx -= n;
        }
    return false;
}
// pages [p_lo, p_hi) of cached keys that split s of S covers
__device__ __forceinline__ void split_pages(const Dev &D, int n_keys, int s, int S, int &p_lo, int &p_hi) {
    const int np = page_of(D, n_keys + D.P - 1), pp = S == 1 ? np : (np + S - 1) / S;
    p_lo = min(np, s * pp);
    p_hi = min(np, (s + 1) * pp);
}

// ---------------------------------------------------------------------------- attention: producer

template <typename WT>
static __device__ void produce_attn(const Dev &D, const Smem &S, Ring &ring, const Stage &st) {
    typedef typename CacheT<WT>::type KVT;
    if (sizeof(KVT) != 2) return;   // the fp32 cache is read straight from global memory
    const bool cross = st.kind != ST_ATTN_SELF, headx = st.kind == ST_ATTN_HEAD;
    const int lane = threadIdx.x & 31;
    void *pool = headx ? D.hckv_pool : cross ? D.ckv_pool : D.kv_pool;
    const int pool_pages = cross ? D.B * D.cpages : D.n_pages;
    AttnItem it;
    for (int idx = blockIdx.x; attn_item_at(D, S.ctl, st.kind, idx, it); idx += gridDim.x) {
        int p_lo, p_hi;
        split_pages(D, cross ? D.C : S.ctl->len[it.b], it.s, it.S, p_lo, p_hi);
        int table = 0;      // block-table entries of 32 consecutive pages, one per lane: one round trip per 32 pages
        for (int pg = p_lo; pg < p_hi; ++pg) {
            const int k32 = (pg - p_lo) & 31;
            if (!cross && k32 == 0 && pg + lane < p_hi) table = __ldcg(D.block_table + (size_t)it.b * D.max_blocks + pg + lane);
            const int page = cross ? it.b * D.cpages + pg : __shfl_sync(0xffffffffu, table, k32);
            const int set = headx ? it.hd : st.layer;
            const KVT *kt = kv_tile<KVT>(D, pool, pool_pages, set, 0, page, it.h);
            const KVT *vt = kv_tile<KVT>(D, pool, pool_pages, set, 1, page, it.h);
            uint32_t dst, bar;
            if (D.kv_one_item) {
                ring_claim(D, S, ring, 2u * (uint32_t)D.tile_bytes, dst, bar);
                if (lane == 0) bulk_g2s(dst, kt, (uint32_t)D.tile_bytes, bar);
                if (lane == 1) bulk_g2s(dst + (uint32_t)D.tile_bytes, vt, (uint32_t)D.tile_bytes, bar);
                ring.pos = ring_add(S, ring.pos, 1);
            } else {
                ring_claim(D, S, ring, (uint32_t)D.tile_bytes, dst, bar);
                if (lane == 0) bulk_g2s(dst, kt, (uint32_t)D.tile_bytes, bar);
                ring.pos = ring_add(S, ring.pos, 1);
                ring_claim(D, S, ring, (uint32_t)D.tile_bytes, dst, bar);
                if (lane == 0) bulk_g2s(dst, vt, (uint32_t)D.tile_bytes, bar);
                ring.pos = ring_add(S, ring.pos, 1);
            }
        }
    }
}

// ---------------------------------------------------------------------------- attention: consumer

// Shared-memory plan of an attention item inside the activation area (K1 <= 16 query rows).
template <int DH> struct AttnSmem {
    static constexpr int QP = DH + 8;                 // bf16 elements between query rows (16 bytes of padding)
    bf16 *qh, *ql;                                    // [16][QP] rotated, scaled queries as hi + lo (rows >= K1 zero)
    float *qf;                                        // [K1][DH] fp32 queries
    float *kw, *vw;                                   // fp32 cache: [K1][DH] window keys (rotated), window values
    __half *kt, *vt;                                  // 16-bit cache: the same as two cache tiles of 32 rows (same bytes as kw, vw)
    float *raw;                                       // [3][K1][DH] unrotated q, k, v; later the merged state
    float *st;                                        // [kConsumerWarps + 1][K1][DH + 2] per-warp softmax states
    __device__ AttnSmem(char *base, int K1) {
        qh = reinterpret_cast<bf16 *>(base);
        ql = qh + 16 * QP;
        qf = reinterpret_cast<float *>(ql + 16 * QP);
        kw = qf + K1 * DH;
        vw = kw + K1 * DH;
        kt = reinterpret_cast<__half *>(kw);
        vt = kt + 32 * DH;
        raw = kw + 32 * DH;                           // 128 DH bytes hold either pair (K1 <= 16)
        st = raw + 3 * K1 * DH;
    }
};

// Online-softmax state of one warp for query rows g and g+8 (base-2 exponentials).
template <int DH> struct WarpState {
    float o[DH / 8][4];
    float m[2], l[2];
};

// 32 keys of one tile against the 16 query rows: S = Q K^T (hi + lo queries), online softmax, O += P V.
// CAUSAL: the keys are those of the query rows themselves, row r sees keys 0..r.
template <int DH, bool CAUSAL>
__device__ __forceinline__ void attn_unit(uint32_t q_hi, uint32_t q_lo, uint32_t k_tile, uint32_t v_tile, int key0, int nvalid,
                                          WarpState<DH> &ws) {
    constexpr int QPB = (DH + 8) * 2, RB = DH * 2;
    constexpr int NK = CAUSAL ? 1 : 2;      // 16-key steps: the window has at most 16 rows
    const int lane = threadIdx.x & 31, t = lane & 3, g = lane >> 2;
    float s[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
        unsigned qh[4], ql[4];
        const uint32_t qo = (uint32_t)(lane & 15) * QPB + (uint32_t)(ks * 16 + (lane >> 4) * 8) * 2u;
        ldmatrix_x4(qh, q_hi + qo);
        ldmatrix_x4(ql, q_lo + qo);
#pragma unroll
        for (int np = 0; np < NK; ++np) {      // key tiles 2np, 2np+1 (8 keys each)
            const int row = key0 + np * 16 + (lane & 7) + ((lane >> 4) << 3);
            const int chunk = 2 * ks + ((lane >> 3) & 1);
            unsigned kb[4];
            ldmatrix_x4(kb, k_tile + (uint32_t)row * RB + (uint32_t)swz(row, chunk, RB) * 16u);
            mma16816_f16(s[2 * np], qh[0], qh[1], qh[2], qh[3], kb[0], kb[1]);
            mma16816_f16(s[2 * np], ql[0], ql[1], ql[2], ql[3], kb[0], kb[1]);
            mma16816_f16(s[2 * np + 1], qh[0], qh[1], qh[2], qh[3], kb[2], kb[3]);
            mma16816_f16(s[2 * np + 1], ql[0], ql[1], ql[2], ql[3], kb[2], kb[3]);
        }
    }
    // mask the keys past the end, row maxima over the 32 keys
    float mx0 = kNegBig, mx1 = kNegBig;
#pragma unroll
    for (int nt = 0; nt < 2 * NK; ++nt) {
        const int k0 = nt * 8 + 2 * t;
        if (k0 >= nvalid) { s[nt][0] = -INFINITY; s[nt][2] = -INFINITY; }
        if (k0 + 1 >= nvalid) { s[nt][1] = -INFINITY; s[nt][3] = -INFINITY; }
        if (CAUSAL) {
            if (k0 > g) s[nt][0] = -INFINITY;
            if (k0 + 1 > g) s[nt][1] = -INFINITY;
            if (k0 > g + 8) s[nt][2] = -INFINITY;
            if (k0 + 1 > g + 8) s[nt][3] = -INFINITY;
        }
        mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
        mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float m0 = fmaxf(ws.m[0], mx0), m1 = fmaxf(ws.m[1], mx1);
    const float c0 = ex2(ws.m[0] - m0), c1 = ex2(ws.m[1] - m1);
    ws.m[0] = m0; ws.m[1] = m1;
    float l0 = 0.f, l1 = 0.f;
    unsigned ph[2][4];             // P as A fragments of the two 16-key steps (fp16: weights in [0, 1])
#pragma unroll
    for (int nt = 0; nt < 2 * NK; ++nt) {
        const float p0 = ex2(s[nt][0] - m0), p1 = ex2(s[nt][1] - m0);
        const float p2 = ex2(s[nt][2] - m1), p3 = ex2(s[nt][3] - m1);
        l0 += p0 + p1; l1 += p2 + p3;
        const int kk = nt >> 1, hi2 = (nt & 1) * 2;     // a0,a1 from the even key tile, a2,a3 from the odd one
        ph[kk][hi2] = pack_f16x2(p0, p1); ph[kk][hi2 + 1] = pack_f16x2(p2, p3);
    }
    ws.l[0] = ws.l[0] * c0 + l0;
    ws.l[1] = ws.l[1] * c1 + l1;
    if (__any_sync(0xffffffffu, c0 != 1.f || c1 != 1.f)) {     // a new maximum somewhere in the warp's rows
#pragma unroll
        for (int dn = 0; dn < DH / 8; ++dn) { ws.o[dn][0] *= c0; ws.o[dn][1] *= c0; ws.o[dn][2] *= c1; ws.o[dn][3] *= c1; }
    }
#pragma unroll
    for (int kk = 0; kk < NK; ++kk) {
#pragma unroll
        for (int dp = 0; dp < DH / 16; ++dp) {   // value columns 16dp .. 16dp+15 (chunks 2dp, 2dp+1)
            const int row = key0 + kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
            const int chunk = 2 * dp + (lane >> 4);
            unsigned vb[4];
            ldmatrix_x4_trans(vb, v_tile + (uint32_t)row * RB + (uint32_t)swz(row, chunk, RB) * 16u);
            mma16816_f16(ws.o[2 * dp], ph[kk][0], ph[kk][1], ph[kk][2], ph[kk][3], vb[0], vb[1]);
            mma16816_f16(ws.o[2 * dp + 1], ph[kk][0], ph[kk][1], ph[kk][2], ph[kk][3], vb[2], vb[3]);
        }
    }
}

// The same unit for at most eight query rows, transposed: S^T = K Q^T puts the 16 keys of a step on the M side of the
// product and the queries on its N side (8 wide: five query rows waste three columns instead of eleven rows), and
// O^T = V^T P^T likewise, so a unit is 24 products instead of 48.  A thread holds queries 2t, 2t+1 (columns of the
// accumulators) and keys / value columns g, g+8 (rows).  P^T reaches the B operand of the second product through
// movmatrix (an 8 x 8 transpose inside the warp).  The query fragments live in registers for the whole item.
template <int DH> struct WarpStateT {
    float o[DH / 16][4];          // rows 16 dp + g (0, 1) and + 8 (2, 3) of O^T; columns 2t (0, 2) and 2t + 1 (1, 3)
    float m[2], l[2];             // queries 2t, 2t + 1; l: this thread's keys only until the state is parked
};
__device__ __forceinline__ unsigned movmatrix_trans(unsigned a) {
    unsigned d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// query fragments (B operands): chunk c of 8 elements of query rows 0..7 -> qf[c]
template <int DH>
__device__ __forceinline__ void load_q_frags(uint32_t q_base, unsigned (&qf)[DH / 8]) {
    constexpr int QPB = (DH + 8) * 2;
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int c4 = 0; c4 < DH / 32; ++c4) {
        unsigned r[4];
        ldmatrix_x4(r, q_base + (uint32_t)(lane & 7) * QPB + (uint32_t)(4 * c4 + (lane >> 3)) * 16u);
        qf[4 * c4] = r[0]; qf[4 * c4 + 1] = r[1]; qf[4 * c4 + 2] = r[2]; qf[4 * c4 + 3] = r[3];
    }
}
template <int DH, bool CAUSAL>
__device__ __forceinline__ void attn_unit_t(const unsigned (&qh)[DH / 8], const unsigned (&ql)[DH / 8], uint32_t k_tile, uint32_t v_tile,
                                            int key0, int nvalid, WarpStateT<DH> &ws) {
    constexpr int RB = DH * 2;
    constexpr int NK = CAUSAL ? 1 : 2;      // 16-key steps: the window has at most 8 rows here
    const int lane = threadIdx.x & 31, t = lane & 3, g = lane >> 2;
    float s[NK][4];
#pragma unroll
    for (int kt = 0; kt < NK; ++kt) s[kt][0] = s[kt][1] = s[kt][2] = s[kt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
#pragma unroll
        for (int kt = 0; kt < NK; ++kt) {
            const int row = key0 + kt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
            const int chunk = 2 * ks + (lane >> 4);
            unsigned ka[4];
            ldmatrix_x4(ka, k_tile + (uint32_t)row * RB + (uint32_t)swz(row, chunk, RB) * 16u);
            mma16816_f16(s[kt], ka[0], ka[1], ka[2], ka[3], qh[2 * ks], qh[2 * ks + 1]);
            mma16816_f16(s[kt], ka[0], ka[1], ka[2], ka[3], ql[2 * ks], ql[2 * ks + 1]);
        }
    }
    // mask the keys past the end (and, window, after the query); column maxima over the keys
    float mx0 = kNegBig, mx1 = kNegBig;
#pragma unroll
    for (int kt = 0; kt < NK; ++kt) {
        const int r0 = kt * 16 + g, r1 = r0 + 8;
        if (r0 >= nvalid) { s[kt][0] = -INFINITY; s[kt][1] = -INFINITY; }
        if (r1 >= nvalid) { s[kt][2] = -INFINITY; s[kt][3] = -INFINITY; }
        if (CAUSAL) {
            if (r0 > 2 * t) s[kt][0] = -INFINITY;
            if (r0 > 2 * t + 1) s[kt][1] = -INFINITY;
            if (r1 > 2 * t) s[kt][2] = -INFINITY;
            if (r1 > 2 * t + 1) s[kt][3] = -INFINITY;
        }
        mx0 = fmaxf(mx0, fmaxf(s[kt][0], s[kt][2]));
        mx1 = fmaxf(mx1, fmaxf(s[kt][1], s[kt][3]));
    }
#pragma unroll
    for (int o = 4; o <= 16; o <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
    }
    const float m0 = fmaxf(ws.m[0], mx0), m1 = fmaxf(ws.m[1], mx1);
    const float c0 = ex2(ws.m[0] - m0), c1 = ex2(ws.m[1] - m1);
    ws.m[0] = m0; ws.m[1] = m1;
    float l0 = 0.f, l1 = 0.f;
    unsigned pb[NK][2];            // P^T as B fragments of the 16-key steps (fp16: weights in [0, 1])
#pragma unroll
    for (int kt = 0; kt < NK; ++kt) {
        const float p0 = ex2(s[kt][0] - m0), p1 = ex2(s[kt][1] - m1);
        const float p2 = ex2(s[kt][2] - m0), p3 = ex2(s[kt][3] - m1);
        l0 += p0 + p2; l1 += p1 + p3;
        pb[kt][0] = movmatrix_trans(pack_f16x2(p0, p1));      // keys 0..7 of the step
        pb[kt][1] = movmatrix_trans(pack_f16x2(p2, p3));      // keys 8..15
    }
    ws.l[0] = ws.l[0] * c0 + l0;
    ws.l[1] = ws.l[1] * c1 + l1;
    if (__any_sync(0xffffffffu, c0 != 1.f || c1 != 1.f)) {     // a new maximum somewhere in the warp's columns
#pragma unroll
        for (int dp = 0; dp < DH / 16; ++dp) { ws.o[dp][0] *= c0; ws.o[dp][1] *= c1; ws.o[dp][2] *= c0; ws.o[dp][3] *= c1; }
    }
#pragma unroll
    for (int kt = 0; kt < NK; ++kt) {
#pragma unroll
        for (int dp = 0; dp < DH / 16; ++dp) {   // value columns 16dp .. 16dp+15 (chunks 2dp, 2dp+1) are rows of O^T
            const int row = key0 + kt * 16 + (lane & 7) + ((lane >> 4) << 3);
            const int chunk = 2 * dp + ((lane >> 3) & 1);
            unsigned va[4];
            ldmatrix_x4_trans(va, v_tile + (uint32_t)row * RB + (uint32_t)swz(row, chunk, RB) * 16u);
            mma16816_f16(ws.o[dp], va[0], va[1], va[2], va[3], pb[kt][0], pb[kt][1]);
        }
    }
}

// One (sequence, head, split) item.  Self-attention: the K+1 window rows (positions len+j) against the
// cached keys of this split's pages; the last split also takes the window's own keys (row j sees window
// keys 0..j; 16-bit caches: one more tensor-core unit over a tile in the cache's format, fp32 caches: FMA) and
// appends them to the cache.  Cross-attention: the same rows against the cached
// condition keys, no mask, no rotation.  Splits leave (m, l, O) partials; the last split merges them.
// T8: the kernel instance runs at most eight token rows (so K + 1 <= 8) and holds the transposed unit only; the other
// instances of 16-bit models choose by K + 1.
template <typename WT, int DH, bool T8>
static __device__ void attn_item(const Dev &D, const Smem &S, Ring &ring, const Stage &st, const AttnItem &it, uint32_t serial) {
    typedef typename CacheT<WT>::type KVT;
    constexpr bool MMA = sizeof(KVT) == 2;
    static_assert(!T8 || MMA, "the transposed unit is for 16-bit caches");
    const bool cross = st.kind != ST_ATTN_SELF, headx = st.kind == ST_ATTN_HEAD;
    const int K1 = D.K1, P = D.P, d = D.d, half = DH / 2, b = it.b, h = it.h;
    const int kv_set = headx ? it.hd : st.layer;                       // which set of cache tiles: layer, or decoding head
    const int part_item = (headx ? it.hd * D.B * D.H : 0) + b * D.H + h;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = cross ? D.C : S.ctl->len[b];
    const bool win = !cross && it.s == it.S - 1;
    const bool merger = it.s == it.S - 1;
    const float *qsrc = headx ? D.qh + (size_t)it.hd * D.M * d : cross ? D.qc : D.qkv;
    const int q_ld = cross ? d : 3 * d;
    void *pool = headx ? D.hckv_pool : cross ? D.ckv_pool : D.kv_pool;
    const int pool_pages = cross ? D.B * D.cpages : D.n_pages;
    float *part = headx ? D.hpart : cross ? D.cpart : D.part;
    float *out = headx ? D.hattn + (size_t)it.hd * D.M * d : cross ? D.cattn : D.attn;
    const uint32_t tag_in = tag_of(serial, st.in), tag_out = tag_of(serial, st.outt), tag_part = tag_of(serial, st.part);
    AttnSmem<DH> A(S.acts, K1);
    const float qscale = D.scale * kLog2e;
    int p_lo, p_hi;
    split_pages(D, n, it.s, it.S, p_lo, p_hi);
    // q (and the window's k, v) of this head: 16-byte words, row r = i / (DH / 4) of [q | k | v][K1]; two per thread
    // are requested at once, and the first two before anything else (their round trip is the longest wait of the item)
    const int nsrc = win ? 3 : 1, n_q = nsrc * K1 * (DH / 4);
    auto q_word = [&](int i, int &row) -> const float * {
        const int r = i / (DH / 4), c4 = i - r * (DH / 4), which = (r >= K1 ? 1 : 0) + (r >= 2 * K1 ? 1 : 0), j = r - which * K1;
        row = r;
        return qsrc + (size_t)(b * K1 + j) * q_ld + which * d + h * DH + c4 * 4;
    };
    uint4 qw[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int i = tid + u * kConsumerThreads;
        int row;
        qw[u] = make_uint4(tag_in, tag_in, tag_in, tag_in);
        if (i < n_q) qw[u] = ld_relaxed_u4(q_word(i, row));
    }

    if (MMA && tid < S.n_slots) {
        // the fill of slot `tid` that precedes this item's first position has landed (a barrier of the CTA lies between).
        // Fills are numbered per item, modulo 4: the trip round the ring that the item starts in is number 1.
        const uint32_t slot0 = ring_slot(S, ring.pos);
        S.ctl->landed[tid] = (unsigned char)((uint32_t)tid < slot0 ? 1u : 0u);
    }
    csync();
    // the rotation table and the pages of the appended rows are fetched while q is awaited.  16-bit caches work on
    // pairs (e, e + half) of a row, one pass for up to seven rows; fp32 caches on single elements.
    constexpr int kRot = MMA ? (16 * half + kConsumerThreads - 1) / kConsumerThreads : (16 * DH + kConsumerThreads - 1) / kConsumerThreads;
    float2 cs_pre[kRot];
#pragma unroll
    for (int q = 0; q < kRot; ++q) {
        const int i = tid + q * kConsumerThreads, j = MMA ? i / half : i / DH, e = MMA ? i - j * half : (i - j * DH) % half;
        cs_pre[q] = make_float2(1.f, 0.f);
        if (!cross && j < K1) cs_pre[q] = __ldcg(D.rope_cs + (n + j) * half + e);
    }
    if constexpr (MMA) {
        // the unused query rows are zero; value rows past the window are multiplied by zero weights and must be finite
        const uint4 z4 = make_uint4(0u, 0u, 0u, 0u);
        const int nq16 = (16 - K1) * A.QP * 2 / 16, nv16 = win ? (16 - K1) * DH * 2 / 16 : 0;
        for (int i = tid; i < 2 * nq16 + nv16; i += kConsumerThreads) {
            uint4 *dst = i < nq16       ? reinterpret_cast<uint4 *>(A.qh + K1 * A.QP) + i
                         : i < 2 * nq16 ? reinterpret_cast<uint4 *>(A.ql + K1 * A.QP) + (i - nq16)
                                        : reinterpret_cast<uint4 *>(A.vt + K1 * DH) + (i - 2 * nq16);
            *dst = z4;
        }
    }
    int page_pre[2] = {0, 0};
    if (win) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int i = tid + q * kConsumerThreads;
            if (i < 2 * K1 * (DH / 8)) {
                const int j = (i - (i >= K1 * (DH / 8) ? K1 * (DH / 8) : 0)) / (DH / 8);
                page_pre[q] = __ldcg(D.block_table + (size_t)b * D.max_blocks + page_of(D, n + j));
            }
        }
    }
    // 1. q (and the window's k, v) arrive: raw[row][DH]
    for (int i0 = 0; i0 < n_q; i0 += 2 * kConsumerThreads) {
        if (i0 > 0) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int i = i0 + tid + u * kConsumerThreads;
                int row;
                if (i < n_q) qw[u] = ld_relaxed_u4(q_word(i, row));
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int i = i0 + tid + u * kConsumerThreads;
            if (i < n_q) {
                int row;
                const float *src = q_word(i, row);
                if (!tags_ok(qw[u], tag_in)) qw[u] = poll_u4(D, S.ctl, src, tag_in);
                *reinterpret_cast<float4 *>(A.raw + (size_t)row * DH + (i % (DH / 4)) * 4) =
                    make_float4(read_word<WT>(qw[u].x), read_word<WT>(qw[u].y), read_word<WT>(qw[u].z), read_word<WT>(qw[u].w));
            }
        }
    }
    csync();
    if (S.ctl->trace_row) trace_mark(D, S.ctl->trace_row);
    // 2. rotate, scale, split (fp32 caches: zero the unused query rows here)
    if constexpr (MMA) {
#pragma unroll
        for (int qq = 0; qq < kRot; ++qq) {
            const int i = tid + qq * kConsumerThreads;
            if (i >= K1 * half) break;
            const int j = i / half, e = i - j * half;
            float q0 = A.raw[j * DH + e], q1 = A.raw[j * DH + e + half];
            if (!cross) {
                const float2 cs = cs_pre[qq];
                const float r0 = q0 * cs.x - q1 * cs.y, r1 = q0 * cs.y + q1 * cs.x;
                q0 = r0; q1 = r1;
                if (win) {
                    const float k0 = A.raw[(K1 + j) * DH + e], k1 = A.raw[(K1 + j) * DH + e + half];
                    A.kt[tile_off<__half>(j, e, DH)] = from_f<__half>(k0 * cs.x - k1 * cs.y);
                    A.kt[tile_off<__half>(j, e + half, DH)] = from_f<__half>(k0 * cs.y + k1 * cs.x);
                    A.vt[tile_off<__half>(j, e, DH)] = from_f<__half>(A.raw[(2 * K1 + j) * DH + e]);
                    A.vt[tile_off<__half>(j, e + half, DH)] = from_f<__half>(A.raw[(2 * K1 + j) * DH + e + half]);
                }
            }
            unsigned hi, lo;
            split_f16(q0 * qscale, hi, lo);
            A.qh[j * A.QP + e] = __ushort_as_bfloat16((unsigned short)hi);
            A.ql[j * A.QP + e] = __ushort_as_bfloat16((unsigned short)lo);
            split_f16(q1 * qscale, hi, lo);
            A.qh[j * A.QP + e + half] = __ushort_as_bfloat16((unsigned short)hi);
            A.ql[j * A.QP + e + half] = __ushort_as_bfloat16((unsigned short)lo);
        }
    } else {
#pragma unroll
        for (int qq = 0; qq < kRot; ++qq) {
            const int i = tid + qq * kConsumerThreads;
            if (i >= 16 * DH) break;
            const int j = i / DH, e = i - j * DH;
            float q = 0.f;
            if (j < K1) {
                q = A.raw[j * DH + e];
                if (!cross) {
                    const float2 cs = cs_pre[qq];
                    const float o = A.raw[j * DH + (e < half ? e + half : e - half)];
                    q = e < half ? q * cs.x - o * cs.y : o * cs.y + q * cs.x;
                    if (win) {
                        const float kr = A.raw[(K1 + j) * DH + e], ko = A.raw[(K1 + j) * DH + (e < half ? e + half : e - half)];
                        const float kn = e < half ? kr * cs.x - ko * cs.y : ko * cs.y + kr * cs.x, vn = A.raw[(2 * K1 + j) * DH + e];
                        A.kw[j * DH + e] = kn;
                        A.vw[j * DH + e] = vn;
                    }
                }
                q *= qscale;
                A.qf[j * DH + e] = q;
            }
        }
    }
    csync();
    // 3. append the window's keys and values to the cache (positions n .. n+K1-1)
    if (win) {
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
            const int i = tid + qq * kConsumerThreads;
            if (i >= 2 * K1 * (DH / 8)) break;
            const int kv = i >= K1 * (DH / 8) ? 1 : 0, rem = i - kv * K1 * (DH / 8), j = rem / (DH / 8), c = rem - j * (DH / 8);
            const int pos = n + j, page = page_pre[qq], r = row_in_page(D, pos);
            KVT *tile = kv_tile<KVT>(D, pool, pool_pages, kv_set, kv, page, h);
            KVT *dst = tile + tile_off<KVT>(r, c * 8, DH);
            if constexpr (MMA) {
                // the window tiles hold the rows in the cache's own format: chunk c of row j goes to chunk c of row r
                *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>((kv ? A.vt : A.kt) + tile_off<__half>(j, c * 8, DH));
            } else {
                const float *src = (kv ? A.vw : A.kw) + j * DH + c * 8;
#pragma unroll
                for (int q = 0; q < 8; ++q) dst[q] = from_f<KVT>(src[q]);
            }
        }
    }
    // 4. the cached keys of this split
    WarpState<DH> ws;
#pragma unroll
    for (int dn = 0; dn < DH / 8; ++dn) ws.o[dn][0] = ws.o[dn][1] = ws.o[dn][2] = ws.o[dn][3] = 0.f;
    ws.m[0] = ws.m[1] = kNegBig;
    ws.l[0] = ws.l[1] = 0.f;
    WarpStateT<DH> wt;
#pragma unroll
    for (int dp = 0; dp < DH / 16; ++dp) wt.o[dp][0] = wt.o[dp][1] = wt.o[dp][2] = wt.o[dp][3] = 0.f;
    wt.m[0] = wt.m[1] = kNegBig;
    wt.l[0] = wt.l[1] = 0.f;
    float *my_st = A.st + (size_t)warp * K1 * (DH + 2);
    if constexpr (MMA) {
        const uint32_t q_hi = smem_u32(A.qh), q_lo = smem_u32(A.ql);
        const bool t8 = T8 || K1 <= 8;
        unsigned qfh[DH / 8], qfl[DH / 8];
        if (t8) { load_q_frags<DH>(q_hi, qfh); load_q_frags<DH>(q_lo, qfl); }
        // one unit of 32 cached keys, one of the window's own keys
        auto unit = [&](uint32_t ks, uint32_t vs, int key0, int nv) {
            if (t8) attn_unit_t<DH, false>(qfh, qfl, ks, vs, key0, nv, wt);
            else if constexpr (!T8) attn_unit<DH, false>(q_hi, q_lo, ks, vs, key0, nv, ws);
        };
        auto unit_window = [&]() {
            if (t8) attn_unit_t<DH, true>(qfh, qfl, smem_u32(A.kt), smem_u32(A.vt), 0, K1, wt);
            else if constexpr (!T8) attn_unit<DH, true>(q_hi, q_lo, smem_u32(A.kt), smem_u32(A.vt), 0, K1, ws);
        };
        const int upp = P / 32;   // 32-key units per page
        // Who touches a page.  Where a page is one ring item and the ring has a slot per consumer warp, the 32-key units
        // of the item go round the warps, unit u of page i to warp (i * upp + u) mod 7, and only the warps that own a
        // unit of a page look at it: they wait for the page and free the slot between them (seven arrivals: the owner
        // of unit 0 gives what the others leave); the other warps never touch that page (their per-page bookkeeping
        // would cost more than the units).  A warp that skips pages skips phases of a slot's barrier, and a parity
        // wait cannot tell "the fill before mine is still on its way" from "mine has landed".  So every owner records
        // the number (modulo 4) of the fill it has seen land (ctl->landed), and an owner tests the barrier only once
        // its slot's previous fill, or the awaited one (by a fellow owner), is recorded; with at least seven slots the
        // fill two before had completed when the owner's previous page landed, so two bits are enough.  Otherwise
        // every warp passes every page.
        const bool own = D.kv_one_item && S.n_slots >= kConsumerWarps && upp <= kConsumerWarps;
        const int n_it = D.kv_one_item ? 1 : 2, n_pages = p_hi - p_lo;
        if (own) {
            // this warp's units: slots warp, warp + 7, ... of the item's (page, unit) sequence
            uint32_t pos = ring.pos;
            uint32_t fill = 1u;                     // number of the trip round the ring that `pos` is in
            int cur = 0;                            // the page (relative to p_lo) that `pos` stands at
            for (int us = warp; us < n_pages * upp; us += kConsumerWarps) {
                const int rel = upp == 2 ? us >> 1 : upp == 1 ? us : us / upp, du = us - rel * upp;
                if (rel > cur) {                    // at most seven pages further: no more than one trip round the ring
                    if (ring_slot(S, pos) + (uint32_t)(rel - cur) >= (uint32_t)S.n_slots) ++fill;
                    pos = ring_add(S, pos, rel - cur);
                    cur = rel;
                }
                Ring r;
                r.pos = pos;
                const uint32_t slot = ring_slot(S, pos);
                if (lane == 0) {
                    const unsigned char prev = (unsigned char)((fill - 1u) & 3u), now = (unsigned char)(fill & 3u);
                    unsigned it2 = 0;
                    for (;;) {
                        const unsigned char seen = S.ctl->landed[slot];
                        if (seen == prev || seen == now || S.ctl->dead) break;
                        if (++it2 > D.mbar_limit) { raise_timeout(D, S.ctl); break; }
                    }
                }
                __syncwarp();
                const char *ks = ring_wait(D, S, r);
                if (lane == 0) S.ctl->landed[slot] = (unsigned char)(fill & 3u);
                const int nv = min(32, min(P, n - (p_lo + rel) * P) - du * 32);
                if (nv > 0) unit(smem_u32(ks), smem_u32(ks + D.tile_bytes), du * 32, nv);
                __syncwarp();
                if (lane < (du == 0 ? kConsumerWarps - (upp - 1) : 1)) mbar_arrive(S.empty0 + 8u * slot);
            }
            ring.pos = ring_add(S, ring.pos, n_pages);
        } else {
            uint32_t pos = ring.pos;
            for (int pg = p_lo; pg < p_hi; ++pg, pos = ring_add(S, pos, n_it)) {
                const int rel = pg - p_lo;
                Ring r;
                r.pos = pos;
                const char *ks = ring_wait(D, S, r);
                const char *vs = ks + D.tile_bytes;
                if (n_it == 2) { r.pos = ring_add(S, pos, 1); vs = ring_wait(D, S, r); }
                const int nv_page = min(P, n - pg * P);
                for (int u = 0; u < upp; ++u) {
                    const int nv = min(32, nv_page - u * 32);
                    if (nv > 0 && ((rel * upp + u) % kConsumerWarps) == warp) unit(smem_u32(ks), smem_u32(vs), u * 32, nv);
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(S.empty0 + 8u * ring_slot(S, pos));
                    if (n_it == 2) mbar_arrive(S.empty0 + 8u * ring_slot(S, r.pos));
                }
            }
            ring.pos = pos;
        }
        // the window's own keys, under the causal mask, as one more unit for the warp whose turn is next
        if (win && ((n_pages * upp) % kConsumerWarps) == warp) unit_window();
        const int g = lane >> 2, t = lane & 3;
        if (t8) {
            // the denominators over the key rows (lanes of equal t), then the state [query][element | m | l]
#pragma unroll
            for (int o = 4; o <= 16; o <<= 1) {
                wt.l[0] += __shfl_xor_sync(0xffffffffu, wt.l[0], o);
                wt.l[1] += __shfl_xor_sync(0xffffffffu, wt.l[1], o);
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int q = 2 * t + i;
                if (q < K1) {
#pragma unroll
                    for (int dp = 0; dp < DH / 16; ++dp) {
                        my_st[q * (DH + 2) + dp * 16 + g] = wt.o[dp][i];
                        my_st[q * (DH + 2) + dp * 16 + g + 8] = wt.o[dp][2 + i];
                    }
                    if (g == 0) { my_st[q * (DH + 2) + DH] = wt.m[i]; my_st[q * (DH + 2) + DH + 1] = wt.l[i]; }
                }
            }
        } else if constexpr (!T8) {
        // quad-reduce the denominators, park the state in shared memory
        ws.l[0] += __shfl_xor_sync(0xffffffffu, ws.l[0], 1); ws.l[0] += __shfl_xor_sync(0xffffffffu, ws.l[0], 2);
        ws.l[1] += __shfl_xor_sync(0xffffffffu, ws.l[1], 1); ws.l[1] += __shfl_xor_sync(0xffffffffu, ws.l[1], 2);
        if (g < K1) {
#pragma unroll
            for (int dn = 0; dn < DH / 8; ++dn) {
                my_st[g * (DH + 2) + dn * 8 + 2 * t] = ws.o[dn][0];
                my_st[g * (DH + 2) + dn * 8 + 2 * t + 1] = ws.o[dn][1];
            }
            if (t == 0) { my_st[g * (DH + 2) + DH] = ws.m[0]; my_st[g * (DH + 2) + DH + 1] = ws.l[0]; }
        }
        if (g + 8 < K1) {
#pragma unroll
            for (int dn = 0; dn < DH / 8; ++dn) {
                my_st[(g + 8) * (DH + 2) + dn * 8 + 2 * t] = ws.o[dn][2];
                my_st[(g + 8) * (DH + 2) + dn * 8 + 2 * t + 1] = ws.o[dn][3];
            }
            if (t == 0) { my_st[(g + 8) * (DH + 2) + DH] = ws.m[1]; my_st[(g + 8) * (DH + 2) + DH + 1] = ws.l[1]; }
        }
        }
    } else {
        // fp32 cache: one key per warp at a time, straight from global memory, all query rows at once
        constexpr int EPL = (DH + 31) / 32;
        const int e0 = lane * EPL;
        const bool lane_on = e0 < DH;
        const int key_lo = min(n, p_lo * P), key_hi = min(n, p_hi * P);
        for (int j0 = 0; j0 < K1; j0 += 8) {
            const int nq = min(8, K1 - j0);
            float q[8][EPL], acc[8][EPL], mx[8], l[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                mx[j] = kNegBig; l[j] = 0.f;
#pragma unroll
                for (int i = 0; i < EPL; ++i) { acc[j][i] = 0.f; q[j][i] = (j < nq && lane_on) ? A.qf[(j0 + j) * DH + e0 + i] : 0.f; }
            }
            for (int key = key_lo + warp; key < key_hi; key += kConsumerWarps) {
                const int page = cross ? b * D.cpages + key / P : __ldcg(D.block_table + (size_t)b * D.max_blocks + key / P);
                const KVT *kt = kv_tile<KVT>(D, pool, pool_pages, kv_set, 0, page, h) + (size_t)(key % P) * DH + e0;
                const KVT *vt = kv_tile<KVT>(D, pool, pool_pages, kv_set, 1, page, h) + (size_t)(key % P) * DH + e0;
                float kf[EPL], vf[EPL];
#pragma unroll
                for (int i = 0; i < EPL; ++i) {
                    kf[i] = lane_on ? to_f(__ldcg(kt + i)) : 0.f;
                    vf[i] = lane_on ? to_f(__ldcg(vt + i)) : 0.f;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (j < nq) {
                        float dsum = 0.f;
#pragma unroll
                        for (int i = 0; i < EPL; ++i) dsum = fmaf(q[j][i], kf[i], dsum);
                        dsum = warp_sum(dsum);
                        const float mn = fmaxf(mx[j], dsum), corr = exp2f(mx[j] - mn), pw = exp2f(dsum - mn);
                        l[j] = l[j] * corr + pw;
#pragma unroll
                        for (int i = 0; i < EPL; ++i) acc[j][i] = acc[j][i] * corr + pw * vf[i];
                        mx[j] = mn;
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j < nq) {
                    float *sw = my_st + (size_t)(j0 + j) * (DH + 2);
                    if (lane_on) {
#pragma unroll
                        for (int i = 0; i < EPL; ++i) sw[e0 + i] = acc[j][i];
                    }
                    if (lane == 0) { sw[DH] = mx[j]; sw[DH + 1] = l[j]; }
                }
            }
        }
    }
    // 5. fp32 cache: the window's own keys under the causal mask: query row j (one warp each) against window keys 0..j
    if constexpr (!MMA) {
        float *wst = A.st + (size_t)kConsumerWarps * K1 * (DH + 2);
        constexpr int EPL = (DH + 31) / 32;
        for (int j = warp; j < K1; j += kConsumerWarps) {
            float m = kNegBig, l = 0.f, acc[EPL];
#pragma unroll
            for (int i = 0; i < EPL; ++i) acc[i] = 0.f;
            if (win) {
                for (int wk = 0; wk <= j; ++wk) {
                    float dsum = 0.f;
#pragma unroll
                    for (int i = 0; i < EPL; ++i) {
                        const int e = lane + 32 * i;
                        if (e < DH) dsum = fmaf(A.qf[j * DH + e], A.kw[wk * DH + e], dsum);
                    }
                    dsum = warp_sum(dsum);
                    const float mn = fmaxf(m, dsum), corr = exp2f(m - mn), pw = exp2f(dsum - mn);
                    l = l * corr + pw;
#pragma unroll
                    for (int i = 0; i < EPL; ++i) {
                        const int e = lane + 32 * i;
                        if (e < DH) acc[i] = acc[i] * corr + pw * A.vw[wk * DH + e];
                    }
                    m = mn;
                }
            }
#pragma unroll
            for (int i = 0; i < EPL; ++i) {
                const int e = lane + 32 * i;
                if (e < DH) wst[j * (DH + 2) + e] = acc[i];
            }
            if (lane == 0) { wst[j * (DH + 2) + DH] = m; wst[j * (DH + 2) + DH + 1] = l; }
        }
    }
    csync();
    // 6. merge the warps (and, fp32 cache, the window state); element DH = denominator
    constexpr int n_states = MMA ? kConsumerWarps : kConsumerWarps + 1;
    if (it.S == 1) {
        // no other split: one thread per (query row, element) forms numerator and denominator from the same weights
        // and publishes the quotient (the same sums in the same order as the two passes below)
        for (int i = tid; i < K1 * DH; i += kConsumerThreads) {
            const int j = i / DH, e = i - j * DH;
            float m = kNegBig;
#pragma unroll
            for (int w = 0; w < n_states; ++w) m = fmaxf(m, A.st[((size_t)w * K1 + j) * (DH + 2) + DH]);
            float o = 0.f, l = 0.f;
#pragma unroll
            for (int w = 0; w < n_states; ++w) {
                const float *sw = A.st + ((size_t)w * K1 + j) * (DH + 2);
                const float wg = exp2f(sw[DH] - m);
                o += wg * sw[e];
                l += wg * sw[DH + 1];
            }
            st_relaxed_u32(out + (size_t)(b * K1 + j) * d + h * DH + e, publish_word<WT>(o / l, tag_out, false));
        }
        return;
    }
    float *mg = A.raw;    // [K1][DH + 2] merged (O, m, l); raw q/k/v are no longer needed
    for (int i = tid; i < K1 * (DH + 1); i += kConsumerThreads) {
        const int j = i / (DH + 1), e = i - j * (DH + 1);
        float m = kNegBig;
        for (int w = 0; w < n_states; ++w) m = fmaxf(m, A.st[((size_t)w * K1 + j) * (DH + 2) + DH]);
        float o = 0.f;
        for (int w = 0; w < n_states; ++w) {
            const float *sw = A.st + ((size_t)w * K1 + j) * (DH + 2);
            o += exp2f(sw[DH] - m) * (e < DH ? sw[e] : sw[DH + 1]);
        }
        mg[j * (DH + 2) + (e < DH ? e : DH + 1)] = o;
        if (e == DH) mg[j * (DH + 2) + DH] = m;
    }
    csync();
    if (!merger) {
        // leave the partial for the last split
        float *pr = part + ((size_t)part_item * D.S_max + it.s) * K1 * (DH + 2);
        for (int i = tid; i < K1 * (DH + 2); i += kConsumerThreads) st_relaxed_u32(pr + i, tagged(mg[i], tag_part));
        return;
    }
    if (it.S > 1) {
        // wait for the other splits and fold them in (fixed order).  The maximum and one numerator (or the
        // denominator) of up to eight splits are requested together, and the whole batch is requested again until
        // every word carries the tag: the cost is the arrival of the slowest split plus one round trip.
        for (int i = tid; i < K1 * (DH + 1); i += kConsumerThreads) {
            const int j = i / (DH + 1), e = i - j * (DH + 1);
            const int col = e < DH ? e : DH + 1;
            const float *pb = part + ((size_t)part_item * D.S_max) * K1 * (DH + 2) + (size_t)j * (DH + 2);
            const size_t sstride = (size_t)K1 * (DH + 2);
            const int nsp = it.S - 1;
            float m = mg[j * (DH + 2) + DH], o = mg[j * (DH + 2) + col];      // running maximum, sum scaled to it
            for (int s0 = 0; s0 < nsp; s0 += 8) {
                uint32_t wm[8], wo[8];
                for (unsigned tries = 0;; ++tries) {
                    bool ok = true;
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        wm[q] = wo[q] = tag_part;
                        if (s0 + q < nsp) {
                            wm[q] = ld_relaxed_u32(pb + (size_t)(s0 + q) * sstride + DH);
                            wo[q] = ld_relaxed_u32(pb + (size_t)(s0 + q) * sstride + col);
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 8; ++q) ok = ok && (wm[q] & 3u) == tag_part && (wo[q] & 3u) == tag_part;
                    if (ok || S.ctl->dead) break;
                    if (tries > D.spin_limit) { raise_timeout(D, S.ctl); break; }
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (s0 + q < nsp) {
                        const float pm = untag(wm[q]), mn = fmaxf(m, pm);
                        o = o * exp2f(m - mn) + exp2f(pm - mn) * untag(wo[q]);
                        m = mn;
                    }
                }
            }
            A.st[j * (DH + 2) + (e < DH ? e : DH + 1)] = o;   // st is free again: final numerators and denominator
        }
        csync();
        mg = A.st;
    }
    for (int i = tid; i < K1 * DH; i += kConsumerThreads) {
        const int j = i / DH, e = i - j * DH;
        st_relaxed_u32(out + (size_t)(b * K1 + j) * d + h * DH + e, publish_word<WT>(mg[j * (DH + 2) + e] / mg[j * (DH + 2) + DH + 1], tag_out, false));
    }
}

template <typename WT, int DH, bool T8>
static __device__ void consume_attn(const Dev &D, const Smem &S, Ring &ring, const Stage &st, uint32_t serial) {
    AttnItem it;
    for (int idx = blockIdx.x; attn_item_at(D, S.ctl, st.kind, idx, it); idx += gridDim.x)
        attn_item<WT, DH, T8>(D, S, ring, st, it, serial);
}

// ----------------------------------------------------------------- verify / accept length / resample

static __device__ float block_sum(float v, float *sh) {
    v = warp_sum(v);
    csync();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    csync();
    float s = 0.f;
    for (int w = 0; w < kConsumerWarps; ++w) s += sh[w];
    return s;
}
static __device__ float block_max(float v, float *sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    csync();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    csync();
    float s = -INFINITY;
    for (int w = 0; w < kConsumerWarps; ++w) s = fmaxf(s, sh[w]);
    return s;
}
// (logit, token) as one 64-bit key whose unsigned order is the ranking: larger logit first, then smaller token.
// 0 is below every key ("no candidate").  -0.0 ranks with +0.0.
__device__ __forceinline__ unsigned long long rank_key(float z, int idx) {
    uint32_t u = __float_as_uint(z + 0.0f);
    u ^= (u & 0x80000000u) ? 0xFFFFFFFFu : 0x80000000u;
    return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);
}
__device__ __forceinline__ float key_logit(unsigned long long k) {
    uint32_t u = (uint32_t)(k >> 32);
    u ^= (u & 0x80000000u) ? 0x80000000u : 0xFFFFFFFFu;
    return __uint_as_float(u);
}
__device__ __forceinline__ int key_token(unsigned long long k) { return (int)(0xFFFFFFFFu - (uint32_t)k); }
// largest key over the block; every thread gets it
static __device__ unsigned long long block_best(unsigned long long k, unsigned long long *sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, k, o);
        k = other > k ? other : k;
    }
    csync();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = k;
    csync();
    k = sh[0];
#pragma unroll
    for (int w = 1; w < kConsumerWarps; ++w) k = sh[w] > k ? sh[w] : k;
    return k;
}

// copies one tagged logits row into shared memory (waiting for it), tags stripped
static __device__ void fetch_row(const Dev &D, const Smem &S, const float *z, float *row, uint32_t tag) {
    const int V = D.V;
    csync();
    if ((V & 3) == 0) {   // rows start on 16-byte boundaries
        const int n4 = V >> 2;
        for (int i0 = 0; i0 < n4; i0 += kConsumerThreads * kPollBatch) {
            uint4 w[kPollBatch];
            for (;;) {       // the batch at once; after a wait for the first missing word, the batch again
                const float *stale = nullptr;
#pragma unroll
                for (int u = 0; u < kPollBatch; ++u) {
                    const int i = i0 + u * kConsumerThreads + threadIdx.x;
                    w[u] = i < n4 ? ld_relaxed_u4(z + 4 * i) : make_uint4(tag, tag, tag, tag);
                }
#pragma unroll
                for (int u = kPollBatch - 1; u >= 0; --u)
                    if (!tags_ok(w[u], tag)) stale = z + 4 * (i0 + u * kConsumerThreads + threadIdx.x);
                if (stale == nullptr) break;
                poll_u4(D, S.ctl, stale, tag);
                if (S.ctl->dead) break;
            }
#pragma unroll
            for (int u = 0; u < kPollBatch; ++u) {
                const int i = i0 + u * kConsumerThreads + threadIdx.x;
                if (i < n4)
                    *reinterpret_cast<float4 *>(row + 4 * i) = make_float4(untag(w[u].x), untag(w[u].y), untag(w[u].z), untag(w[u].w));
            }
        }
    } else {
        for (int i = threadIdx.x; i < V; i += kConsumerThreads) row[i] = untag(poll_u32(D, S.ctl, z + i, tag));
    }
    csync();
}

// acceptance of token x under backbone logits z (shared memory), block-wide; every thread returns the same answer
static __device__ bool accept_token(const Dev &D, const float *z, int x, float *sh) {
    const int V = D.V;
    if (x < 0 || x >= V) return false;
    if (D.verify_mode == 2) {     // p0(x) > delta
        float m = -INFINITY;
        for (int v = threadIdx.x; v < V; v += kConsumerThreads) m = fmaxf(m, z[v]);
        m = block_max(m, sh);
        float sum = 0.f;
        for (int v = threadIdx.x; v < V; v += kConsumerThreads) sum += expf(z[v] - m);
        sum = block_sum(sum, sh);
        return expf(z[x] - m) / sum > D.delta;
    }
    const int ka = D.verify_mode == 0 ? 1 : D.k_accept;
    const unsigned long long kx = rank_key(z[x], x);
    float cnt = 0.f;
    for (int v = threadIdx.x; v < V; v += kConsumerThreads) cnt += rank_key(z[v], v) > kx ? 1.f : 0.f;
    cnt = block_sum(cnt, sh);
    return (int)cnt < ka;
}

// the k best (logit, token) pairs of z, ranked, left in shared memory: cv[j], ci[j] (behind the reduction scratch in sh)
static __device__ void top_candidates(const Dev &D, const float *z, int k, float *sh) {
    const int V = D.V;
    unsigned long long *shk = reinterpret_cast<unsigned long long *>(sh);   // [kConsumerWarps], 8-byte aligned
    float *cv = sh + 2 * kConsumerWarps + 2;           // candidates (value, index), up to 64
    int *ci = reinterpret_cast<int *>(cv + 64);
    // every thread keeps the best of its own elements; after each pick only the thread that owned the winner
    // looks for its next best (among its elements ranked after the winner)
    unsigned long long mine = 0ull;
    for (int v = threadIdx.x; v < V; v += kConsumerThreads) {
        const unsigned long long kv = rank_key(z[v], v);
        mine = kv > mine ? kv : mine;
    }
    for (int j = 0; j < k; ++j) {
        const unsigned long long win = block_best(mine, shk);
        if (threadIdx.x == 0) { cv[j] = key_logit(win); ci[j] = key_token(win); }
        if (win == mine && j + 1 < k) {      // mine was picked
            mine = 0ull;
            for (int v = threadIdx.x; v < V; v += kConsumerThreads) {
                const unsigned long long kv = rank_key(z[v], v);
                if (kv < win && kv > mine) mine = kv;
            }
        }
    }
}

static __device__ int sample_token(const Dev &D, const float *z, uint32_t r24, float *sh) {
    const int V = D.V;
    float *cv = sh + 2 * kConsumerWarps + 2;
    int *ci = reinterpret_cast<int *>(cv + 64);
    int *pick_s = ci + 64;
    const int k = D.sample_mode == 0 ? 1 : min(max(D.k_sample, 1), min(V, 64));
    top_candidates(D, z, k, sh);
    csync();
    if (threadIdx.x == 0) {
        int pick = ci[0];
        if (D.sample_mode != 0) {
            float total = 0.f;      // the weights are evaluated twice rather than kept in a local array
            for (int j = 0; j < k; ++j) total += expf((cv[j] - cv[0]) / D.temperature);
            const float u = (float)r24 * (1.0f / 16777216.0f);
            float cum = 0.f;
            pick = ci[k - 1];
            for (int j = 0; j < k; ++j) {
                cum += expf((cv[j] - cv[0]) / D.temperature);
                if (cum > u * total) { pick = ci[j]; break; }
            }
        }
        *pick_s = pick;
    }
    csync();
    return *pick_s;
}

// Top-K_s probability tree over the decoding heads (Appendix, Ablation of Sampling Strategies): the leaves are the
// K_s^K paths in lexicographic order of the heads' ranked candidates, a path weighs the product of its tokens'
// full-vocabulary probabilities, paths whose product falls below 1e-5 are pruned, and the first leaf whose cumulative
// weight exceeds u * total is drawn (the last surviving leaf if rounding keeps the sum below; the most probable token of
// every head if no path survives).  One warp; m, tok: [K][8] in shared memory.  Returns the leaf's index.
static __device__ int tree_pick(int K, int ks, const double *m, double u) {
    const int lane = threadIdx.x & 31;
    int n_leaves = 1;
    for (int d = 0; d < K; ++d) n_leaves *= ks;
    auto weight = [&](int idx) -> double {
        if (idx >= n_leaves) return 0.0;
        double w = 1.0;
        int div = n_leaves;
        for (int d = 0; d < K; ++d) {
            div /= ks;
            const int k = idx / div;
            idx -= k * div;
            w *= m[d * 8 + k];
            if (w < 1e-5) return 0.0;
        }
        return w;
    };
    double total = 0.0;
    for (int base = 0; base < n_leaves; base += 32) total += weight(base + lane);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    if (!(total > 0.0)) return 0;
    const double target = u * total;
    double cum = 0.0;
    int last = 0;
    for (int base = 0; base < n_leaves; base += 32) {
        const double w = weight(base + lane);
        double c = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, c, o);
            if (lane >= o) c += up;
        }
        c += cum;
        const unsigned alive = __ballot_sync(0xffffffffu, w > 0.0), hit = __ballot_sync(0xffffffffu, w > 0.0 && c > target);
        if (hit) return base + __ffs(hit) - 1;
        if (alive) last = base + 31 - __clz(alive);
        cum = __shfl_sync(0xffffffffu, c, 31);
    }
    return last;
}

// item (sequence b, slot): slot 0 resamples x_{s*} from the backbone row of the first rejection, slot i
// from head i's logits of the same row (independent sampling).  Every item recomputes the accept length.
// (not inlined, and handed nothing whose address would pin the caller's registers to memory: the shared-memory
// plan is derived again from the kernel's parameters)
static __device__ __noinline__ void sample_stage(const Dev &D, uint32_t serial) {
    extern __shared__ __align__(1024) char smem[];
    const Smem S = carve(smem, D);
    const int K1 = D.K1, K = D.K, V = D.V;
    const TagRef once = {1, 0};
    const uint32_t tag = tag_of(serial, once);
    float *row = reinterpret_cast<float *>(S.acts);
    float *sh = row + ((V + 3) & ~3);
    for (int it = blockIdx.x; it < D.B * K1; it += gridDim.x) {
        const int b = it / K1, slot = it % K1;
        if (S.ctl->flags[b] & 3) continue;
        int a = 0;
        while (a < K) {
            const int x = __ldcg(D.window + b * K1 + a + 1);
            fetch_row(D, S, D.logits0 + (size_t)(b * K1 + a) * V, row, tag);
            if (!accept_token(D, row, x, sh)) break;
            ++a;
        }
        const float *z = slot == 0 ? D.logits0 + (size_t)(b * K1 + a) * V
                                   : D.hlogits + ((size_t)(slot - 1) * D.M + b * K1 + a) * V;
        if (!(slot == 0 && a < K)) fetch_row(D, S, z, row, tag);      // slot 0: the row that rejected its draft is still staged
        if (D.sample_mode == 2 && slot > 0) {
            // probability tree: this head's K_s best tokens and their probabilities for the item of slot 1, which
            // draws one path for all heads
            const int ks = min(max(D.k_sample, 1), min(V, 8));
            float *cv = sh + 2 * kConsumerWarps + 2;
            int *ci = reinterpret_cast<int *>(cv + 64);
            top_candidates(D, row, ks, sh);
            csync();
            const float mx = cv[0];
            float sum = 0.f;
            for (int v = threadIdx.x; v < V; v += kConsumerThreads) sum += expf(row[v] - mx);
            sum = block_sum(sum, sh + 2 * kConsumerWarps + 2 + 192);
            uint32_t *tw = D.treex + ((size_t)(b * K + slot - 1) * 8) * 2;
            if (threadIdx.x < ks) {
                st_relaxed_u32(tw + 2 * threadIdx.x, tagged_int(ci[threadIdx.x], tag));
                st_relaxed_u32(tw + 2 * threadIdx.x + 1, tagged(expf(cv[threadIdx.x] - mx) / sum, tag));
            }
            if (slot == 1) {
                double *m = reinterpret_cast<double *>(sh + 512);          // [K][8], 8-byte aligned (sh is 16-byte aligned)
                int *tk = reinterpret_cast<int *>(m + kMaxDraft * 8);      // [K][8]
                csync();
                for (int i = threadIdx.x; i < K * ks; i += kConsumerThreads) {
                    const int d = i / ks, j = i - d * ks;
                    const uint32_t *src = D.treex + ((size_t)(b * K + d) * 8 + j) * 2;
                    tk[d * 8 + j] = untag_int(poll_u32(D, S.ctl, src, tag));
                    m[d * 8 + j] = (double)untag(poll_u32(D, S.ctl, src + 1, tag));
                }
                csync();
                if (threadIdx.x < 32) {
                    const double u = (double)rand24(D, b, __ldcg(D.step_idx + b), 1u, 0u) * (1.0 / 16777216.0);
                    int leaf = tree_pick(K, ks, m, u);
                    int div = 1;
                    for (int d = 0; d < K; ++d) div *= ks;
                    for (int d = 0; d < K; ++d) {
                        div /= ks;
                        const int k = leaf / div;
                        leaf -= k * div;
                        if (threadIdx.x == 0) st_relaxed_u32(D.candx + (size_t)b * (K1 + 1) + 1 + d, tagged_int(tk[d * 8 + k], tag));
                    }
                }
            }
            continue;
        }
        const uint32_t r = rand24(D, b, __ldcg(D.step_idx + b), (uint32_t)slot, 0u);
        const int tok = sample_token(D, row, r, sh);
        if (threadIdx.x == 0) {
            st_relaxed_u32(D.candx + (size_t)b * (K1 + 1) + slot, tagged_int(tok, tag));
            if (slot == 0) st_relaxed_u32(D.candx + (size_t)b * (K1 + 1) + K1, tagged_int(a, tag));
        }
    }
}

// ---------------------------------------------------------------------------- commit / next window

// After the length and the window of sequence b are final: reserve cache pages for positions < len + K + 1,
// gather the embeddings of the window into the residual stream (master copy and tagged copy for the step
// `serial`), and tabulate cos/sin of the window rows' positions.  Threads 0..nthr-1 take part; `win` may point to
// shared or global memory; nb_held = pages the sequence holds already.
template <typename WT> __device__ void prepare_window(const Dev &D, int b, uint32_t serial, int len, int nb_held, const int *win, int nthr,
                                                      float *scratch) {
    const int K1 = D.K1, d = D.d;
    const TagRef hemb = {3 * D.L + 1, 0};
    const uint32_t tag = tag_of(serial, hemb);
    if (threadIdx.x == 0) {
        const int need = (len + K1 + D.P - 1) / D.P;
        int nb = nb_held;
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
        if (nb != nb_held) __stcg(D.n_blocks + b, nb);
    }
    const WT *E = reinterpret_cast<const WT *>(D.E);
    const WT *g0 = reinterpret_cast<const WT *>(D.gain_first);
    // Embedding -> master copy and published copy (bf16 models: times the gain of the step's first RMSNorm, with
    // the row's sum of squares as this writer's share and zero shares for the rest).  A task is 16 bytes of one
    // embedding row; every thread keeps two of them in flight (more would raise the
    // register demand of the whole kernel).
    constexpr int EPC = 16 / (int)sizeof(WT);       // elements per task
    const int nch = d / EPC, total = K1 * nch;
    for (int t0 = threadIdx.x; t0 < total; t0 += 2 * nthr) {
        uint4 ev[2], gv[2];
        int tj[2], tc[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int t = t0 + u * nthr;
            tj[u] = -1; tc[u] = 0;
            if (t < total) {
                tj[u] = t / nch; tc[u] = t - tj[u] * nch;
                const int tok = min(max(win[tj[u]], 0), D.V - 1);
                ev[u] = __ldg(reinterpret_cast<const uint4 *>(E + (size_t)tok * d) + tc[u]);
                if (sizeof(WT) == 2) gv[u] = __ldg(reinterpret_cast<const uint4 *>(g0) + tc[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (tj[u] < 0) continue;
            const int row = b * K1 + tj[u];
            float v[EPC], gn[EPC];
            if (sizeof(WT) == 2) {
                const uint32_t ew[4] = {ev[u].x, ev[u].y, ev[u].z, ev[u].w}, gw[4] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    v[2 * q] = __uint_as_float(ew[q] << 16); v[2 * q + 1] = __uint_as_float(ew[q] & 0xFFFF0000u);
                    gn[2 * q] = __uint_as_float(gw[q] << 16); gn[2 * q + 1] = __uint_as_float(gw[q] & 0xFFFF0000u);
                }
            } else {
                v[0] = __uint_as_float(ev[u].x); v[1] = __uint_as_float(ev[u].y);
                v[2] = __uint_as_float(ev[u].z); v[3] = __uint_as_float(ev[u].w);
#pragma unroll
                for (int q = 0; q < EPC; ++q) gn[q] = 1.f;
            }
            float ssq = 0.f;
            float *hm = D.h + (size_t)row * d + tc[u] * EPC;
            float *hp = D.hpub + (size_t)row * d + tc[u] * EPC;
#pragma unroll
            for (int q = 0; q < EPC; q += 4) {
                __stcg(reinterpret_cast<float4 *>(hm + q), make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]));
                uint4 pw;
                pw.x = publish_word<WT>(v[q] * gn[q], tag, false); pw.y = publish_word<WT>(v[q + 1] * gn[q + 1], tag, false);
                pw.z = publish_word<WT>(v[q + 2] * gn[q + 2], tag, false); pw.w = publish_word<WT>(v[q + 3] * gn[q + 3], tag, false);
                __stcg(reinterpret_cast<uint4 *>(hp + q), pw);
                ssq += v[q] * v[q] + v[q + 1] * v[q + 1] + v[q + 2] * v[q + 2] + v[q + 3] * v[q + 3];
            }
            if (sizeof(WT) == 2) scratch[tj[u] * nch + tc[u]] = ssq;
        }
    }
    if (sizeof(WT) == 2) {
        if (nthr == kConsumerThreads) csync(); else __syncthreads();
        // the partial sums of a row are added in one fixed order
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = nthr >> 5;
        for (int j = warp; j < K1; j += nwarps) {
            float ssq = 0.f;
            for (int c = lane; c < nch; c += 32) ssq += scratch[j * nch + c];
            ssq = warp_sum(ssq);
            const int row = b * K1 + j;
            for (int c = lane; c < D.grid; c += 32) st_relaxed_u32(ss_word(D, c, row), tagged(c == 0 ? ssq : 0.f, tag));
        }
    }
}

// publishes the header of sequence b for step `serial` (after everything else of the sequence is written);
// threads 0..3 of the block write one word each
static __device__ void publish_header(const Dev &D, int b, uint32_t serial, int len, int flags) {
    const TagRef once = {1, 0};
    const uint32_t tag = tag_of(serial, once);
    uint32_t *hd = D.header + (size_t)b * kHeaderWords;
    if (threadIdx.x < kHeaderWords)
        st_relaxed_u32(hd + threadIdx.x, tagged_int(threadIdx.x == 0 ? len : threadIdx.x == 1 ? flags : 0, tag));
}

static __device__ void draw_initial_drafts(const Dev &D, int b, int *win) {
    for (int i = 1; i <= D.K; ++i) {
        const unsigned long long m = rand24(D, b, 0u, (uint32_t)i, 1u);
        win[i] = (int)((m * (unsigned long long)D.V) >> 24);
    }
}

// Algorithm 1 line 12 and the loop guard: commit x_{s+1..s*}, s <- s*, next window <- candidates.
template <typename WT> __device__ __noinline__ void commit_stage(const Dev &D, uint32_t serial) {
    extern __shared__ __align__(1024) char smem[];
    const Smem S = carve(smem, D);
    const int K1 = D.K1, tid = threadIdx.x;
    const TagRef once = {1, 0};
    const uint32_t tag = tag_of(serial, once);
    // scratch words in shared memory
    int *sm = reinterpret_cast<int *>(S.acts);
    int *s_cand = sm + 8;                 // [K1] resampled tokens, [K1] accept length
    int *s_state = sm + 40;               // len, ingest_left, n_gen, step_idx, n_blocks
    int *s_win = sm + 64;                 // [K1] window before, then after
    enum { O_LEN = 0, O_FLAGS = 1 };      // sm[0], sm[1]: new length and flags
    if ((int)blockIdx.x < D.B) {
        for (int c = tid; c < (int)gridDim.x; c += kConsumerThreads) poll_u32(D, S.ctl, D.done + c, tag);
        __threadfence();
    }
    for (int b = blockIdx.x; b < D.B; b += gridDim.x) {
        csync();
        const int fl = S.ctl->flags[b];
        // every word the commit needs, fetched side by side
        if (!(fl & 1)) {
            if (tid <= K1 && !(fl & 2)) s_cand[tid] = untag_int(poll_u32(D, S.ctl, D.candx + (size_t)b * (K1 + 1) + tid, tag));
            if (tid == 32) s_state[0] = __ldcg(D.len + b);
            if (tid == 33) s_state[1] = __ldcg(D.ingest_left + b);
            if (tid == 34) s_state[2] = __ldcg(D.n_gen + b);
            if (tid == 35) s_state[3] = (int)__ldcg(D.step_idx + b);
            if (tid == 36) s_state[4] = __ldcg(D.n_blocks + b);
            if (tid >= 64 && tid < 64 + K1) s_win[tid - 64] = __ldcg(D.window + b * K1 + tid - 64);
        }
        csync();
        if (tid == 0) {
            int len = S.ctl->len[b], flags = fl;
            if (!(fl & 1)) {
                len = s_state[0];
                const int left = s_state[1];
                if (left > 0) {
                    // prompt ingestion: the window held prompt tokens; all of them that are prompt enter the cache
                    const int n = min(K1, left);
                    len += n;
                    __stcg(D.ingest_left + b, left - n);
                    __stcg(D.step_n_new + b, 0);
                    const int *pr = D.prompt + (size_t)b * D.prompt_len;
                    if (left - n > 0) {
                        for (int j = 0; j < K1; ++j) s_win[j] = len + j < D.prompt_len ? pr[len + j] : 0;
                        flags = 2;
                    } else {
                        s_win[0] = pr[D.prompt_len - 1];
                        draw_initial_drafts(D, b, s_win);
                        flags = 0;
                    }
                } else {
                    const int a = min(max(s_cand[K1], 0), D.K);
                    __stcg(D.acc_len + b, a);
                    // scripted drafts: the token at the first rejected position is the script's as well, so that a near-tie
                    // of the backbone's two best logits cannot take the run off the script for good
                    if (D.script != nullptr && len + a + 1 < D.script_n) s_cand[0] = D.script[(size_t)b * D.script_n + len + a + 1];
                    int n_gen = s_state[2], fin = 0, n_out = 0;
                    for (int j = 0; j <= a; ++j) {
                        const int tok = j < a ? s_win[j + 1] : s_cand[0];
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
                    __stcg(D.n_gen + b, n_gen);
                    for (int j = 0; j < K1; ++j) {
                        s_win[j] = s_cand[j];
                        __stcg(D.cand + b * K1 + j, s_cand[j]);
                    }
                    if (D.script != nullptr) {
                        // scripted drafts: the next window drafts the script's tokens; the first `keep` stay as they
                        // are, the others are made wrong (a forced accept length for a backbone that reproduces the script)
                        const long long t = (long long)s_state[3] + 1;
                        const int keep = (int)((((t + 1) * D.script_acc) >> 10) - ((t * D.script_acc) >> 10));
                        const int *sc = D.script + (size_t)b * D.script_n;
                        for (int j = 1; j < K1; ++j) {
                            const int pos = len + j;
                            int tok = pos < D.script_n ? sc[pos] : 0;
                            if (j > keep) tok = tok + 1 < D.V ? tok + 1 : 0;
                            s_win[j] = tok;
                        }
                    }
                    __stcg(D.step_idx + b, (uint32_t)s_state[3] + 1u);
                    atomicAdd(D.hist + (size_t)b * (kMaxDraft + 1) + a, 1ull);
                    atomicAdd(D.steps + b, 1ull);
                    if (fin) {
                        __stcg(D.finished + b, 1);
                        atomicSub(D.n_active, 1);
                        flags = 1;
                    }
                }
                __stcg(D.len + b, len);
                for (int j = 0; j < K1; ++j) __stcg(D.window + b * K1 + j, s_win[j]);
            } else {
                __stcg(D.step_n_new + b, 0);
            }
            sm[O_LEN] = len;
            sm[O_FLAGS] = flags;
        }
        csync();
        if (!(sm[O_FLAGS] & 1))
            prepare_window<WT>(D, b, serial + 1u, sm[O_LEN], s_state[4], s_win, kConsumerThreads, reinterpret_cast<float *>(sm + 128));
        __threadfence();
        csync();
        publish_header(D, b, serial + 1u, sm[O_LEN], sm[O_FLAGS]);
    }
}

// ------------------------------------------------------------------------------------ step kernel

// The projection and attention stages [p_lo, p_hi) of one step, consumer side.  Returns the ring position.
template <typename WT, int NTM, int DH>
static __device__ __forceinline__ uint32_t consume_stages(const Dev &D, const Smem &S, uint32_t serial, uint32_t ring_pos,
                                                          int p_lo, int p_hi, int tracing) {
    Ring ring;
    ring.pos = ring_pos;
    for (int p = p_lo; p < p_hi; ++p) {
        const Stage st = stage_at(D, S, p);
        if (threadIdx.x == 0) S.ctl->trace_row = tracing ? 1 + 2 * p : 0;
        if (st.kind == ST_GEMV) gemv_stage<WT, NTM, false>(D, S, ring, st, serial);
        else if (st.kind == ST_ATTN_SELF || st.kind == ST_ATTN_CROSS || st.kind == ST_ATTN_HEAD) consume_attn<WT, DH, sizeof(WT) == 2 && NTM == 1>(D, S, ring, st, serial);
        if (tracing) trace_mark(D, 2 + 2 * p);
    }
    return ring.pos;
}

// the same stages seen by the producer warp
template <typename WT, int NTM>
static __device__ __forceinline__ uint32_t produce_stages(const Dev &D, const Smem &S, uint32_t ring_pos, int p_lo, int p_hi) {
    Ring ring;
    ring.pos = ring_pos;
    for (int p = p_lo; p < p_hi; ++p) {
        const Stage st = stage_at(D, S, p);
        if (st.kind == ST_GEMV) gemv_stage<WT, NTM, true>(D, S, ring, st, 0u);
        else if (st.kind == ST_ATTN_SELF || st.kind == ST_ATTN_CROSS || st.kind == ST_ATTN_HEAD) produce_attn<WT>(D, S, ring, st);
    }
    return ring.pos;
}

// One instance per (weight type, token capacity, head width): each carries only its own code path.
// The last two stages of a step are verify/resample and commit; all stages before them stream through the ring.
template <typename WT, int NTM, int DH>
__global__ void __launch_bounds__(kThreads, 1)
step_kernel(const __grid_constant__ Dev D, int st_lo, int st_hi, int n_steps, uint32_t serial0) {
    extern __shared__ __align__(1024) char smem[];
    const Smem S = carve(smem, D);
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        for (int i = 0; i < S.n_slots; ++i) {
            mbar_init(S.full0 + 8u * i, 1u);
            mbar_init(S.empty0 + 8u * i, (uint32_t)kConsumerWarps);
        }
        mbar_init(S.go_bar, 1u);
        mbar_init(S.abar0, 1u);
        mbar_init(S.abar0 + 8u, 1u);
        mbar_init(S.dbar, (uint32_t)umma_issuers(D.M));
        mbar_init(S.sbar0, (uint32_t)(kConsumerWarps - umma_issuers(D.M)));
        mbar_init(S.sbar0 + 8u, (uint32_t)(kConsumerWarps - umma_issuers(D.M)));
        S.ctl->dead = 0;
        S.ctl->dead_allowance = 1 << 22;
        S.ctl->go = 0;
        S.ctl->umma_chunks = 0u;
        S.ctl->umma_tiles = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    {   // the tables move to shared memory once per launch
        const uint32_t *src = reinterpret_cast<const uint32_t *>(D.tables);
        uint32_t *dst = reinterpret_cast<uint32_t *>(smem + kSmemHeader);
        for (int i = tid; i < min(D.tab_bytes, (int)sizeof(Tables)) / 4; i += kThreads) dst[i] = __ldg(src + i);
    }
    __syncthreads();
    plan_segments<WT>(D, S);
    const bool use_tmem = sizeof(WT) == 2 && NTM > 1 && D.umma != 0;
    if (use_tmem && warp == 0) {     // the accumulator columns of the tcgen05 projections, held until the launch ends
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&S.ctl->tmem)), "r"(kUmmaTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        tcgen05_before_sync();
    }
    __syncthreads();
    if (use_tmem) tcgen05_after_sync();
    uint32_t ring_pos = 0;
    const TagRef once = {1, 0};
    const int p_sample = D.n_stages - 2, p_commit = D.n_stages - 1;
    const int ring_hi = min(st_hi, p_sample);          // stages [st_lo, ring_hi) use the ring
    if (warp == kConsumerWarps) {
        // ---- producer warp
        for (int t = 0; t < n_steps; ++t) {
            mbar_wait(D, S.ctl, S.go_bar, (uint32_t)t & 1u);
            if (!S.ctl->go) break;
            fence_proxy_async();   // cache rows written by other CTAs in the previous step, read below by bulk copies
            ring_pos = produce_stages<WT, NTM>(D, S, ring_pos, st_lo, ring_hi);
        }
        return;
    }
    // ---- consumer warps
    for (int t = 0; t < n_steps; ++t) {
        const uint32_t serial = serial0 + (uint32_t)t;
        // the step header: length and flags of every sequence, published by the previous commit (or by prefill)
        csync();
        int any = 0;
        {
            const uint32_t tag = tag_of(serial, once);
            for (int b = tid; b < D.B; b += kConsumerThreads) {
                const uint32_t *hd = D.header + (size_t)b * kHeaderWords;
                S.ctl->len[b] = untag_int(poll_u32(D, S.ctl, hd, tag));
                S.ctl->flags[b] = untag_int(poll_u32(D, S.ctl, hd + 1, tag));
            }
            __threadfence();   // what the publisher wrote before the header (pages, rope table, master h) is visible now
            csync();
            for (int m = tid; m < D.M; m += kConsumerThreads) S.ctl->row_dead[m] = (unsigned char)(S.ctl->flags[m / D.K1] & 1);
            int fin = 0;
            for (int b = 0; b < D.B; ++b) { any |= !(S.ctl->flags[b] & 1); fin |= S.ctl->flags[b] & 1; }
            if (tid == 0) S.ctl->any_dead = fin;
            if (S.ctl->dead) any = 0;
        }
        if (tid == 0) {
            S.ctl->go = any;
            mbar_arrive(S.go_bar);
        }
        if (!any) break;
        const int tracing = D.trace != nullptr && t == 0;
        if (tracing) trace_mark(D, 0);
        ring_pos = consume_stages<WT, NTM, DH>(D, S, serial, ring_pos, st_lo, ring_hi, tracing);
        if (st_lo <= p_sample && p_sample < st_hi) {
            // everything this CTA wrote in the step (cache rows above all) is ordered before its mark;
            // the commit waits for every CTA's mark before it publishes the next step's header
            __threadfence();
            csync();
            if (tid == 0) st_relaxed_u32(D.done + blockIdx.x, tagged_int(0, tag_of(serial, once)));
            sample_stage(D, serial);
            if (tracing) trace_mark(D, 2 + 2 * p_sample);
        }
        if (st_lo <= p_commit && p_commit < st_hi) {
            commit_stage<WT>(D, serial);
            if (tracing) trace_mark(D, 2 + 2 * p_commit);
        }
    }
    if (use_tmem) {     // every product has been waited for; the columns go back before the CTA ends
        tcgen05_before_sync();
        csync();
        if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(S.ctl->tmem), "r"(kUmmaTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------ host side of the step kernel

template <typename WT, int NTM, int DH>
cudaError_t launch_step_instance(const Dev &D, int st_lo, int st_hi, int n_steps, uint32_t serial0, int grid, int smem_bytes,
                                 cudaStream_t st, int *max_grid) {
    const void *fn = (const void *)step_kernel<WT, NTM, DH>;
    // largest dynamic shared memory this instance has been opened for, per device (the attribute is per device)
    static std::atomic<int> attr_bytes[kMaxDevices];
    cudaError_t e;
    int cur_dev = 0;
    if ((e = cudaGetDevice(&cur_dev)) != cudaSuccess) return e;
    if (cur_dev < 0 || cur_dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (smem_bytes > attr_bytes[cur_dev].load()) {
        if ((e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes)) != cudaSuccess) return e;
        attr_bytes[cur_dev].store(smem_bytes);
    }
    if (max_grid != nullptr) {     // set-up query: how many CTAs can be resident
        int dev = 0, sms = 0, per_sm = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, smem_bytes)) != cudaSuccess) return e;
        *max_grid = per_sm >= 1 ? sms : 0;
        return cudaSuccess;
    }
    void *args[] = {(void *)&D, &st_lo, &st_hi, &n_steps, &serial0};
    // cooperative: every CTA must be resident, they wait for one another's data
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kThreads), args, (size_t)smem_bytes, st);
}

// picks the instance for the weight type and the number of token rows M
template <int DH>
cudaError_t launch_step_dh(const Dev &D, int dtype, int st_lo, int st_hi, int n_steps, uint32_t serial0, int grid, int smem_bytes,
                           cudaStream_t st, int *max_grid) {
    const int M = D.M;
#define XSM_GO(WT, NTM) return launch_step_instance<WT, NTM, DH>(D, st_lo, st_hi, n_steps, serial0, grid, smem_bytes, st, max_grid)
    if (dtype == 1) {
        if (M <= 8 && D.small) XSM_GO(bf16, 1);
        if (M <= 16) XSM_GO(bf16, 2);
        if (M <= 32) XSM_GO(bf16, 4);
        if (M <= 80) XSM_GO(bf16, 10);
        XSM_GO(bf16, 16);
    }
    if (M <= 8) XSM_GO(float, 8);
    if (M <= 16) XSM_GO(float, 16);
    XSM_GO(float, 24);
#undef XSM_GO
}

}  // namespace xsm
