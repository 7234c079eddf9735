// Decode-step kernels of one partition: weight-streaming linear layers with fused
// norm prologues and bias / activation / rotary / cache-append / residual / argmax
// epilogues, and split-sequence attention over the paged key/value cache.
//
// A launch serves up to MAXB "items".  An item is one new position of one slot:
// in the recurrent schedule the items are the samples of the group that reached
// the partition together (they share one pass over the weights); during the first
// visit of a sample they are consecutive prompt positions of one slot.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mdi {

constexpr int MAXB = 8;          // items per launch
constexpr int LIN_THREADS = 256; // 8 warps, one 2-row unit per warp
constexpr int LIN_WARPS = LIN_THREADS / 32;
constexpr int ATT_THREADS = 128;
constexpr int ATT_WARPS = ATT_THREADS / 32;

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may start
// while its predecessor in the stream is still running; it must not touch the predecessor's results before
// pdl_wait() (which returns once the predecessor has completed and flushed).  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

struct Batch {
    int n;
    int slot[MAXB]; // slot of the item
    int off[MAXB];  // position of the item = pos[slot] + off
    int adv[MAXB];  // added to pos[slot] by the last kernel of a partition step
};

// Paged key/value cache of one partition.  Page layout: [2 (K,V)][n_kv_head][page_tokens][head_dim].
struct KvView {
    void *pool;
    const int *page_table; // [n_slots][n_layers_local][pages_per_seq]
    int n_layers_local, pages_per_seq, page_tokens, page_shift;
    int n_kv_head, head_dim;
    size_t page_elems;
};

enum LinMode { LIN_QKV = 0, LIN_ACT = 1, LIN_GATEUP = 2, LIN_HEAD = 3, LIN_RESID = 4 };
enum NormKind { NORM_NONE = 0, NORM_LAYER = 1, NORM_RMS = 2 };

struct LinArgs {
    const void *W;      // [n_rows][in_dim]; LIN_GATEUP: gate matrix
    const void *W2;     // LIN_GATEUP: up matrix
    const float *bias;  // [n_rows] or null
    int n_rows, in_dim;
    const float *x_in;  // [n][in_dim] input rows (pre-norm activations, or plain input for LIN_RESID)
    int norm;           // NormKind applied to x_in in the prologue
    const float *gamma, *beta;
    float eps;
    int act;            // LIN_ACT: 0 tanh-GELU, 1 erf-GELU
    // LIN_QKV
    float *q_out;       // [n][q_rows]
    int q_rows, kv_rows, rope;      // rope: 1 = rotate q and k (rows paired i, i + head_dim/2)
    const float *rope_cos, *rope_sin; // [n_ctx][head_dim/2]
    KvView kv;
    int layer_local;
    const int *pos;     // [n_slots] rows already cached per slot in this partition
    // LIN_ACT / LIN_GATEUP
    float *h_out;       // [n][n_rows]
    // LIN_RESID
    const float *x_res; // [n][n_rows] residual input
    float *x_out;       // [n][n_rows]
    int *pos_adv;       // non-null: block 0 adds bt.adv[i] to pos_adv[slot_i] at the end
    // LIN_HEAD
    float *logits;      // [n_slots][n_rows] (indexed by slot) or, if logits_by_item, [n][n_rows]
    int logits_by_item;
    float *part_val;    // [MAXB][gridDim.x]
    int *part_idx;
    unsigned *ticket;
    int *tok_out;       // optional [n]: argmax per item
    int *cur_tok;       // optional [n_slots]: token to feed next
    int *tok_log;       // optional [n_slots][log_stride]: argmax history
    int *gen_count;     // optional [n_slots]
    const int *teacher; // optional [n_slots][log_stride]
    const int *n_teacher;
    int log_stride;
    // sampling from the pmf instead of the argmax (temperature > 0): top_k most likely tokens, counter-based uniform
    float temperature;
    int top_k;
    unsigned long long sample_seed;
};

// ---- 16-byte weight vectors ------------------------------------------------------------------
template <typename WT> struct WVec;
template <> struct WVec<float> {
    static constexpr int N = 4;
    float4 v;
    __device__ __forceinline__ void load(const float *p) { v = __ldg(reinterpret_cast<const float4 *>(p)); }
    __device__ __forceinline__ void unpack(float *w) const { w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w; }
};
template <> struct WVec<__nv_bfloat16> {
    static constexpr int N = 8;
    uint4 v;
    __device__ __forceinline__ void load(const __nv_bfloat16 *p) { v = __ldg(reinterpret_cast<const uint4 *>(p)); }
    __device__ __forceinline__ void unpack(float *w) const {
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            w[2 * i] = __uint_as_float(u[i] << 16);
            w[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
        }
    }
};

template <> struct WVec<__half> {     // key/value cache rows only
    static constexpr int N = 8;
    uint4 v;
    __device__ __forceinline__ void load(const __half *p) { v = __ldg(reinterpret_cast<const uint4 *>(p)); }
    __device__ __forceinline__ void unpack(float *w) const {
        const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(h[i]);
            w[2 * i] = f.x;
            w[2 * i + 1] = f.y;
        }
    }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float block_sum(float v, float *red /* [LIN_WARPS] */) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < LIN_WARPS; ++w) t += red[w];
    return t;
}

__device__ __forceinline__ float gelu_tanh_f(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float gelu_erf_f(float x) { return 0.5f * x * (1.f + erff(x * 0.7071067811865475f)); }
__device__ __forceinline__ float silu_f(float x) { return x / (1.f + expf(-x)); }

template <typename KT> __device__ __forceinline__ void kv_store(KT *p, float v);
template <> __device__ __forceinline__ void kv_store<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void kv_store<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ void kv_store<__half>(__half *p, float v) { *p = __float2half_rn(v); }

// Element address of (K or V, kv head, row, e) of a slot's cache in one local layer.
template <typename KT>
__device__ __forceinline__ KT *kv_addr(const KvView &kv, int slot, int layer_local, int which, int head, int row, int e) {
    const int page = kv.page_table[((size_t)slot * kv.n_layers_local + layer_local) * kv.pages_per_seq + (row >> kv.page_shift)];
    return reinterpret_cast<KT *>(kv.pool) + (size_t)page * kv.page_elems +
           ((size_t)(which * kv.n_kv_head + head) * kv.page_tokens + (row & (kv.page_tokens - 1))) * kv.head_dim + e;
}

// ---- embedding --------------------------------------------------------------------------------
// x[i][:] = wte[tok_i][:] (+ wpe[pos_i][:]).  Token of item i: tok_src[tok_index_i] where the index is
// the slot (decode: the slot's pending token) or the item's offset into a prompt (first visit).
template <typename WT>
__global__ void k_embed(const WT *wte, const WT *wpe, int d, int vocab, const int *tok_src, int tok_by_slot,
                        const int *pos, Batch bt, float *x) {
    const int i = blockIdx.y;
    if (i >= bt.n) return;
    const int slot = bt.slot[i];
    int tok = tok_by_slot ? tok_src[slot] : tok_src[bt.off[i]];
    tok = min(max(tok, 0), vocab - 1);
    const int p = pos[slot] + bt.off[i];
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < d; e += gridDim.x * blockDim.x) {
        float v;
        if constexpr (sizeof(WT) == 4) v = wte[(size_t)tok * d + e]; else v = __bfloat162float(wte[(size_t)tok * d + e]);
        if (wpe) {
            if constexpr (sizeof(WT) == 4) v += wpe[(size_t)p * d + e]; else v += __bfloat162float(wpe[(size_t)p * d + e]);
        }
        x[(size_t)i * d + e] = v;
    }
}

// ---- sampling ---------------------------------------------------------------------------------
// Counter-based uniform in [0,1) for (seed, sample, step): two rounds of the splitmix64 output function.
__device__ __forceinline__ unsigned long long sm64(unsigned long long z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__device__ __forceinline__ double sample_uniform(unsigned long long seed, int sample, int step) {
    const unsigned long long h = sm64(sm64(seed ^ ((unsigned long long)(unsigned)sample << 32)) + (unsigned long long)(unsigned)step);
    return (double)(h >> 11) * (1.0 / 9007199254740992.0);
}

// Whole block (LIN_THREADS threads): the top_k (<= 64) largest of lg[0..n) in the order "larger value first,
// lower index first on ties", then one draw from softmax(values / temperature) restricted to them, with the
// cumulative sum taken in that order in fp64.  Returns the chosen index (valid in every thread).
__device__ int block_sample_top_k(const float *lg, int n, int top_k, float temperature, double u, float *sv /*[64]*/, int *si /*[64]*/,
                                  float *wv /*[LIN_WARPS]*/, int *wi /*[LIN_WARPS]*/, int *result) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float pv = INFINITY;
    int pi = -1;
    for (int r = 0; r < top_k; ++r) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int i = tid; i < n; i += LIN_THREADS) {
            const float v = __ldcg(lg + i);
            const bool after_prev = v < pv || (v == pv && i > pi);
            if (after_prev && (v > bv || (v == bv && i < bi))) { bv = v; bi = i; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v = __shfl_xor_sync(0xffffffffu, bv, o);
            const int ix = __shfl_xor_sync(0xffffffffu, bi, o);
            if (v > bv || (v == bv && ix < bi)) { bv = v; bi = ix; }
        }
        if (lane == 0) { wv[warp] = bv; wi[warp] = bi; }
        __syncthreads();
        bv = wv[0];
        bi = wi[0];
#pragma unroll
        for (int w = 1; w < LIN_WARPS; ++w)
            if (wv[w] > bv || (wv[w] == bv && wi[w] < bi)) { bv = wv[w]; bi = wi[w]; }
        if (tid == 0) { sv[r] = bv; si[r] = bi; }
        pv = bv;
        pi = bi;
        __syncthreads();
    }
    if (tid == 0) {
        const int k = top_k < n ? top_k : n;
        double z = 0.0, p[64];
        for (int j = 0; j < k; ++j) { p[j] = exp(((double)sv[j] - (double)sv[0]) / (double)temperature); z += p[j]; }
        const double target = u * z;
        double c = 0.0;
        int pick = si[k - 1];
        for (int j = 0; j < k; ++j) { c += p[j]; if (c > target) { pick = si[j]; break; } }
        *result = pick;
    }
    __syncthreads();
    return *result;
}

// Last stage of the output layers, shared by the kernels that produce logits: every block has left its best
// (value, row) per item in part_val / part_idx; the block that takes the last ticket picks the tokens (greedy: best
// candidate, lowest row on ties; or a draw from the pmf of the top_k logits) and advances the slots' token state.
__device__ __forceinline__ void head_finish(const LinArgs &a, const Batch &bt, bool *is_last, float *smp_v, int *smp_i, float *smp_wv,
                                            int *smp_w, int *smp_res) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __threadfence();
    __syncthreads();
    if (tid == 0) *is_last = atomicAdd(a.ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (*is_last && a.temperature > 0.f && a.gen_count) {
        // draw from the pmf instead of taking the argmax: one item at a time, the whole block on each
        __threadfence();
        for (int i = 0; i < bt.n; ++i) {
            const int slot = bt.slot[i];
            const int g = a.gen_count[slot];
            const float *lg = a.logits + (size_t)(a.logits_by_item ? i : slot) * a.n_rows;
            const int tok = block_sample_top_k(lg, a.n_rows, a.top_k, a.temperature, sample_uniform(a.sample_seed, slot, g), smp_v, smp_i,
                                               smp_wv, smp_w, smp_res);
            __syncthreads();
            if (tid == 0) {
                if (a.tok_out) a.tok_out[i] = tok;
                if (g < a.log_stride) a.tok_log[(size_t)slot * a.log_stride + g] = tok;
                int feed = tok;
                if (a.teacher && g < a.n_teacher[slot]) feed = a.teacher[(size_t)slot * a.log_stride + g];
                a.cur_tok[slot] = feed;
                a.gen_count[slot] = g + 1;
            }
            __syncthreads();
        }
        if (tid == 0) *a.ticket = 0u;
    } else if (*is_last) {
        __threadfence();
        for (int i = warp; i < bt.n; i += LIN_WARPS) {
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            for (int c = lane; c < (int)gridDim.x; c += 32) {
                const float v = __ldcg(a.part_val + (size_t)i * gridDim.x + c);
                const int ix = __ldcg(a.part_idx + (size_t)i * gridDim.x + c);
                if (v > bv || (v == bv && ix < bi)) { bv = v; bi = ix; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float v = __shfl_xor_sync(0xffffffffu, bv, o);
                const int ix = __shfl_xor_sync(0xffffffffu, bi, o);
                if (v > bv || (v == bv && ix < bi)) { bv = v; bi = ix; }
            }
            if (lane == 0) {
                const int slot = bt.slot[i];
                if (a.tok_out) a.tok_out[i] = bi;
                if (a.gen_count) {
                    const int g = a.gen_count[slot];
                    if (g < a.log_stride) a.tok_log[(size_t)slot * a.log_stride + g] = bi;
                    int feed = bi;
                    if (a.teacher && g < a.n_teacher[slot]) feed = a.teacher[(size_t)slot * a.log_stride + g];
                    a.cur_tok[slot] = feed;
                    a.gen_count[slot] = g + 1;
                }
            }
        }
        if (tid == 0) *a.ticket = 0u;
    }
}

// Token choice from finished logits y[item][n_rows] (what a tensor-core contraction left): copies them to the
// context's logits (by slot), finds every block's best row per item over its slice of the rows, then head_finish.
// grid (row slices), LIN_THREADS threads.
__global__ void __launch_bounds__(LIN_THREADS) k_head_pick(const LinArgs a, const Batch bt, const float *y) {
    __shared__ float hv[LIN_WARPS][MAXB];
    __shared__ int hi_[LIN_WARPS][MAXB];
    __shared__ bool is_last;
    __shared__ float smp_v[64];
    __shared__ int smp_i[64], smp_w[LIN_WARPS], smp_res;
    __shared__ float smp_wv[LIN_WARPS];
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = (a.n_rows + gridDim.x - 1) / gridDim.x, r_lo = blockIdx.x * per, r_hi = min(a.n_rows, r_lo + per);
    for (int i = 0; i < bt.n; ++i) {
        float *lg = a.logits + (size_t)(a.logits_by_item ? i : bt.slot[i]) * a.n_rows;
        const float *src = y + (size_t)i * a.n_rows;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int r = r_lo + tid; r < r_hi; r += LIN_THREADS) {
            const float v = __ldcg(src + r);
            lg[r] = v;
            if (v > bv) { bv = v; bi = r; } // rows ascend within a thread: the first maximum is the lowest row
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v = __shfl_xor_sync(0xffffffffu, bv, o);
            const int ix = __shfl_xor_sync(0xffffffffu, bi, o);
            if (v > bv || (v == bv && ix < bi)) { bv = v; bi = ix; }
        }
        if (lane == 0) { hv[warp][i] = bv; hi_[warp][i] = bi; }
    }
    __syncthreads();
    if (tid < bt.n) {
        float bv = hv[0][tid];
        int bi = hi_[0][tid];
#pragma unroll
        for (int w = 1; w < LIN_WARPS; ++w) {
            const float v = hv[w][tid];
            const int i = hi_[w][tid];
            if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
        }
        a.part_val[(size_t)tid * gridDim.x + blockIdx.x] = bv;
        a.part_idx[(size_t)tid * gridDim.x + blockIdx.x] = bi;
    }
    head_finish(a, bt, &is_last, smp_v, smp_i, smp_wv, smp_w, &smp_res);
}

// ---- weight-streaming linear layer ------------------------------------------------------------
// Each warp owns one unit of two weight rows and streams them once with 16-byte loads; the NB
// input vectors sit in shared memory as fp32 (normalised in the prologue where asked).
template <int NB, typename WT, int MODE, typename KT = WT>
__global__ void __launch_bounds__(LIN_THREADS) k_linear(const LinArgs a, const Batch bt) {
    extern __shared__ __align__(16) float xs[]; // [NB][in_dim]
    __shared__ float red[LIN_WARPS];
    __shared__ float hv[LIN_WARPS][NB];
    __shared__ int hi_[LIN_WARPS][NB];
    __shared__ bool is_last;
    __shared__ float smp_v[64];
    __shared__ int smp_i[64], smp_w[LIN_WARPS], smp_res;
    __shared__ float smp_wv[LIN_WARPS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = a.in_dim;

    // ---- prologue: stage (and normalise) the inputs
    for (int b = 0; b < NB; ++b) {
        const bool live = b < bt.n;
        float s = 0.f;
        for (int i = tid; i < K; i += LIN_THREADS) {
            float v = live ? a.x_in[(size_t)b * K + i] : 0.f;
            xs[b * K + i] = v;
            s += v;
        }
        if (a.norm == NORM_NONE) continue;
        float mean = 0.f;
        if (a.norm == NORM_LAYER) mean = block_sum(s, red) / (float)K;
        float ss = 0.f;
        for (int i = tid; i < K; i += LIN_THREADS) { float c = xs[b * K + i] - mean; ss += c * c; }
        const float rstd = rsqrtf(block_sum(ss, red) / (float)K + a.eps);
        for (int i = tid; i < K; i += LIN_THREADS) {
            float v = (xs[b * K + i] - mean) * rstd * a.gamma[i];
            if (a.beta) v += a.beta[i];
            xs[b * K + i] = v;
        }
    }
    __syncthreads();

    // ---- rows of this warp's unit
    const int u = blockIdx.x * LIN_WARPS + warp;
    int r0, r1;
    const WT *w0, *w1;
    bool v0, v1;
    if constexpr (MODE == LIN_GATEUP) {
        r0 = r1 = u;
        v0 = v1 = u < a.n_rows;
        const int rc = v0 ? u : 0;
        w0 = reinterpret_cast<const WT *>(a.W) + (size_t)rc * K;
        w1 = reinterpret_cast<const WT *>(a.W2) + (size_t)rc * K;
    } else {
        if (MODE == LIN_QKV && a.rope) {
            const int half = a.kv.head_dim >> 1;
            r0 = (u / half) * a.kv.head_dim + (u % half);
            r1 = r0 + half;
        } else {
            r0 = 2 * u;
            r1 = 2 * u + 1;
        }
        v0 = r0 < a.n_rows;
        v1 = r1 < a.n_rows;
        w0 = reinterpret_cast<const WT *>(a.W) + (size_t)(v0 ? r0 : 0) * K;
        w1 = reinterpret_cast<const WT *>(a.W) + (size_t)(v1 ? r1 : 0) * K;
    }

    constexpr int VEC = WVec<WT>::N;
    constexpr int U = 4;
    float acc0[NB], acc1[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc0[b] = acc1[b] = 0.f;

    for (int k0 = lane * VEC; k0 < K; k0 += 32 * VEC * U) {
        WVec<WT> a0[U], a1[U];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int k = k0 + j * 32 * VEC;
            if (k < K) { a0[j].load(w0 + k); a1[j].load(w1 + k); }
        }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int k = k0 + j * 32 * VEC;
            if (k < K) {
                float f0[VEC], f1[VEC];
                a0[j].unpack(f0);
                a1[j].unpack(f1);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const float4 *xp = reinterpret_cast<const float4 *>(xs + b * K + k);
#pragma unroll
                    for (int q = 0; q < VEC / 4; ++q) {
                        const float4 x = xp[q];
                        acc0[b] = fmaf(f0[4 * q + 0], x.x, acc0[b]); acc1[b] = fmaf(f1[4 * q + 0], x.x, acc1[b]);
                        acc0[b] = fmaf(f0[4 * q + 1], x.y, acc0[b]); acc1[b] = fmaf(f1[4 * q + 1], x.y, acc1[b]);
                        acc0[b] = fmaf(f0[4 * q + 2], x.z, acc0[b]); acc1[b] = fmaf(f1[4 * q + 2], x.z, acc1[b]);
                        acc0[b] = fmaf(f0[4 * q + 3], x.w, acc0[b]); acc1[b] = fmaf(f1[4 * q + 3], x.w, acc1[b]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) { acc0[b] = warp_sum(acc0[b]); acc1[b] = warp_sum(acc1[b]); }

    // ---- epilogue: lane b finishes item b
    float y0 = 0.f, y1 = 0.f;
#pragma unroll
    for (int b = 0; b < NB; ++b) if (lane == b) { y0 = acc0[b]; y1 = acc1[b]; }
    const int b = lane;
    const bool item = b < bt.n && b < NB;

    if constexpr (MODE == LIN_QKV) {
        if (item && v0) {
            if (a.bias) { y0 += a.bias[r0]; if (v1) y1 += a.bias[r1]; }
            const int slot = bt.slot[b];
            const int p = a.pos[slot] + bt.off[b];
            const int hd = a.kv.head_dim;
            if (a.rope && r0 < a.q_rows + a.kv_rows) {
                const int i = r0 % hd; // < hd/2 by construction
                const float c = a.rope_cos[(size_t)p * (hd >> 1) + i], s = a.rope_sin[(size_t)p * (hd >> 1) + i];
                const float t0 = y0 * c - y1 * s, t1 = y1 * c + y0 * s;
                y0 = t0; y1 = t1;
            }
            const int rr[2] = {r0, r1};
            const float yy[2] = {y0, y1};
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (j == 1 && !v1) break;
                const int r = rr[j];
                if (r < a.q_rows) a.q_out[(size_t)b * a.q_rows + r] = yy[j];
                else {
                    const int rk = r - a.q_rows;
                    const int which = rk >= a.kv_rows;
                    const int rl = rk - which * a.kv_rows;
                    kv_store<KT>(kv_addr<KT>(a.kv, slot, a.layer_local, which, rl / hd, p, rl % hd), yy[j]);
                }
            }
        }
    } else if constexpr (MODE == LIN_ACT) {
        if (item && v0) {
            if (a.bias) { y0 += a.bias[r0]; if (v1) y1 += a.bias[r1]; }
            a.h_out[(size_t)b * a.n_rows + r0] = a.act == 0 ? gelu_tanh_f(y0) : gelu_erf_f(y0);
            if (v1) a.h_out[(size_t)b * a.n_rows + r1] = a.act == 0 ? gelu_tanh_f(y1) : gelu_erf_f(y1);
        }
    } else if constexpr (MODE == LIN_GATEUP) {
        if (item && v0) a.h_out[(size_t)b * a.n_rows + r0] = silu_f(y0) * y1;
    } else if constexpr (MODE == LIN_RESID) {
        if (item && v0) {
            if (a.bias) { y0 += a.bias[r0]; if (v1) y1 += a.bias[r1]; }
            a.x_out[(size_t)b * a.n_rows + r0] = a.x_res[(size_t)b * a.n_rows + r0] + y0;
            if (v1) a.x_out[(size_t)b * a.n_rows + r1] = a.x_res[(size_t)b * a.n_rows + r1] + y1;
        }
        if (a.pos_adv && blockIdx.x == 0 && tid < bt.n && bt.adv[tid]) a.pos_adv[bt.slot[tid]] += bt.adv[tid];
    } else { // LIN_HEAD
        if (lane < NB) {
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            if (item && v0) {
                float *lg = a.logits + (size_t)(a.logits_by_item ? b : bt.slot[b]) * a.n_rows;
                lg[r0] = y0;
                bv = y0; bi = r0;
                if (v1) { lg[r1] = y1; if (y1 > bv) { bv = y1; bi = r1; } }
            }
            hv[warp][lane] = bv;
            hi_[warp][lane] = bi;
        }
        __syncthreads();
        if (tid < NB) {
            float bv = hv[0][tid];
            int bi = hi_[0][tid];
#pragma unroll
            for (int w = 1; w < LIN_WARPS; ++w) {
                const float v = hv[w][tid];
                const int i = hi_[w][tid];
                if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
            }
            a.part_val[(size_t)tid * gridDim.x + blockIdx.x] = bv;
            a.part_idx[(size_t)tid * gridDim.x + blockIdx.x] = bi;
        }
        head_finish(a, bt, &is_last, smp_v, smp_i, smp_wv, smp_w, &smp_res);
    }
}

// ---- decode attention over the paged cache --------------------------------------------------------
struct AttnArgs {
    const float *q;   // [n][n_head*head_dim]
    float *o;         // [n][n_head*head_dim]
    float *part;      // [MAXB][n_head][n_split][head_dim + 2]
    unsigned *ticket; // [MAXB][n_head]
    KvView kv;
    int layer_local, n_head, n_split;
    const int *pos;
    float scale;
    __nv_bfloat16 *o_hi, *o_lo; // optional: the merged output also as two bf16 planes (input of a tensor-core GEMM)
};

// grid (n_head, n_split, n_items).  A block scans its share of the cached rows of one head of one
// item with an online softmax; LPR lanes cooperate on one row with one 16-byte load each, so a warp
// covers 32/LPR rows per step.  The block that finishes last for a (item, head) merges the splits.
template <typename KT, int HD>
__global__ void __launch_bounds__(ATT_THREADS) k_attn_decode(const AttnArgs a, const Batch bt) {
    constexpr int EPL = 16 / sizeof(KT);        // elements per lane
    constexpr int LPR = HD / EPL;               // lanes per row
    constexpr int RPW = 32 / LPR;               // rows per warp per step
    constexpr int NG = ATT_WARPS * RPW;         // row groups per block
    static_assert(LPR <= 32 && LPR >= 1, "head_dim too large for one warp");
    __shared__ float sm_m[NG], sm_l[NG];
    __shared__ float sm_o[NG][HD];
    __shared__ bool is_last;

    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.x, sp = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const int slot = bt.slot[b];
    const int n_keys = a.pos[slot] + bt.off[b] + 1;
    const int per = (n_keys + a.n_split - 1) / a.n_split;
    const int lo = sp * per, hi = min(n_keys, lo + per);
    const int kvh = h / (a.n_head / a.kv.n_kv_head);
    float *part = a.part + (((size_t)b * a.n_head + h) * a.n_split + sp) * (HD + 2);

    if (lo < hi) {
        float q[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) q[e] = a.q[(size_t)b * a.n_head * HD + h * HD + sub * EPL + e] * a.scale;
        float m = -INFINITY, l = 0.f, o[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[e] = 0.f;
        // four rows per lane group in flight: the loads of a round are issued before any of them is used
        constexpr int UR = 4;
        for (int j0 = lo + warp * RPW; j0 < hi; j0 += NG * UR) {
            WVec<KT> kvv[UR], vvv[UR];
#pragma unroll
            for (int u = 0; u < UR; ++u) {
                const int j = j0 + u * NG + grp;
                const int jj = j < hi ? j : lo;
                const KT *kp = kv_addr<KT>(a.kv, slot, a.layer_local, 0, kvh, jj, sub * EPL);
                const KT *vp = kp + (size_t)a.kv.n_kv_head * a.kv.page_tokens * HD;
                kvv[u].load(kp);
                vvv[u].load(vp);
            }
#pragma unroll
            for (int u = 0; u < UR; ++u) {
                const bool live = j0 + u * NG + grp < hi;
                float kf[EPL], vf[EPL];
                kvv[u].unpack(kf);
                vvv[u].unpack(vf);
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) s = fmaf(q[e], kf[e], s);
#pragma unroll
                for (int w = LPR / 2; w > 0; w >>= 1) s += __shfl_xor_sync(0xffffffffu, s, w);
                if (live) {
                    const float mn = fmaxf(m, s);
                    const float corr = expf(m - mn); // m = -inf gives 0
                    const float p = expf(s - mn);
                    l = l * corr + p;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) o[e] = o[e] * corr + p * vf[e];
                    m = mn;
                }
            }
        }
        const int g = warp * RPW + grp;
        if (sub == 0) { sm_m[g] = m; sm_l[g] = l; }
#pragma unroll
        for (int e = 0; e < EPL; ++e) sm_o[g][sub * EPL + e] = o[e];
        __syncthreads();
        if (tid < HD) {
            float M = -INFINITY;
#pragma unroll
            for (int g2 = 0; g2 < NG; ++g2) M = fmaxf(M, sm_m[g2]);
            float L = 0.f, O = 0.f;
#pragma unroll
            for (int g2 = 0; g2 < NG; ++g2) {
                const float w = sm_m[g2] == -INFINITY ? 0.f : expf(sm_m[g2] - M);
                L += sm_l[g2] * w;
                O += sm_o[g2][tid] * w;
            }
            part[2 + tid] = O;
            if (tid == 0) { part[0] = M; part[1] = L; }
        }
    } else if (tid < HD) {
        part[2 + tid] = 0.f;
        if (tid == 0) { part[0] = -INFINITY; part[1] = 0.f; }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(a.ticket + b * a.n_head + h, 1u) == (unsigned)a.n_split - 1;
    __syncthreads();
    if (is_last) {
        __threadfence();
        const float *pb = a.part + ((size_t)b * a.n_head + h) * a.n_split * (HD + 2);
        if (tid < HD) {
            float M = -INFINITY;
            for (int s2 = 0; s2 < a.n_split; ++s2) M = fmaxf(M, __ldcg(pb + (size_t)s2 * (HD + 2)));
            float L = 0.f, O = 0.f;
            for (int s2 = 0; s2 < a.n_split; ++s2) {
                const float ms = __ldcg(pb + (size_t)s2 * (HD + 2));
                const float w = ms == -INFINITY ? 0.f : expf(ms - M);
                L += __ldcg(pb + (size_t)s2 * (HD + 2) + 1) * w;
                O += __ldcg(pb + (size_t)s2 * (HD + 2) + 2 + tid) * w;
            }
            const float ov = O / L;
            a.o[(size_t)b * a.n_head * HD + h * HD + tid] = ov;
            if (a.o_hi) {
                const __nv_bfloat16 hv = __float2bfloat16_rn(ov);
                a.o_hi[(size_t)b * a.n_head * HD + h * HD + tid] = hv;
                a.o_lo[(size_t)b * a.n_head * HD + h * HD + tid] = __float2bfloat16_rn(ov - __bfloat162float(hv));
            }
        }
        if (tid == 0) a.ticket[b * a.n_head + h] = 0u;
    }
}

} // namespace mdi
