// Persistent tensor-core decode kernel: the whole recurrent pipeline of one generate call (paper, Section III-C,
// Algorithms 1 and 2) in ONE cooperative launch, for models whose blocks are large (bf16 weights, groups of up to
// eight samples per message).
//
// As in k_persistent_decode the grid (one thread block per SM) is split into K teams, one per partition ("node"),
// which hand activations to one another through ring slots and release/acquire flags.  What differs is how a team
// multiplies:  every linear layer is a dense contraction  D[128 rows][16] += W[128 rows][64] * B[16][64]^T  issued
// by one thread with tcgen05.mma, the weight tile arriving by TMA (128-byte swizzle, no multicast) in a ring of
// 16 KB stages that a producer warp fills ahead of the consumers across phases, barriers and ticks, and the
// accumulator living in tensor memory.  The B operand holds the group's activations as bf16 pairs: rows 0..7 the
// high halves of the up to eight samples, rows 8..15 the low halves (x = hi + lo to about 16 mantissa bits), so one
// instruction serves both and the two column halves of D are added when the accumulator is read back.
//
// Work of a linear layer is cut into units (matrix, 128-row tile, range of k-blocks) dealt out evenly over the
// team's blocks.  A unit leaves a raw partial sum in global memory and takes a ticket of its row tile; the unit that
// arrives last adds the tile's partial sums in a fixed order (so results do not depend on timing), adds bias and
// residual, and writes the finished rows: the residual stream, the q/k/v rows, the pre-activations, the logits.
// Everything else that is not a contraction happens in the next phase's prologue, which reads finished values
// only: it normalises, applies GELU / SwiGLU, splits into bf16 pairs and writes its own range of the B operand
// straight into shared memory in the swizzled layout the tensor core reads.  A block of the model costs five team
// barriers: q/k/v rows | attention | output projection | MLP up | MLP down.
//
// Attention (rotary embedding of q and k, append of the new cache row, online softmax over the slot's cached
// rows) runs on the CUDA cores: (sample, head, sequence split) units dealt out over the team's warps, sixteen
// cache rows in flight per warp, page-table entries fetched once per unit; the last split to arrive merges.
//
// Every wait (flag, team barrier, mbarrier) is bounded in wall time as in k_persistent_decode: when a limit is hit
// an error word is set, nobody waits any more, tensor memory is freed and the kernel returns.
#pragma once
#include "persistent_decode.cuh"
#include "tc_gemm.cuh"

namespace mdi {

constexpr int TD_THREADS = 256;                 // warp 0: weight producer; warp 1: MMA issuer; warps 4..7 read accumulators
constexpr int TD_CWARPS = 7;                    // warps 1..7 run prologues and attention together (16 warps of 128 registers were
                                                // measured slower: the attention loop then spills its rows in flight)
constexpr int TD_CTHREADS = TD_CWARPS * 32;
constexpr int TD_MAX_STAGES = 9;                // weight ring: up to 9 stages of 16 KB
constexpr int TD_W_BYTES = 16384;               // one stage: 128 rows x 64 columns of bf16
constexpr int TD_MAXB = 8;                      // samples per group
constexpr int TD_OPERAND_BYTES = 11 * TD_W_BYTES; // shared memory for the ring and the B operand together: the B operand
                                                // holds b_kb k-blocks (64 columns, 16 rows x 128 bytes each), the ring the rest
__host__ __device__ inline int td_stages(int b_kb) { const int n = (TD_OPERAND_BYTES - b_kb * 2048) / TD_W_BYTES; return n < TD_MAX_STAGES ? n : TD_MAX_STAGES; }
constexpr int TD_ACC = 4;                       // accumulators in tensor memory (16 columns each)
constexpr int TD_MAX_PHASES = 64;
constexpr int TD_MAX_SPLITS = 16;               // attention splits over the sequence

enum TdKind { TD_QKV = 0, TD_ATTN = 1, TD_OUT = 2, TD_UP = 3, TD_DOWN = 4, TD_HEAD = 5 };
enum TdPro { TDP_NORM = 0, TDP_COPY = 1, TDP_ACT = 2 };

struct TdPhase {
    int kind, layer_local;
    // contraction: n_mat matrices [n_rows][K] (2: gate and up), n_tiles row tiles, n_split ranges of kb_per_split k-blocks
    int n_mat, n_rows, K, n_tiles, n_kb, n_split, kb_per_split, n_units;
    const CUtensorMap *wmap[2];
    float *part;             // raw partial sums [n_mat][n_split][TD_MAXB][n_rows] (unused when n_split == 1)
    int *ticket;             // [n_mat * n_tiles] arrivals per (matrix, row tile), zero between uses (unused when n_split == 1)
    // what the unit that completes a row tile does: fin[mat][i][row] = sum + fin_bias[row] + resid[i][row]
    const float *fin_bias;   // [n_rows] or null
    const float *fin_resid;  // [TD_MAXB][n_rows] or null
    int fin_resid_ring;      // 1: the residual is the previous partition's ring slot (first block of a step)
    float *fin;              // [n_mat][TD_MAXB][n_rows] (output layer: the context's logits, by slot)
    int fin_ring;            // 1: the result goes to this partition's ring slot (last block of a step)
    // prologue: what the B operand is made of
    int pro;                 // TdPro
    int first_of_step;       // NORM: the input is the previous partition's ring slot, or the token embedding
    const float *src;        // NORM: residual stream [TD_MAXB][d]; COPY: [TD_MAXB][K]; ACT: [n_mat][TD_MAXB][K]; attention: q/k/v rows
    float *dst;              // NORM of the very first block: where the embedded tokens are kept [TD_MAXB][d]
    const float *gamma, *beta;
};

struct TdTeam {
    int first_cta, n_cta, phase_begin, n_phases, is_first, is_last, n_att_split;
    KvView kv;
    const float *ring_in;
    float *ring_out;
    float *att_part;         // [TD_MAXB][n_head][n_att_split][head_dim + 4]: max, sum, -, -, o[head_dim]
    float *att_out;          // [TD_MAXB][n_head * head_dim]
    int *att_ticket;         // [TD_MAXB][n_head]
    float *head_pv;          // last partition: argmax candidates [TD_MAXB][4 * row tiles of the vocabulary]
    int *head_pi;
    int *pos;
    unsigned *bar, *flag_out;
    const unsigned *flag_in;
};

struct TdParams {
    int d, n_head, n_kv_head, head_dim, d_ff, vocab, norm, act, rope, K, G, n_samples, gmax, n_pass;
    int b_kb;                // k-blocks of the resident B operand (ranges of the contractions never exceed it)
    float eps, scale;
    const TdTeam *teams;
    const TdPhase *phases;
    const void *wte, *wpe;
    const float *rope_cos, *rope_sin;
    float *logits;
    int *cur_tok, *tok_log, *gen_count;
    const int *teacher, *n_teacher;
    int log_stride;
    int *err;
    unsigned long long wait_ns;
    int withhold_partition;
    unsigned long long *prof; // optional [grid][PK_PROF_N]: [0] input edge, [1] prologues, [2] contraction, [3] team barriers,
                              // [4] attention, [5] token choice, [6] producer waiting for a free stage, [7] producer total,
                              // [8] team barrier after the output layer, [9] the output layer's contraction, and inside [2] / [9]:
                              // [10] the MMA thread waiting for weight tiles, [11] waiting for a free accumulator
};

struct TdSmem {
    size_t ring, stats, red, s_flag, s_dead, bars, tmem_slot, s_ph, total;
};
__host__ __device__ inline TdSmem td_smem_layout() {
    TdSmem L;
    size_t o = 0;
    auto take = [&](size_t bytes, size_t align) { o = (o + align - 1) / align * align; const size_t r = o; o += bytes; return r; };
    L.ring = take((size_t)TD_OPERAND_BYTES, 1024); // the B operand sits behind the ring's stages
    L.stats = take(4 * 2 * TD_MAXB, 16);
    L.red = take(4 * 2 * TD_MAXB * TD_CWARPS, 16);
    L.s_flag = take(8, 8);
    L.s_dead = take(8, 8);
    L.bars = take(8 * (2 * TD_MAX_STAGES + 2 * TD_ACC + 1), 8);
    L.tmem_slot = take(8, 8);
    L.s_ph = take(sizeof(TdPhase) * TD_MAX_PHASES, 16);
    L.total = o + 1024; // slack to align the base to 1024 bytes
    return L;
}

__host__ __device__ inline bool td_is_gemm(int kind) { return kind == TD_QKV || kind == TD_OUT || kind == TD_UP || kind == TD_DOWN || kind == TD_HEAD; }
__device__ __forceinline__ void td_bar() { asm volatile("bar.sync 1, %0;" ::"n"(TD_CTHREADS) : "memory"); }

// unit u of a phase -> (k range, matrix, row tile); units are ordered k-range-major so that a block's units share B
struct TdUnit { int ks, mat, tile, kb_lo, kb_hi; };
__device__ __forceinline__ TdUnit td_unit(const TdPhase &ph, int u) {
    TdUnit t;
    const int per = ph.n_mat * ph.n_tiles;
    t.ks = u / per;
    const int r = u - t.ks * per;
    t.mat = r / ph.n_tiles;
    t.tile = r - t.mat * ph.n_tiles;
    t.kb_lo = t.ks * ph.kb_per_split;
    t.kb_hi = min(ph.n_kb, t.kb_lo + ph.kb_per_split);
    return t;
}

// byte offset of element (row r of 16, column c) inside a B operand whose first column is c_lo (a multiple of 64):
// per k-block 16 rows of 128 bytes, 8-row groups 1024 bytes apart, 16-byte chunks XOR-swizzled with the row
__device__ __forceinline__ uint32_t td_b_off(int r, int c_rel) {
    const int kb = c_rel >> 6, cc = c_rel & 63;
    return (uint32_t)(kb * 2048 + (r >> 3) * 1024 + (r & 7) * 128 + ((((cc >> 3) ^ (r & 7)) & 7) << 4) + (cc & 7) * 2);
}
// four consecutive values (columns c_rel .. c_rel+3, c_rel a multiple of 4) of sample i: high halves to row i, low to row i+8
__device__ __forceinline__ void td_b_store4(unsigned char *B, int i, int c_rel, const float4 v) {
    const float f[4] = {v.x, v.y, v.z, v.w};
    uint16_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat16 h = __float2bfloat16_rn(f[e]);
        hi[e] = __bfloat16_as_ushort(h);
        lo[e] = __bfloat16_as_ushort(__float2bfloat16_rn(f[e] - __bfloat162float(h)));
    }
    *reinterpret_cast<uint2 *>(B + td_b_off(i, c_rel)) = make_uint2((uint32_t)hi[0] | ((uint32_t)hi[1] << 16), (uint32_t)hi[2] | ((uint32_t)hi[3] << 16));
    *reinterpret_cast<uint2 *>(B + td_b_off(i + 8, c_rel)) = make_uint2((uint32_t)lo[0] | ((uint32_t)lo[1] << 16), (uint32_t)lo[2] | ((uint32_t)lo[3] << 16));
}

// Take a ticket: the increment releases what this warp wrote before it (the lanes meet in __syncwarp first) and acquires
// what earlier ticket holders wrote, so whoever draws the last ticket may read every partial result.
__device__ __forceinline__ int td_ticket(int *p) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(p) : "memory");
    return old;
}

__device__ __forceinline__ float4 td_add4(float4 a, const float4 b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; return a; }
__device__ __forceinline__ float4 td_ldcg4(const float *p) { return __ldcg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ float4 td_bf16x4(const __nv_bfloat16 *p) {
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(p));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
}

// ---- attention of one (sample, head, sequence split) by one warp ------------------------------------------------
// q, and the new row's k and v, are finished rows of the q/k/v contraction (bias included); rotary embedding is
// applied here; the warp whose split ends at the new row uses it from registers, and for the first query head of a
// key/value head also appends it to the cache.  Leaves (max, sum, o[head_dim]) of the split in att_part; the split
// that arrives last merges all of them (in split order) into att_out.
template <typename KT, int HD>
__device__ __forceinline__ void td_attn_unit(const TdParams &P, const TdTeam &T, const TdPhase &ph, int i, int slot, int pos, int h, int sp,
                                             int lane) {
    constexpr int EPL = 16 / (int)sizeof(KT), LPR = HD / EPL, RPW = 32 / LPR, U = 16 / RPW; // 16 cache rows in flight per warp
    static_assert(LPR >= 2 && LPR <= 32, "head_dim");
    const int sub = lane % LPR, grp = lane / LPR;
    const int qw = P.n_head * HD, kw = P.n_kv_head * HD, rows_all = qw + 2 * kw;
    const int kvh = h / (P.n_head / P.n_kv_head);
    const int nsp = T.n_att_split;
    const int n_keys = pos + 1;
    const int per = (n_keys + nsp - 1) / nsp;
    const int lo = sp * per, hi = min(n_keys, lo + per);
    float *part = T.att_part + (((size_t)i * P.n_head + h) * nsp + sp) * (HD + 4);
    float m = -INFINITY, l = 0.f, o[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[e] = 0.f;
    if (lo < hi) {
        const bool has_new = hi == n_keys;
        const float *src = ph.src + (size_t)i * rows_all;
        float q[EPL], kn[EPL], vn[EPL];
        // all three rows are requested before any is used
#pragma unroll
        for (int e4 = 0; e4 < EPL / 4; ++e4) {
            const float4 a = td_ldcg4(src + h * HD + sub * EPL + 4 * e4);
            q[4 * e4] = a.x; q[4 * e4 + 1] = a.y; q[4 * e4 + 2] = a.z; q[4 * e4 + 3] = a.w;
            if (has_new) {
                const float4 b = td_ldcg4(src + qw + kvh * HD + sub * EPL + 4 * e4), c = td_ldcg4(src + qw + kw + kvh * HD + sub * EPL + 4 * e4);
                kn[4 * e4] = b.x; kn[4 * e4 + 1] = b.y; kn[4 * e4 + 2] = b.z; kn[4 * e4 + 3] = b.w;
                vn[4 * e4] = c.x; vn[4 * e4 + 1] = c.y; vn[4 * e4 + 2] = c.z; vn[4 * e4 + 3] = c.w;
            } else {
                kn[4 * e4] = kn[4 * e4 + 1] = kn[4 * e4 + 2] = kn[4 * e4 + 3] = 0.f;
                vn[4 * e4] = vn[4 * e4 + 1] = vn[4 * e4 + 2] = vn[4 * e4 + 3] = 0.f;
            }
        }
        // page-table entries of the split's rows: one per lane, handed out by shuffles (a split spans at most 32 pages,
        // which the host's choice of splits guarantees)
        const int pg_lo = lo >> T.kv.page_shift;
        const int my_pg = min(pg_lo + lane, T.kv.pages_per_seq - 1);
        const int my_entry = T.kv.page_table[((size_t)slot * T.kv.n_layers_local + ph.layer_local) * T.kv.pages_per_seq + my_pg];
        if (P.rope) {
            // split-halves pairing: element e pairs with e + HD/2, which another lane of the row holds
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                const int idx = sub * EPL + e, ir = idx & (HD / 2 - 1);
                const float c = P.rope_cos[(size_t)pos * (HD / 2) + ir], s = P.rope_sin[(size_t)pos * (HD / 2) + ir];
                const float oq = __shfl_xor_sync(0xffffffffu, q[e], LPR / 2), ok = __shfl_xor_sync(0xffffffffu, kn[e], LPR / 2);
                q[e] = idx < HD / 2 ? q[e] * c - oq * s : q[e] * c + oq * s;
                kn[e] = idx < HD / 2 ? kn[e] * c - ok * s : kn[e] * c + ok * s;
            }
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) q[e] *= P.scale;
        auto row_ptr = [&](int row) -> const KT * {
            const int entry = __shfl_sync(0xffffffffu, my_entry, (row >> T.kv.page_shift) - pg_lo);
            return reinterpret_cast<const KT *>(T.kv.pool) + (size_t)entry * T.kv.page_elems +
                   ((size_t)kvh * T.kv.page_tokens + (row & (T.kv.page_tokens - 1))) * HD + sub * EPL;
        };
        if (has_new && h % (P.n_head / P.n_kv_head) == 0) {
            KT *kp = const_cast<KT *>(row_ptr(pos));
            KT *vp = kp + (size_t)T.kv.n_kv_head * T.kv.page_tokens * HD;
            if (grp == 0) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) { kv_store<KT>(kp + e, kn[e]); kv_store<KT>(vp + e, vn[e]); }
            }
        }
        const int hi_old = has_new ? hi - 1 : hi;
        auto fold = [&](float s, const float *vf) {
            const float mn = fmaxf(m, s), corr = expf(m - mn), pr = expf(s - mn);
            l = l * corr + pr;
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[e] = o[e] * corr + pr * vf[e];
            m = mn;
        };
        for (int j0 = lo; j0 < hi_old; j0 += RPW * U) {
            uint4 kk[U], vv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int jr = j0 + u * RPW + grp;
                const KT *kp = row_ptr(jr < hi_old ? jr : lo);
                const KT *vp = kp + (size_t)T.kv.n_kv_head * T.kv.page_tokens * HD;
                kk[u] = __ldcg(reinterpret_cast<const uint4 *>(kp));
                vv[u] = __ldcg(reinterpret_cast<const uint4 *>(vp));
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float kf[EPL], vf[EPL];
                kv_unpack<KT>(kk[u], kf);
                kv_unpack<KT>(vv[u], vf);
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) s = fmaf(q[e], kf[e], s);
#pragma unroll
                for (int w = LPR / 2; w > 0; w >>= 1) s += __shfl_xor_sync(0xffffffffu, s, w);
                if (j0 + u * RPW + grp < hi_old) fold(s, vf);
            }
        }
        if (has_new) {
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) s = fmaf(q[e], kn[e], s);
#pragma unroll
            for (int w = LPR / 2; w > 0; w >>= 1) s += __shfl_xor_sync(0xffffffffu, s, w);
            if (grp == 0) fold(s, vn);
        }
        // merge the row groups of the warp
#pragma unroll
        for (int w = LPR; w < 32; w <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m, w), l2 = __shfl_xor_sync(0xffffffffu, l, w);
            const float mn = fmaxf(m, m2);
            const float c1 = m == -INFINITY ? 0.f : expf(m - mn), c2 = m2 == -INFINITY ? 0.f : expf(m2 - mn);
            l = l * c1 + l2 * c2;
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[e] = o[e] * c1 + __shfl_xor_sync(0xffffffffu, o[e], w) * c2;
            m = mn;
        }
    }
    float *out = T.att_out + (size_t)i * qw + h * HD;
    if (nsp == 1) {
        if (grp == 0) {
            const float inv = 1.f / l;
#pragma unroll
            for (int e = 0; e < EPL; ++e) out[sub * EPL + e] = o[e] * inv;
        }
        return;
    }
    if (grp == 0) {
        if (sub == 0) { part[0] = m; part[1] = l; }
#pragma unroll
        for (int e = 0; e < EPL; ++e) part[4 + sub * EPL + e] = o[e];
    }
    __syncwarp();
    int last = 0;
    if (lane == 0) {
        int *tk = T.att_ticket + i * P.n_head + h;
        last = td_ticket(tk) == nsp - 1;
        if (last) *tk = 0;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) return;
    // every lane reads all split headers, then its four output elements of every split (HD <= 128: lanes 0 .. HD/4-1)
    const float *pb = T.att_part + ((size_t)i * P.n_head + h) * nsp * (HD + 4);
    float ms[TD_MAX_SPLITS], ls[TD_MAX_SPLITS];
    float4 os[TD_MAX_SPLITS];
    const bool act = 4 * lane < HD;
#pragma unroll
    for (int s2 = 0; s2 < TD_MAX_SPLITS; ++s2) {
        if (s2 < nsp) {
            const float2 hdr = __ldcg(reinterpret_cast<const float2 *>(pb + (size_t)s2 * (HD + 4)));
            ms[s2] = hdr.x; ls[s2] = hdr.y;
            os[s2] = act ? td_ldcg4(pb + (size_t)s2 * (HD + 4) + 4 + 4 * lane) : make_float4(0.f, 0.f, 0.f, 0.f);
        } else { ms[s2] = -INFINITY; ls[s2] = 0.f; os[s2] = make_float4(0.f, 0.f, 0.f, 0.f); }
    }
    float M = -INFINITY;
#pragma unroll
    for (int s2 = 0; s2 < TD_MAX_SPLITS; ++s2) M = fmaxf(M, ms[s2]);
    float Ls = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int s2 = 0; s2 < TD_MAX_SPLITS; ++s2) {
        const float w = ms[s2] == -INFINITY ? 0.f : expf(ms[s2] - M);
        Ls += ls[s2] * w;
        acc.x += os[s2].x * w; acc.y += os[s2].y * w; acc.z += os[s2].z * w; acc.w += os[s2].w * w;
    }
    if (act) {
        const float inv = 1.f / Ls;
        *reinterpret_cast<float4 *>(out + 4 * lane) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    }
}

template <typename KT>
__device__ __noinline__ void td_attn_dispatch(const TdParams &P, const TdTeam &T, const TdPhase &ph, int i, int slot, int pos, int h, int sp, int lane) {
    switch (P.head_dim) {
        case 32: td_attn_unit<KT, 32>(P, T, ph, i, slot, pos, h, sp, lane); break;
        case 64: td_attn_unit<KT, 64>(P, T, ph, i, slot, pos, h, sp, lane); break;
        default: td_attn_unit<KT, 128>(P, T, ph, i, slot, pos, h, sp, lane); break;
    }
}

template <typename KT>
__global__ void __launch_bounds__(TD_THREADS, 1) k_tc_decode(const TdParams P) {
    extern __shared__ unsigned char td_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)td_raw + 1023) & ~(uintptr_t)1023);
    const TdSmem L = td_smem_layout();
    unsigned char *ring = smem + L.ring;
    const int TD_STAGES = td_stages(P.b_kb);
    unsigned char *Bsm = ring + (size_t)TD_STAGES * TD_W_BYTES;
    float *stats = reinterpret_cast<float *>(smem + L.stats);   // [TD_MAXB][2]: mean, 1/std
    float *red = reinterpret_cast<float *>(smem + L.red);       // [TD_CWARPS][TD_MAXB][2]
    int *s_dead = reinterpret_cast<int *>(smem + L.s_dead);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L.tmem_slot);
    TdPhase *s_ph = reinterpret_cast<TdPhase *>(smem + L.s_ph);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ct = tid - 32; // index among the 224 threads of warps 1..7
    int p = 0;
    while (p + 1 < P.K && (int)blockIdx.x >= P.teams[p + 1].first_cta) ++p;
    const TdTeam T = P.teams[p];
    const int cta = blockIdx.x - T.first_cta;
    const int K = P.K, G = P.G, d = P.d;
    const uint32_t ring_u32 = smem_u32(ring), b_u32 = smem_u32(Bsm);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + TD_MAX_STAGES), accf0 = smem_u32(bars + 2 * TD_MAX_STAGES),
                   acce0 = smem_u32(bars + 2 * TD_MAX_STAGES + TD_ACC), done_bar = smem_u32(bars + 2 * TD_MAX_STAGES + 2 * TD_ACC);

    if (tid == 0) {
        for (int s = 0; s < TD_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < TD_ACC; ++a) { mbar_init(accf0 + 8 * a, 1); mbar_init(acce0 + 8 * a, 4); }
        mbar_init(done_bar, 1);
        *s_dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < T.n_phases * (int)(sizeof(TdPhase) / 8); i += TD_THREADS)
        reinterpret_cast<unsigned long long *>(s_ph)[i] = reinterpret_cast<const unsigned long long *>(P.phases + T.phase_begin)[i];
    for (int i = tid; i < P.b_kb * 2048 / 16; i += TD_THREADS) reinterpret_cast<uint4 *>(Bsm)[i] = make_uint4(0u, 0u, 0u, 0u);
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(64u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const TdPhase *phases = s_ph;
    const long total_slots = (long)P.n_pass * K;
    bool dead = false;
    const bool prof_on = P.prof != nullptr && lane == 0 && (warp == 0 || warp == 1);
    unsigned long long pf[PK_PROF_N] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}, pf_t = prof_on ? pk_now() : 0;
    auto lap = [&](int cat) { if (prof_on) pk_lap(pf, &pf_t, cat); };

    if (warp == 0) {
        // =========================== weight producer ===========================
        if (lane == 0) {
            // tensor maps live in global memory, written by the host before the launch
            for (int pi = 0; pi < T.n_phases; ++pi)
                for (int mi = 0; mi < 2; ++mi)
                    if (td_is_gemm(phases[pi].kind) && phases[pi].wmap[mi])
                        asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(phases[pi].wmap[mi]) : "memory");
            unsigned issued = 0;
            int stage = 0;
            uint32_t par = 0;
            for (long v = 0; v < total_slots && !dead; ++v) {
                if ((int)(v % K) >= G) continue;
                for (int pi = 0; pi < T.n_phases && !dead; ++pi) {
                    const TdPhase &ph = phases[pi];
                    if (!td_is_gemm(ph.kind)) continue;
                    const int u0 = (int)((long)cta * ph.n_units / T.n_cta), u1 = (int)((long)(cta + 1) * ph.n_units / T.n_cta);
                    for (int u = u0; u < u1 && !dead; ++u) {
                        const TdUnit un = td_unit(ph, u);
                        for (int kb = un.kb_lo; kb < un.kb_hi; ++kb) {
                            lap(7);
                            if (issued >= (unsigned)TD_STAGES) wait_mbar(empty0 + 8 * stage, par ^ 1u, P.err, PKE_EMPTY, dead, P.wait_ns);
                            lap(6);
                            if (dead) break;
                            mbar_expect_tx(full0 + 8 * stage, TD_W_BYTES);
                            tg_tma_2d(ring_u32 + stage * TD_W_BYTES, ph.wmap[un.mat], kb * TG_BK, un.tile * TG_BM, full0 + 8 * stage);
                            ++issued;
                            if (++stage == TD_STAGES) { stage = 0; par ^= 1u; }
                        }
                    }
                }
            }
            if (dead) {
                // copies already issued target this block's shared memory: give them bounded time to land
                const unsigned long long t0 = pk_now();
                for (unsigned q = issued > (unsigned)TD_STAGES ? issued - TD_STAGES : 0; q < issued; ++q)
                    while (!mbar_try_wait(full0 + 8 * (int)(q % TD_STAGES), (uint32_t)((q / TD_STAGES) & 1)) && pk_now() - t0 < 100000000ull) {}
            }
            if (prof_on) {
                lap(7);
                P.prof[(size_t)blockIdx.x * PK_PROF_N + 6] = pf[6];
                P.prof[(size_t)blockIdx.x * PK_PROF_N + 7] = pf[7] + pf[6];
            }
        }
        __syncwarp();
    } else {
        // =========================== warps 1..7 ===========================
        unsigned bar_epoch = 0;
        auto team_barrier = [&]() {
            td_bar();
            if (ct == 0) {
                ++bar_epoch;
                if (T.n_cta > 1) {
                    red_release_add(T.bar, 1u);
                    wait_ge(T.bar, bar_epoch * (unsigned)T.n_cta, P.err, PKE_BARRIER, dead, P.wait_ns);
                }
                if (dead) *s_dead = 1;
            }
            td_bar();
            if (*(volatile int *)s_dead) dead = true;
        };
        // ring cursor (kept by the MMA thread) and accumulator count (the same in every thread)
        int stage = 0;
        uint32_t spar = 0;
        unsigned acc_cnt = 0;

        for (long v = 0; v < total_slots; ++v) {
            const int j = (int)(v % K);
            if (j >= G) continue;
            const unsigned r = (unsigned)(v / K);
            int nb = 0, slots[TD_MAXB], pos[TD_MAXB];
#pragma unroll
            for (int i = 0; i < TD_MAXB; ++i) {
                const int s = j + i * G;
                slots[i] = s < P.n_samples ? s : j;
                if (s < P.n_samples) nb = i + 1;
            }
            // ---- input edge
            if (ct == 0) {
                if (!T.is_first) wait_ge(T.flag_in + j, r + 1, P.err, PKE_FLAG, dead, P.wait_ns);
                else if (r > 0) wait_ge(T.flag_in + j, r, P.err, PKE_FLAG, dead, P.wait_ns);
                if (dead) *s_dead = 1;
            }
            td_bar();
            if (*(volatile int *)s_dead) dead = true;
            lap(0);
#pragma unroll
            for (int i = 0; i < TD_MAXB; ++i) pos[i] = __ldcg(T.pos + slots[i]) + (int)r;
            const float *ring_in = T.is_first ? nullptr : T.ring_in + (size_t)j * P.gmax * d;
            float *ring_out = T.is_last ? nullptr : T.ring_out + (size_t)j * P.gmax * d;

            // residual stream entering a normalising phase at (sample i, columns 4*c4..)
            auto x_in4 = [&](const TdPhase &ph, int i, int c4) -> float4 {
                if (!ph.first_of_step) return td_ldcg4(ph.src + (size_t)i * d + 4 * c4);
                if (!T.is_first) return td_ldcg4(ring_in + (size_t)i * d + 4 * c4);
                const int tok = min(max(__ldcg(P.cur_tok + slots[i]), 0), P.vocab - 1);
                float4 x = td_bf16x4(reinterpret_cast<const __nv_bfloat16 *>(P.wte) + (size_t)tok * d + 4 * c4);
                if (P.wpe) x = td_add4(x, td_bf16x4(reinterpret_cast<const __nv_bfloat16 *>(P.wpe) + (size_t)pos[i] * d + 4 * c4));
                return x;
            };

            for (int pi = 0; pi < T.n_phases; ++pi) {
                const TdPhase &ph = phases[pi];
                if (ph.kind == TD_ATTN) {
                    // ---------------- attention: (sample, head, split) units over the team's warps
                    const int nsp = T.n_att_split, n_units = nb * P.n_head * nsp;
                    for (int u = cta * TD_CWARPS + (warp - 1); u < n_units; u += T.n_cta * TD_CWARPS) {
                        const int sp = u % nsp, h = (u / nsp) % P.n_head, i = u / (nsp * P.n_head);
                        int slot = slots[0], ps = pos[0];
#pragma unroll
                        for (int q = 1; q < TD_MAXB; ++q) if (i == q) { slot = slots[q]; ps = pos[q]; }
                        td_attn_dispatch<KT>(P, T, ph, i, slot, ps, h, sp, lane);
                    }
                    lap(4);
                    team_barrier();
                    lap(3);
                    continue;
                }
                // ---------------- contraction phase
                const int u0 = (int)((long)cta * ph.n_units / T.n_cta), u1 = (int)((long)(cta + 1) * ph.n_units / T.n_cta);
                const bool keep_embedding = ph.pro == TDP_NORM && ph.first_of_step && T.is_first; // the first block's residual input
                if (ph.pro == TDP_NORM && (u0 < u1 || keep_embedding)) {
                    // moments of every sample's row (blocks with units); a copy of the embedded tokens, every block its columns
                    float s1[TD_MAXB], s2[TD_MAXB];
#pragma unroll
                    for (int i = 0; i < TD_MAXB; ++i) s1[i] = s2[i] = 0.f;
                    const int n4 = d >> 2, w_lo = (int)((long)cta * n4 / T.n_cta), w_hi = (int)((long)(cta + 1) * n4 / T.n_cta);
                    const int c_beg = u0 < u1 ? 0 : w_lo, c_end = u0 < u1 ? n4 : w_hi;
                    for (int c4 = c_beg + ct; c4 < c_end; c4 += 2 * TD_CTHREADS) {
                        float4 xa[TD_MAXB], xb[TD_MAXB];
                        const bool two = c4 + TD_CTHREADS < c_end;
#pragma unroll
                        for (int i = 0; i < TD_MAXB; ++i) {
                            xa[i] = i < nb ? x_in4(ph, i, c4) : make_float4(0.f, 0.f, 0.f, 0.f);
                            xb[i] = (i < nb && two) ? x_in4(ph, i, c4 + TD_CTHREADS) : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int i = 0; i < TD_MAXB; ++i) {
                            if (i < nb) {
                                if (keep_embedding && c4 >= w_lo && c4 < w_hi) *reinterpret_cast<float4 *>(ph.dst + (size_t)i * d + 4 * c4) = xa[i];
                                if (keep_embedding && two && c4 + TD_CTHREADS >= w_lo && c4 + TD_CTHREADS < w_hi)
                                    *reinterpret_cast<float4 *>(ph.dst + (size_t)i * d + 4 * (c4 + TD_CTHREADS)) = xb[i];
                                s1[i] += ((xa[i].x + xa[i].y) + (xa[i].z + xa[i].w)) + ((xb[i].x + xb[i].y) + (xb[i].z + xb[i].w));
                                s2[i] += ((xa[i].x * xa[i].x + xa[i].y * xa[i].y) + (xa[i].z * xa[i].z + xa[i].w * xa[i].w)) +
                                         ((xb[i].x * xb[i].x + xb[i].y * xb[i].y) + (xb[i].z * xb[i].z + xb[i].w * xb[i].w));
                            }
                        }
                    }
                    if (u0 < u1) {
#pragma unroll
                        for (int i = 0; i < TD_MAXB; ++i) {
                            s1[i] = warp_sum(s1[i]);
                            s2[i] = warp_sum(s2[i]);
                            if (lane == 0) { red[((warp - 1) * TD_MAXB + i) * 2] = s1[i]; red[((warp - 1) * TD_MAXB + i) * 2 + 1] = s2[i]; }
                        }
                        td_bar();
                        if (ct < TD_MAXB) {
                            float a = 0.f, b = 0.f;
                            for (int w = 0; w < TD_CWARPS; ++w) { a += red[(w * TD_MAXB + ct) * 2]; b += red[(w * TD_MAXB + ct) * 2 + 1]; }
                            const float mean = P.norm == NORM_LAYER ? a / (float)d : 0.f;
                            stats[2 * ct] = mean;
                            stats[2 * ct + 1] = rsqrtf(fmaxf(b / (float)d - mean * mean, 0.f) + P.eps);
                        }
                        td_bar();
                    }
                }
                for (int ub = u0; ub < u1;) {
                    const TdUnit first = td_unit(ph, ub);
                    int ue = ub + 1; // units [ub, ue) share the k range
                    while (ue < u1 && td_unit(ph, ue).ks == first.ks) ++ue;
                    const int c_lo = first.kb_lo * TG_BK, c_hi = min(ph.K, first.kb_hi * TG_BK);
                    // ---- prologue: this block's range of the B operand, eight independent loads in flight per thread
                    {
                        const int n4r = (c_hi - c_lo) >> 2, tot = n4r * nb;
                        constexpr int PB = 8;
                        const bool swiglu = ph.pro == TDP_ACT && ph.n_mat == 1 && P.act == 2;
                        const float *src2 = ph.src + (size_t)TD_MAXB * ph.K; // ACT with SwiGLU: the "up" rows follow the "gate" rows
                        for (int e0 = ct; e0 < tot; e0 += PB * TD_CTHREADS) {
                            float4 xv[PB], yv[PB];
                            int ii[PB], cc[PB];
#pragma unroll
                            for (int u = 0; u < PB; ++u) {
                                const int e = e0 + u * TD_CTHREADS;
                                ii[u] = e / n4r;
                                cc[u] = (c_lo >> 2) + (e - ii[u] * n4r);
                                if (e < tot) {
                                    if (ph.pro == TDP_NORM) {
                                        xv[u] = x_in4(ph, ii[u], cc[u]);
                                        yv[u] = *reinterpret_cast<const float4 *>(ph.gamma + 4 * cc[u]);
                                    } else {
                                        xv[u] = td_ldcg4(ph.src + (size_t)ii[u] * ph.K + 4 * cc[u]);
                                        if (swiglu) yv[u] = td_ldcg4(src2 + (size_t)ii[u] * ph.K + 4 * cc[u]);
                                    }
                                }
                            }
#pragma unroll
                            for (int u = 0; u < PB; ++u) {
                                const int e = e0 + u * TD_CTHREADS;
                                if (e >= tot) break;
                                float4 x = xv[u];
                                if (ph.pro == TDP_NORM) {
                                    const float mean = stats[2 * ii[u]], rstd = stats[2 * ii[u] + 1];
                                    x.x = (x.x - mean) * rstd * yv[u].x; x.y = (x.y - mean) * rstd * yv[u].y;
                                    x.z = (x.z - mean) * rstd * yv[u].z; x.w = (x.w - mean) * rstd * yv[u].w;
                                    if (ph.beta) x = td_add4(x, *reinterpret_cast<const float4 *>(ph.beta + 4 * cc[u]));
                                } else if (ph.pro == TDP_ACT) {
                                    if (swiglu) x = make_float4(pk_silu(x.x) * yv[u].x, pk_silu(x.y) * yv[u].y, pk_silu(x.z) * yv[u].z, pk_silu(x.w) * yv[u].w);
                                    else x = make_float4(pk_act(x.x, P.act), pk_act(x.y, P.act), pk_act(x.z, P.act), pk_act(x.w, P.act));
                                }
                                td_b_store4(Bsm, ii[u], 4 * cc[u] - c_lo, x);
                            }
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    td_bar();
                    lap(1);
                    // ---- the units: one thread issues the MMAs, four warps read accumulators back
                    const unsigned acc_base = acc_cnt;
                    if (warp == 1 && lane == 0) {
                        const uint32_t idesc = tg_idesc(TG_BM, 16);
                        for (int u = ub; u < ue; ++u) {
                            const unsigned ac = acc_base + (unsigned)(u - ub);
                            const int a = (int)(ac % TD_ACC);
                            lap(2);
                            if (ac >= (unsigned)TD_ACC) wait_mbar(acce0 + 8 * a, ((ac / TD_ACC) - 1u) & 1u, P.err, PKE_EMPTY, dead, P.wait_ns);
                            lap(11);
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                            const uint32_t dcol = tmem_base + (uint32_t)(a * 16);
                            for (int kb = first.kb_lo; kb < first.kb_hi; ++kb) {
                                wait_mbar(full0 + 8 * stage, spar, P.err, PKE_FULL, dead, P.wait_ns);
                                lap(10);
                                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                                const uint32_t wbase = ring_u32 + stage * TD_W_BYTES, bbase = b_u32 + (uint32_t)(kb - first.kb_lo) * 2048u;
#pragma unroll
                                for (int k = 0; k < TG_BK / 16; ++k)
                                    tg_mma(dcol, tg_desc(wbase + k * 32), tg_desc(bbase + k * 32), idesc, (kb > first.kb_lo || k > 0) ? 1u : 0u);
                                tg_commit(empty0 + 8 * stage);
                                if (++stage == TD_STAGES) { stage = 0; spar ^= 1u; }
                            }
                            tg_commit(accf0 + 8 * a);
                        }
                        if (dead) *s_dead = 1;
                    } else if (warp >= 4 && warp < 8) {
                        const int lane_base = (warp & 3) * 32;
                        for (int u = ub; u < ue; ++u) {
                            const TdUnit un = td_unit(ph, u);
                            const unsigned ac = acc_base + (unsigned)(u - ub);
                            const int a = (int)(ac % TD_ACC);
                            wait_mbar(accf0 + 8 * a, (ac / TD_ACC) & 1u, P.err, PKE_FULL, dead, P.wait_ns);
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                            uint32_t rr[16];
                            const uint32_t taddr = tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(a * 16);
                            asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                                         : "=r"(rr[0]), "=r"(rr[1]), "=r"(rr[2]), "=r"(rr[3]), "=r"(rr[4]), "=r"(rr[5]), "=r"(rr[6]), "=r"(rr[7]),
                                           "=r"(rr[8]), "=r"(rr[9]), "=r"(rr[10]), "=r"(rr[11]), "=r"(rr[12]), "=r"(rr[13]), "=r"(rr[14]), "=r"(rr[15])
                                         : "r"(taddr) : "memory");
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                            __syncwarp();
                            if (lane == 0) mbar_arrive(acce0 + 8 * a, 1u);
                            const int row = un.tile * TG_BM + lane_base + lane;
                            const bool rv = row < ph.n_rows;
                            float val[TD_MAXB];
#pragma unroll
                            for (int i = 0; i < TD_MAXB; ++i) val[i] = __uint_as_float(rr[i]) + __uint_as_float(rr[i + 8]);
                            bool finish = true;
                            if (ph.n_split > 1) {
                                // leave the partial sum, take a ticket of the row tile; whoever takes the last one adds them all up
                                float *pp = ph.part + ((size_t)(un.mat * ph.n_split + un.ks) * TD_MAXB) * ph.n_rows + row;
                                if (rv) {
#pragma unroll
                                    for (int i = 0; i < TD_MAXB; ++i)
                                        if (i < nb) pp[(size_t)i * ph.n_rows] = val[i];
                                }
                                // (a ticket per warp: its 32 rows of the tile; no block-wide step in between)
                                __syncwarp();
                                int lastone = 0;
                                if (lane == 0) {
                                    int *tk = ph.ticket + (un.mat * ph.n_tiles + un.tile) * 4 + (warp & 3);
                                    lastone = td_ticket(tk) == ph.n_split - 1;
                                    if (lastone) *tk = 0;
                                }
                                finish = __shfl_sync(0xffffffffu, lastone, 0) != 0;
                                if (finish && rv) {
                                    const float *p0 = ph.part + ((size_t)(un.mat * ph.n_split) * TD_MAXB) * ph.n_rows + row;
#pragma unroll
                                    for (int i = 0; i < TD_MAXB; ++i) val[i] = 0.f;
                                    for (int ks0 = 0; ks0 < ph.n_split; ks0 += 4) {
                                        float t[4][TD_MAXB];
#pragma unroll
                                        for (int q = 0; q < 4; ++q)
#pragma unroll
                                            for (int i = 0; i < TD_MAXB; ++i)
                                                t[q][i] = (ks0 + q < ph.n_split && i < nb) ? __ldcg(p0 + ((size_t)(ks0 + q) * TD_MAXB + i) * ph.n_rows) : 0.f;
#pragma unroll
                                        for (int q = 0; q < 4; ++q)
#pragma unroll
                                            for (int i = 0; i < TD_MAXB; ++i) val[i] += t[q][i];
                                    }
                                }
                            }
                            if (finish && ph.kind != TD_HEAD) {
                                if (rv && !dead) {
                                    const float b = ph.fin_bias ? ph.fin_bias[row] : 0.f;
                                    const float *resid = ph.fin_resid_ring ? ring_in : ph.fin_resid;
                                    float *dst = ph.fin_ring ? ring_out : ph.fin + (size_t)un.mat * TD_MAXB * ph.n_rows;
                                    float rs[TD_MAXB];
#pragma unroll
                                    for (int i = 0; i < TD_MAXB; ++i) rs[i] = (resid && i < nb) ? __ldcg(resid + (size_t)i * ph.n_rows + row) : 0.f;
#pragma unroll
                                    for (int i = 0; i < TD_MAXB; ++i)
                                        if (i < nb) dst[(size_t)i * ph.n_rows + row] = val[i] + b + rs[i];
                                }
                            } else if (finish) {
                                // output layer: logits by slot, and this warp's best (value, row) per sample
#pragma unroll
                                for (int i = 0; i < TD_MAXB; ++i) {
                                    if (i >= nb) break;
                                    float bv = rv ? val[i] : -INFINITY;
                                    int bi = rv ? row : 0x7fffffff;
                                    if (rv && !dead) P.logits[(size_t)slots[i] * ph.n_rows + row] = val[i];
#pragma unroll
                                    for (int o = 16; o > 0; o >>= 1) {
                                        const float v2 = __shfl_xor_sync(0xffffffffu, bv, o);
                                        const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
                                        if (v2 > bv || (v2 == bv && i2 < bi)) { bv = v2; bi = i2; }
                                    }
                                    if (lane == 0) {
                                        T.head_pv[(size_t)i * 4 * ph.n_tiles + un.tile * 4 + (warp & 3)] = bv;
                                        T.head_pi[(size_t)i * 4 * ph.n_tiles + un.tile * 4 + (warp & 3)] = bi;
                                    }
                                }
                            }
                        }
                        if (dead) *s_dead = 1;
                    }
                    acc_cnt = acc_base + (unsigned)(ue - ub);
                    lap(2);
                    td_bar(); // the accumulators of this range were read, hence every MMA that read B has completed
                    lap(ph.kind == TD_HEAD ? 9 : 2);
                    if (*(volatile int *)s_dead) dead = true;
                    ub = ue;
                }
                lap(ph.kind == TD_HEAD ? 9 : 2);
                team_barrier();
                lap(ph.kind == TD_HEAD ? 8 : 3);
                if (ph.kind == TD_HEAD && cta == 0) {
                    // ---- token choice: best candidate per sample, lowest id on ties
                    const int n_cand = 4 * ph.n_tiles;
                    for (int i = warp - 1; i < nb; i += TD_CWARPS) {
                        float b = -INFINITY;
                        int bi2 = 0x7fffffff;
                        for (int c2 = lane; c2 < n_cand; c2 += 32) {
                            const float v2 = __ldcg(T.head_pv + (size_t)i * n_cand + c2);
                            const int i2 = __ldcg(T.head_pi + (size_t)i * n_cand + c2);
                            if (v2 > b || (v2 == b && i2 < bi2)) { b = v2; bi2 = i2; }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            const float v2 = __shfl_xor_sync(0xffffffffu, b, o);
                            const int i2 = __shfl_xor_sync(0xffffffffu, bi2, o);
                            if (v2 > b || (v2 == b && i2 < bi2)) { b = v2; bi2 = i2; }
                        }
                        if (lane == 0) {
                            const int slot = j + i * G;
                            const int g = P.gen_count[slot];
                            if (g < P.log_stride) P.tok_log[(size_t)slot * P.log_stride + g] = bi2;
                            int feed = bi2;
                            if (g < P.n_teacher[slot]) feed = P.teacher[(size_t)slot * P.log_stride + g];
                            P.cur_tok[slot] = feed;
                            P.gen_count[slot] = g + 1;
                        }
                    }
                    lap(5);
                }
            }
            // ---- output edge
            if (cta == 0) {
                td_bar();
                if (ct == 0 && P.withhold_partition != p) st_release(T.flag_out + j, r + 1);
            }
        }
        // positions advance by the passes of this launch
        if (cta == 0)
            for (int s = ct; s < P.n_samples; s += TD_CTHREADS) T.pos[s] += P.n_pass;
        if (prof_on)
            for (int i = 0; i < PK_PROF_N; ++i)
                if (i != 6 && i != 7) P.prof[(size_t)blockIdx.x * PK_PROF_N + i] = pf[i];
        if (warp == 1 && lane == 0) {
            // no MMA may be in flight when tensor memory is freed (after a time-out some could still be)
            tg_commit(done_bar);
            const unsigned long long t0 = pk_now();
            while (!mbar_try_wait(done_bar, 0u) && pk_now() - t0 < 100000000ull) {}
        }
        __syncwarp();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(64u) : "memory");
    }
}

} // namespace mdi
