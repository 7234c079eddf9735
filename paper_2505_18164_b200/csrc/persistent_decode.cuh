// Persistent decode kernel: the whole recurrent pipeline of one generate call in ONE launch.
//
// The grid (one block per SM, cooperative launch so that all blocks are resident) is split into K
// teams, one per partition.  A team loops over its ticks of the schedule; per tick it waits for the
// flag of its input edge (the previous partition's activation ring slot, or for partition 0 the token
// chosen by the last partition), runs its blocks phase by phase with a team-wide barrier in between,
// and raises the flag of its output edge.  This replaces the paper's sockets and queues between
// nodes (Section III-A) by flags and ring slots in device memory.
//
// Inside a block, warp 8 is a producer: it walks the same static schedule as the 8 consumer warps
// but only issues bulk copies of weight tiles (16 row segments of up to 2 KB) into a ring of shared
// memory slots, each guarded by a full/empty mbarrier pair.  Weights do not depend on activations, so
// the producer runs ahead across phases, barriers and ticks and the HBM stream never stops while the
// consumers sit in a barrier or in a norm prologue.  A consumer warp owns whole tiles (row blocks
// b0+w, b0+w+8, ... of the block's share of a matrix): 16 independent accumulators per item, one
// transpose-reduce, and a lane-per-row epilogue, so up to 8 tiles are in work at a time.
//
// Every wait (flag, team barrier, mbarrier) is bounded in wall time: when a limit is hit an error
// word is set, the thread stops waiting for good, and the kernel runs to its end without further
// waits; the host then reports MDI_ERR_TIMEOUT.  Nothing traps.
#pragma once
#include <type_traits>

#include "step_kernels.cuh"

namespace mdi {

constexpr int PK_CWARPS = 8;
constexpr int PK_CTHREADS = PK_CWARPS * 32;
constexpr int PK_THREADS = PK_CTHREADS + 32;
constexpr int PK_SEGS = 16;
constexpr int PK_SLOT_BYTES = 32768;
constexpr int PK_MAX_SLOTS = 6;
constexpr int PK_MAXNB = 4;
constexpr int PK_SMEM_PHASES = 48; // phase descriptors of a team kept in shared memory (more: read from global memory)
constexpr unsigned long long PK_WAIT_NS = 2000000000ull; // default limit of a wait: 2 s

enum PkKind { PK_QKV = 0, PK_ATTN = 1, PK_OUT = 2, PK_FC1 = 3, PK_GATEUP = 4, PK_FC2 = 5, PK_HEAD = 6 };
enum PkProf { PF_FLAG = 0, PF_PROLOGUE = 1, PF_TILES = 2, PF_BARRIER = 3, PF_ATTN = 4, PF_HEADFIN = 5, PF_PROD_WAIT = 6,
              PF_PROD_TOTAL = 7, PF_TWAIT = 8, PF_TCOMP = 9, PF_TEPI = 10, PK_PROF_N = 12 };
enum PkErr { PKE_FLAG = 1, PKE_BARRIER = 2, PKE_FULL = 3, PKE_EMPTY = 4 };

struct PkPhase {
    int kind, n_rows, in_dim, n_blocks, layer_local, first_layer;
    const void *W, *W2;
    const float *bias, *gamma, *beta;
};

struct PkTeam {
    int first_cta, n_cta, phase_begin, n_phases, is_first, is_last, n_split;
    KvView kv;
    float *qbuf, *part, *hbuf, *x_embed, *x_last;
    const float *ring_in; // previous partition's ring (null for partition 0)
    float *ring_out;      // this partition's ring (null for the last partition)
    int *pos;             // [n_slots]
    unsigned *bar;        // team barrier counter (zero at launch)
    unsigned *flag_out;   // [G] passes this partition has finished per group (zero at launch)
    const unsigned *flag_in; // [G] the same of the previous partition (for partition 0: of the last)
};

struct PkParams {
    int d, n_head, n_kv_head, head_dim, d_ff, vocab, norm, act, rope, K, G, n_samples, gmax, n_pass, n_slots_ring, xs_floats;
    float eps, scale;
    const PkTeam *teams;
    const PkPhase *phases;
    const void *wte, *wpe;
    const float *rope_cos, *rope_sin;
    float *logits, *head_pv;
    int *head_pi;
    int *cur_tok, *tok_log, *gen_count;
    const int *teacher, *n_teacher;
    int log_stride;
    int *err;
    int hd_shift;               // log2(head_dim)
    unsigned long long wait_ns; // limit of every wait
    int withhold_partition;     // >= 0: that partition never raises its output flags (checks the time-out path)
    unsigned long long *prof; // optional [grid][PK_PROF_N] nanoseconds per category (thread 0 and the producer of each block)
};

// ---- PTX helpers ----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    // the last operand lets the hardware suspend the thread for up to that many nanoseconds while the phase is pending,
    // so that a waiting warp does not take issue slots and shared-memory bandwidth from the warps that compute
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned *p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(unsigned *p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(PK_CTHREADS) : "memory"); }
__device__ __forceinline__ unsigned long long pk_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded waits: the first probe is inline; the polling loop lives out of line (one copy, keeps the kernel's
// instruction footprint small).  A wait gives up after PK_WAIT_NS of wall time, records why in *err and marks
// the thread `dead`; `dead` is sticky, so after a failure (its own or one it sees in *err) a thread never waits again.
enum PkWaitKind { PKW_GLOBAL_GE = 0, PKW_MBAR = 1, PKW_SMEM_GE = 2 };
__device__ __forceinline__ bool pk_probe(int kind, const void *p, uint32_t a) {
    if (kind == PKW_GLOBAL_GE) return ld_acquire(reinterpret_cast<const unsigned *>(p)) >= a;
    if (kind == PKW_MBAR) return mbar_try_wait((uint32_t)(uintptr_t)p, a);
    return *reinterpret_cast<const volatile int *>(p) >= (int)a;
}
__device__ __noinline__ bool pk_wait_slow(int kind, const void *p, uint32_t a, int *err, int code, unsigned long long limit_ns) {
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        if (pk_probe(kind, p, a)) return false;
        if ((it & 63u) == 63u) {
            if (*(volatile int *)err) return true;
            const unsigned long long now = pk_now();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) break;
        }
    }
    atomicCAS(err, 0, code);
    return true;
}
__device__ __forceinline__ void wait_ge(const unsigned *p, unsigned target, int *err, int code, bool &dead, unsigned long long lim) {
    if (dead || pk_probe(PKW_GLOBAL_GE, p, target)) return;
    dead = pk_wait_slow(PKW_GLOBAL_GE, p, target, err, code, lim);
}
__device__ __forceinline__ void wait_mbar(uint32_t bar, uint32_t parity, int *err, int code, bool &dead, unsigned long long lim) {
    if (dead || pk_probe(PKW_MBAR, (const void *)(uintptr_t)bar, parity)) return;
    dead = pk_wait_slow(PKW_MBAR, (const void *)(uintptr_t)bar, parity, err, code, lim);
}
__device__ __forceinline__ void wait_smem_ge(const volatile int *p, int target, int *err, int code, bool &dead, unsigned long long lim) {
    if (dead || *p >= target) return;
    dead = pk_wait_slow(PKW_SMEM_GE, (const void *)p, (uint32_t)target, err, code, lim);
}
__device__ __noinline__ void pk_lap(unsigned long long *pf, unsigned long long *t, int cat) {
    const unsigned long long n = pk_now();
    pf[cat] += n - *t;
    *t = n;
}
__device__ __noinline__ float pk_act(float y, int act) { return act == 0 ? gelu_tanh_f(y) : gelu_erf_f(y); }
__device__ __noinline__ float pk_silu(float y) { return silu_f(y); }
// Merge of the attention splits for element e of one (item, head): partials are (max, sum, o[head_dim]) per split.
__device__ __noinline__ float pk_merge_splits(const float *pb, int n_split, int hd, int e) {
    float M = -INFINITY, L = 0.f, O = 0.f;
#pragma unroll 4
    for (int s2 = 0; s2 < n_split; ++s2) {
        const float ms = __ldcg(pb + (size_t)s2 * (hd + 2)), ls = __ldcg(pb + (size_t)s2 * (hd + 2) + 1),
                    os = __ldcg(pb + (size_t)s2 * (hd + 2) + 2 + e);
        if (ms != -INFINITY) {
            const float mn = fmaxf(M, ms), c0 = expf(M - mn), c1 = expf(ms - mn);
            L = L * c0 + ls * c1;
            O = O * c0 + os * c1;
            M = mn;
        }
    }
    return O / L;
}

// Which matrix row sits in segment i of row block blk.  Segments i and i+8 are partners: the two halves
// of a rotary pair (rows r and r + head_dim/2), or a gate row and its up row; otherwise rows are in order.
__device__ __forceinline__ int pk_seg_row(const PkPhase &ph, int rope, int hd, int blk, int i, bool &second) {
    second = false;
    if (ph.kind == PK_GATEUP) { second = i >= 8; return blk * 8 + (i & 7); }
    if (ph.kind == PK_QKV && rope) {
        // head_dim is a power of two: u / half and u % half as shift and mask
        const int u = blk * 8 + (i & 7), half = hd >> 1, hs = 31 - __clz(half);
        return ((u >> hs) << (hs + 1)) + (u & (half - 1)) + (i >= 8 ? half : 0);
    }
    return blk * PK_SEGS + i;
}

template <typename WT> __device__ __forceinline__ float wt_to_f(WT v);
template <> __device__ __forceinline__ float wt_to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float wt_to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// 16 bytes of weights widened to fp32
template <int ES> __device__ __forceinline__ void pk_unpack(const uint4 &v, float *w) {
    if constexpr (ES == 4) {
        w[0] = __uint_as_float(v.x); w[1] = __uint_as_float(v.y); w[2] = __uint_as_float(v.z); w[3] = __uint_as_float(v.w);
    } else {
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { w[2 * i] = __uint_as_float(u[i] << 16); w[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
    }
}

// 16 bytes of cache elements widened to fp32
template <typename KT> __device__ __forceinline__ void kv_unpack(const uint4 &v, float *w) {
    if constexpr (sizeof(KT) == 4) pk_unpack<4>(v, w);
    else if constexpr (std::is_same<KT, __half>::value) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) { const float2 f = __half22float2(h[i]); w[2 * i] = f.x; w[2 * i + 1] = f.y; }
    } else pk_unpack<2>(v, w);
}

// Position of logical column i inside an item's staged input row.  For 2-byte weights a lane consumes
// 8 consecutive columns per step as two float4 reads; columns are laid out so that each of those reads
// is contiguous across the 32 lanes (no bank conflicts): within every group of 256 columns, first the
// low halves of all lanes' 8-column runs, then the high halves.
template <int ES> __device__ __forceinline__ int xs_perm(int i) {
    if constexpr (ES == 2) return (i & ~255) | (((i >> 2) & 1) << 7) | (((i & 255) >> 3) << 2) | (i & 3);
    else return i;
}

__device__ __forceinline__ float cblock_sum(float v, float *red) { // over the 256 consumer threads
    v = warp_sum(v);
    consumer_bar();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    consumer_bar();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < PK_CWARPS; ++w) t += red[w];
    return t;
}

__device__ __forceinline__ void cblock_sum2(float &a, float &b, float *red /* [2 * PK_CWARPS] */) {
    a = warp_sum(a);
    b = warp_sum(b);
    consumer_bar();
    if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = a; red[PK_CWARPS + (threadIdx.x >> 5)] = b; }
    consumer_bar();
    a = b = 0.f;
#pragma unroll
    for (int w = 0; w < PK_CWARPS; ++w) { a += red[w]; b += red[PK_CWARPS + w]; }
}

template <typename WT, int NB, typename KT>
__global__ void __launch_bounds__(PK_THREADS, 1) k_persistent_decode(const PkParams P) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int ES = sizeof(WT);
    constexpr int VEC = 16 / ES;
    constexpr int KC = PK_SLOT_BYTES / (PK_SEGS * ES); // columns per tile
    unsigned char *ring_mem = smem;
    float *xs = reinterpret_cast<float *>(smem + (size_t)P.n_slots_ring * PK_SLOT_BYTES);
    float *att_o = xs + P.xs_floats;          // [256 * 8]
    float *att_m = att_o + 256 * 8;           // [128]
    float *att_l = att_m + 128;               // [128]
    float *red = att_l + 128;                 // [16]
    float *hbest_v = red + 16;                // [8][PK_MAXNB]
    int *hbest_i = reinterpret_cast<int *>(hbest_v + PK_CWARPS * PK_MAXNB);
    int *s_dead = hbest_i + PK_CWARPS * PK_MAXNB;  // [2]
    volatile int *s_cons = s_dead + 2;        // [PK_MAX_SLOTS] tiles consumed so far from each ring slot
    uint64_t *bars = reinterpret_cast<uint64_t *>(s_dead + 2 + PK_MAX_SLOTS); // [2 * n_slots]; 8-byte aligned (xs_floats is even)
    PkPhase *s_ph = reinterpret_cast<PkPhase *>(bars + 2 * PK_MAX_SLOTS);     // [PK_SMEM_PHASES]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int p = 0;
    while (p + 1 < P.K && (int)blockIdx.x >= P.teams[p + 1].first_cta) ++p;
    const PkTeam T = P.teams[p];
    const int cta = blockIdx.x - T.first_cta;
    const int K = P.K, G = P.G, d = P.d, hd = P.head_dim, NS = P.n_slots_ring;
    const uint32_t slot_base = smem_u32(ring_mem), full_base = smem_u32(bars), empty_base = smem_u32(bars + NS);

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full_base + 8 * s, 1);
            mbar_init(empty_base + 8 * s, PK_CWARPS); // one arrival per consumer warp (a warp that owns a tile brings all 8)
        }
        *s_dead = 0;
        for (int s = 0; s < PK_MAX_SLOTS; ++s) s_cons[s] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const bool ph_in_smem = T.n_phases <= PK_SMEM_PHASES;
    if (ph_in_smem)
        for (int i = tid; i < T.n_phases * (int)(sizeof(PkPhase) / 8); i += PK_THREADS)
            reinterpret_cast<unsigned long long *>(s_ph)[i] = reinterpret_cast<const unsigned long long *>(P.phases + T.phase_begin)[i];
    const PkPhase *phases = ph_in_smem ? s_ph : P.phases + T.phase_begin;
    __syncthreads();
    bool dead = false;
    const long total_slots = (long)P.n_pass * K;
    const bool prof_on = P.prof != nullptr && lane == 0 && (warp == 0 || warp == PK_CWARPS);
    unsigned long long pf[PK_PROF_N] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}, pf_t = prof_on ? pk_now() : 0;
    auto lap = [&](int cat) { if (prof_on) pk_lap(pf, &pf_t, cat); };

    if (warp == PK_CWARPS) {
        // =========================== producer ===========================
        // All 32 lanes walk the schedule; lane 0 waits for the ring slot and posts the byte count, then either
        // lane 0 copies the whole tile at once (rows contiguous in memory) or lanes 0..15 copy one segment each.
        unsigned seq = 0;   // tiles issued so far (fits 32 bits: checked on the host)
        int pslot = 0;
        uint32_t ppar = 0;
        for (long v = 0; v < total_slots && !dead; ++v) {
            if ((int)(v % K) >= G) continue;
            for (int pi = 0; pi < T.n_phases && !dead; ++pi) {
                const PkPhase ph = phases[pi];
                if (ph.kind == PK_ATTN) continue;
                const bool whole = ph.in_dim <= KC && ph.kind != PK_GATEUP && !(ph.kind == PK_QKV && P.rope);
                const int b0 = (int)((unsigned)cta * (unsigned)ph.n_blocks / (unsigned)T.n_cta), b1 = (int)((unsigned)(cta + 1) * (unsigned)ph.n_blocks / (unsigned)T.n_cta);
                for (int blk = b0; blk < b1 && !dead; ++blk)
                    for (int kc0 = 0; kc0 < ph.in_dim; kc0 += KC, ++seq) {
                        const int kc_len = min(KC, ph.in_dim - kc0);
                        const uint32_t seg_bytes = (uint32_t)kc_len * ES;
                        const int slot = pslot;
                        const uint32_t par = ppar;
                        if (++pslot == NS) { pslot = 0; ppar ^= 1u; }
                        lap(PF_PROD_TOTAL);
                        if (lane == 0 && seq >= (unsigned)NS) wait_mbar(empty_base + 8 * slot, par ^ 1, P.err, PKE_EMPTY, dead, P.wait_ns);
                        dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
                        lap(PF_PROD_WAIT);
                        if (dead) break;
                        const uint32_t full = full_base + 8 * slot, dst = slot_base + slot * PK_SLOT_BYTES;
                        if (whole) {
                            if (lane == 0) {
                                const int rows = min(PK_SEGS, ph.n_rows - blk * PK_SEGS);
                                mbar_expect_tx(full, rows * seg_bytes);
                                bulk_g2s(dst, reinterpret_cast<const WT *>(ph.W) + (size_t)blk * PK_SEGS * ph.in_dim, rows * seg_bytes, full);
                            }
                        } else {
                            bool second = false;
                            const int row = lane < PK_SEGS ? pk_seg_row(ph, P.rope, hd, blk, lane, second) : ph.n_rows;
                            const bool valid = row < ph.n_rows;
                            const unsigned mask = __ballot_sync(0xffffffffu, valid);
                            if (lane == 0) mbar_expect_tx(full, __popc(mask) * seg_bytes);
                            __syncwarp();
                            if (valid)
                                bulk_g2s(dst + lane * seg_bytes, reinterpret_cast<const WT *>(second ? ph.W2 : ph.W) + (size_t)row * ph.in_dim + kc0,
                                         seg_bytes, full);
                        }
                    }
            }
        }
        if (prof_on) {
            lap(PF_PROD_TOTAL);
            P.prof[(size_t)blockIdx.x * PK_PROF_N + PF_PROD_WAIT] = pf[PF_PROD_WAIT];
            P.prof[(size_t)blockIdx.x * PK_PROF_N + PF_PROD_TOTAL] = pf[PF_PROD_TOTAL] + pf[PF_PROD_WAIT];
        }
        if (dead && lane == 0) {
            // copies already issued target this block's shared memory: give them bounded time to land
            const unsigned long long t0 = pk_now();
            for (unsigned q = seq > (unsigned)NS ? seq - NS : 0; q < seq; ++q)
                while (!mbar_try_wait(full_base + 8 * (int)(q % NS), (uint32_t)((q / NS) & 1)) && pk_now() - t0 < 100000000ull) {}
        }
        return;
    }

    // =========================== consumers ===========================
    unsigned bar_epoch = 0;
    unsigned tile_seq = 0; // tiles this block has consumed so far (same in every consumer warp; fits 32 bits)
    auto team_barrier = [&]() {
        consumer_bar();
        if (tid == 0) {
            ++bar_epoch;
            if (T.n_cta > 1) {
                red_release_add(T.bar, 1u);
                wait_ge(T.bar, bar_epoch * (unsigned)T.n_cta, P.err, PKE_BARRIER, dead, P.wait_ns);
            }
            if (dead) *s_dead = 1;
        }
        consumer_bar();
        if (*(volatile int *)s_dead) dead = true;
    };
    const int qw = P.n_head * hd, kw = P.n_kv_head * hd;

    for (long v = 0; v < total_slots; ++v) {
        const int j = (int)(v % K);
        if (j >= G) continue;
        const unsigned r = (unsigned)(v / K);
        int nb = 0;
        int slots[NB], pos[NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const int s = j + i * G;
            slots[i] = s < P.n_samples ? s : j;
            if (s < P.n_samples) nb = i + 1;
        }
        // ---- input edge
        if (tid == 0) {
            if (!T.is_first) wait_ge(T.flag_in + j, r + 1, P.err, PKE_FLAG, dead, P.wait_ns);
            else if (r > 0) wait_ge(T.flag_in + j, r, P.err, PKE_FLAG, dead, P.wait_ns);
            if (dead) *s_dead = 1;
        }
        consumer_bar();
        if (*(volatile int *)s_dead) dead = true;
        lap(PF_FLAG);
#pragma unroll
        for (int i = 0; i < NB; ++i) pos[i] = __ldcg(T.pos + slots[i]) + (int)r;
        const float *x_in = T.is_first ? T.x_embed : T.ring_in + (size_t)j * P.gmax * d;
        float *x_out = T.is_last ? T.x_last : T.ring_out + (size_t)j * P.gmax * d;

        for (int pi = 0; pi < T.n_phases; ++pi) {
            const PkPhase ph = phases[pi];
            const int Kd = ph.in_dim, Kpad = (Kd + 255) & ~255;
            if (ph.kind == PK_ATTN) {
                // ---------------- attention over the cache: items (item, head, split) dealt to the team's blocks
                constexpr int EPL = 16 / (int)sizeof(KT);
                const int LPR = hd / EPL, RPW = 32 / LPR, NG = PK_CWARPS * RPW;
                const int sub = lane & (LPR - 1), grp = lane >> (31 - __clz(LPR));
                const int n_items = nb * P.n_head * T.n_split;
                for (int it = cta; it < n_items; it += T.n_cta) {
                    const int sp = it % T.n_split, h = (it / T.n_split) % P.n_head, b = it / (T.n_split * P.n_head);
                    int slot = slots[0], n_keys = pos[0] + 1;
#pragma unroll
                    for (int i = 1; i < NB; ++i) if (b == i) { slot = slots[i]; n_keys = pos[i] + 1; }
                    const int per = (n_keys + T.n_split - 1) / T.n_split;
                    const int lo = sp * per, hi = min(n_keys, lo + per);
                    const int kvh = h / (P.n_head / P.n_kv_head);
                    float *part = T.part + (((size_t)b * P.n_head + h) * T.n_split + sp) * (hd + 2);
                    if (lo < hi) {
                        float q[EPL], o[EPL];
#pragma unroll
                        for (int e = 0; e < EPL; ++e) { q[e] = __ldcg(T.qbuf + (size_t)b * qw + h * hd + sub * EPL + e) * P.scale; o[e] = 0.f; }
                        float m = -INFINITY, l = 0.f;
                        for (int j0 = lo + warp * RPW; j0 < hi; j0 += NG) {
                            const int jr = j0 + grp;
                            const bool live = jr < hi;
                            const KT *kp = kv_addr<KT>(T.kv, slot, ph.layer_local, 0, kvh, live ? jr : lo, sub * EPL);
                            const KT *vp = kp + (size_t)T.kv.n_kv_head * T.kv.page_tokens * hd;
                            float kf[EPL], vf[EPL];
                            const uint4 kk = __ldcg(reinterpret_cast<const uint4 *>(kp)), vv = __ldcg(reinterpret_cast<const uint4 *>(vp));
                            kv_unpack<KT>(kk, kf);
                            kv_unpack<KT>(vv, vf);
                            float s = 0.f;
#pragma unroll
                            for (int e = 0; e < EPL; ++e) s = fmaf(q[e], kf[e], s);
                            for (int w = LPR >> 1; w > 0; w >>= 1) s += __shfl_xor_sync(0xffffffffu, s, w);
                            if (live) {
                                const float mn = fmaxf(m, s), corr = expf(m - mn), pr = expf(s - mn);
                                l = l * corr + pr;
#pragma unroll
                                for (int e = 0; e < EPL; ++e) o[e] = o[e] * corr + pr * vf[e];
                                m = mn;
                            }
                        }
                        const int g = warp * RPW + grp;
                        if (sub == 0) { att_m[g] = m; att_l[g] = l; }
#pragma unroll
                        for (int e = 0; e < EPL; ++e) att_o[g * hd + sub * EPL + e] = o[e];
                        consumer_bar();
                        if (tid < hd) {
                            float M = -INFINITY;
                            for (int g2 = 0; g2 < NG; ++g2) M = fmaxf(M, att_m[g2]);
                            float L = 0.f, O = 0.f;
                            for (int g2 = 0; g2 < NG; ++g2) {
                                const float w = att_m[g2] == -INFINITY ? 0.f : expf(att_m[g2] - M);
                                L += att_l[g2] * w;
                                O += att_o[g2 * hd + tid] * w;
                            }
                            part[2 + tid] = O;
                            if (tid == 0) { part[0] = M; part[1] = L; }
                        }
                        consumer_bar();
                    } else if (tid < hd) {
                        part[2 + tid] = 0.f;
                        if (tid == 0) { part[0] = -INFINITY; part[1] = 0.f; }
                    }
                }
                lap(PF_ATTN);
                team_barrier();
                lap(PF_BARRIER);
                continue;
            }

            // ---------------- linear phase: stage the inputs (fp32) into shared memory
            for (int b = 0; b < NB; ++b) {
                const bool live = b < nb;
                const int slot = slots[b];
                // columns past the row's end (up to the next multiple of 256) meet zero weights in the last chunk:
                // they must be finite, whatever the shared memory held before
                for (int i = Kd + tid; i < Kpad; i += PK_CTHREADS) xs[b * Kpad + xs_perm<ES>(i)] = 0.f;
                // Common case (the source is a plain fp32 vector of at most 4096 elements: every phase but the
                // embedding and the split merge): float4 loads, the values stay in registers through the norm
                // statistics, and shared memory is written once.
                const bool plain = !(ph.kind == PK_QKV && ph.first_layer && T.is_first) && ph.kind != PK_OUT;
                if (plain && Kd <= 4 * 4 * PK_CTHREADS) {
                    const float *src = ph.kind == PK_QKV ? (ph.first_layer ? x_in : x_out) + (size_t)b * d
                                       : ph.kind == PK_FC2 ? T.hbuf + (size_t)b * Kd
                                                           : x_out + (size_t)b * d;
                    const float4 *src4 = reinterpret_cast<const float4 *>(src);
                    const int n4 = Kd >> 2;
                    float4 v[4], g4[4], o4[4];
                    const bool layer_norm = ph.gamma && P.norm == NORM_LAYER;
                    const float pilot = (live && layer_norm) ? __ldcg(src) : 0.f;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i4 = tid + u * PK_CTHREADS;
                        const bool in = i4 < n4;
                        v[u] = (live && in) ? __ldcg(src4 + i4) : make_float4(0.f, 0.f, 0.f, 0.f);
                        g4[u] = (ph.gamma && in) ? reinterpret_cast<const float4 *>(ph.gamma)[i4] : make_float4(0.f, 0.f, 0.f, 0.f);
                        o4[u] = (ph.gamma && ph.beta && in) ? reinterpret_cast<const float4 *>(ph.beta)[i4] : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    if (ph.gamma) {
                        // one reduction for both moments, taken about a pilot value (the row's first element) so that
                        // the variance does not cancel when the mean is large
                        float s1 = 0.f, s2 = 0.f;
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (tid + u * PK_CTHREADS < n4) {
                                const float c0 = v[u].x - pilot, c1 = v[u].y - pilot, c2 = v[u].z - pilot, c3 = v[u].w - pilot;
                                s1 += (c0 + c1) + (c2 + c3);
                                s2 += (c0 * c0 + c1 * c1) + (c2 * c2 + c3 * c3);
                            }
                        cblock_sum2(s1, s2, red);
                        const float dm = layer_norm ? s1 / (float)Kd : 0.f, mean = pilot + dm;
                        const float rstd = rsqrtf(fmaxf(s2 / (float)Kd - dm * dm, 0.f) + P.eps);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            v[u].x = (v[u].x - mean) * rstd * g4[u].x + o4[u].x;
                            v[u].y = (v[u].y - mean) * rstd * g4[u].y + o4[u].y;
                            v[u].z = (v[u].z - mean) * rstd * g4[u].z + o4[u].z;
                            v[u].w = (v[u].w - mean) * rstd * g4[u].w + o4[u].w;
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i4 = tid + u * PK_CTHREADS;
                        if (i4 < n4) *reinterpret_cast<float4 *>(xs + b * Kpad + xs_perm<ES>(4 * i4)) = v[u];
                    }
                    continue;
                }
                // Source of the staged row: a plain fp32 vector for most phases (loads issued in batches of 8 per
                // thread so that a batch costs one round trip to L2); the embedding and the split merge have
                // their own short loops.
                float s = 0.f;
                if (ph.kind == PK_QKV && ph.first_layer && T.is_first) {
                    const int tok = live ? min(max(__ldcg(P.cur_tok + slot), 0), P.vocab - 1) : 0;
                    const WT *te = reinterpret_cast<const WT *>(P.wte) + (size_t)tok * d;
                    const WT *pe = P.wpe ? reinterpret_cast<const WT *>(P.wpe) + (size_t)pos[b] * d : nullptr;
                    for (int i = tid; i < Kd; i += PK_CTHREADS) {
                        float xv = 0.f;
                        if (live) { xv = wt_to_f<WT>(te[i]); if (pe) xv += wt_to_f<WT>(pe[i]); }
                        xs[b * Kpad + xs_perm<ES>(i)] = xv;
                        if (live && cta == 0) T.x_embed[(size_t)b * d + i] = xv;
                    }
                } else if (ph.kind == PK_OUT) {
                    for (int i = tid; i < Kd; i += PK_CTHREADS) {
                        const int h = i >> P.hd_shift;
                        xs[b * Kpad + xs_perm<ES>(i)] =
                            live ? pk_merge_splits(T.part + ((size_t)b * P.n_head + h) * T.n_split * (hd + 2), T.n_split, hd, i - h * hd) : 0.f;
                    }
                } else {
                    const float *src = ph.kind == PK_QKV ? (ph.first_layer ? x_in : x_out) + (size_t)b * d
                                       : ph.kind == PK_FC2 ? T.hbuf + (size_t)b * Kd
                                                           : x_out + (size_t)b * d;
                    constexpr int SU = 8;
                    for (int i0 = tid; i0 < Kd; i0 += PK_CTHREADS * SU) {
                        float v[SU];
#pragma unroll
                        for (int u = 0; u < SU; ++u) {
                            const int i = i0 + u * PK_CTHREADS;
                            v[u] = (live && i < Kd) ? __ldcg(src + i) : 0.f;
                        }
#pragma unroll
                        for (int u = 0; u < SU; ++u) {
                            const int i = i0 + u * PK_CTHREADS;
                            if (i < Kd) xs[b * Kpad + xs_perm<ES>(i)] = v[u];
                        }
                    }
                }
                (void)s;
                if (ph.gamma) {
                    // gains and offsets do not depend on the activations: fetch them while the statistics reduce
                    constexpr int PRE = 8;
                    float gp[PRE], bp[PRE];
                    const bool pre = Kd <= PRE * PK_CTHREADS;
                    if (pre) {
#pragma unroll
                        for (int u = 0; u < PRE; ++u) {
                            const int i = tid + u * PK_CTHREADS;
                            gp[u] = i < Kd ? ph.gamma[i] : 0.f;
                            bp[u] = (i < Kd && ph.beta) ? ph.beta[i] : 0.f;
                        }
                    }
                    // one reduction for both moments; the variance is taken about a pilot value (the item's first
                    // element) so that it does not cancel when the mean is large
                    consumer_bar(); // the pilot element was staged by another thread
                    const float pilot = P.norm == NORM_LAYER ? xs[b * Kpad] : 0.f;
                    float s1 = 0.f, s2 = 0.f;
                    for (int i = tid; i < Kd; i += PK_CTHREADS) { const float c = xs[b * Kpad + xs_perm<ES>(i)] - pilot; s1 += c; s2 += c * c; }
                    cblock_sum2(s1, s2, red);
                    const float dm = P.norm == NORM_LAYER ? s1 / (float)Kd : 0.f;
                    const float mean = pilot + dm;
                    const float rstd = rsqrtf(fmaxf(s2 / (float)Kd - dm * dm, 0.f) + P.eps);
                    if (pre) {
#pragma unroll
                        for (int u = 0; u < PRE; ++u) {
                            const int i = tid + u * PK_CTHREADS;
                            if (i < Kd) xs[b * Kpad + xs_perm<ES>(i)] = (xs[b * Kpad + xs_perm<ES>(i)] - mean) * rstd * gp[u] + bp[u];
                        }
                    } else {
                        for (int i = tid; i < Kd; i += PK_CTHREADS) {
                            float xv = (xs[b * Kpad + xs_perm<ES>(i)] - mean) * rstd * ph.gamma[i];
                            if (ph.beta) xv += ph.beta[i];
                            xs[b * Kpad + xs_perm<ES>(i)] = xv;
                        }
                    }
                }
            }
            consumer_bar();
            lap(PF_PROLOGUE);

            // ---------------- stream the weight tiles.  Two ways to split the work, chosen per phase:
            //  ROWS = 2: all 8 consumer warps share every tile, warp w taking the partner segments w and w+8
            //            (lowest latency when this block has only a few tiles in the phase);
            //  ROWS = 16: a warp owns whole tiles (row blocks b0+w, b0+w+8, ...), so up to 8 tiles are in work
            //            at once (the long output-layer phase).
            // Either way the totals end up one row per even lane: lane 2i finishes the warp's i-th row.
            const int b0 = (int)((unsigned)cta * (unsigned)ph.n_blocks / (unsigned)T.n_cta), b1 = (int)((unsigned)(cta + 1) * (unsigned)ph.n_blocks / (unsigned)T.n_cta);
            const int n_chunks = (Kd + KC - 1) / KC;
            float best_v[NB];
            int best_i[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) { best_v[b] = -INFINITY; best_i[b] = 0x7fffffff; }
            size_t page_off[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b)
                page_off[b] = ph.kind == PK_QKV
                                  ? (size_t)T.kv.page_table[((size_t)slots[b] * T.kv.n_layers_local + ph.layer_local) * T.kv.pages_per_seq + (pos[b] >> T.kv.page_shift)] * T.kv.page_elems
                                  : 0;
            const float *xres = (ph.kind == PK_OUT && ph.first_layer) ? x_in : x_out;

            auto run_tiles = [&](auto rows_c) {
                constexpr int ROWS = decltype(rows_c)::value;
                constexpr bool SHARED = ROWS == 2;            // tile shared by all warps
                constexpr int KSB = SHARED ? 4 : 1;           // k-steps whose loads are issued together
                constexpr int RB = (ROWS == 16 && NB > 2) ? 8 : ROWS; // rows whose loads are issued together
                const int my_i = lane >> 1;                   // which of the warp's rows this lane finishes
                const int seg = SHARED ? warp + 8 * (my_i & 1) : my_i;
                const bool fin = (lane & 1) == 0 && my_i < ROWS;
                for (int blk = SHARED ? b0 : b0 + warp; blk < b1; blk += SHARED ? 1 : PK_CWARPS) {
                    // everything the epilogue needs besides the dot products is requested before waiting for the tile
                    // and not touched until the epilogue, so the loads stay in flight during the wait
                    bool sec;
                    const int row = pk_seg_row(ph, P.rope, hd, blk, seg, sec);
                    const bool rv = fin && row < ph.n_rows;
                    float eb = 0.f, xr[NB], rc[NB], rs[NB];
#pragma unroll
                    for (int b = 0; b < NB; ++b) { xr[b] = 0.f; rc[b] = 1.f; rs[b] = 0.f; }
                    if (rv) {
                        if (ph.kind != PK_GATEUP && ph.bias) eb = ph.bias[row];
#pragma unroll
                        for (int b = 0; b < NB; ++b) {
                            if (b < nb && (ph.kind == PK_OUT || ph.kind == PK_FC2)) xr[b] = __ldcg(xres + (size_t)b * d + row);
                            if (b < nb && ph.kind == PK_QKV && P.rope && row < qw + kw) {
                                const int i = row & ((hd >> 1) - 1);
                                rc[b] = P.rope_cos[(size_t)pos[b] * (hd >> 1) + i];
                                rs[b] = P.rope_sin[(size_t)pos[b] * (hd >> 1) + i];
                            }
                        }
                    }
                    float acc[ROWS][NB][2];
#pragma unroll
                    for (int r2 = 0; r2 < ROWS; ++r2)
#pragma unroll
                        for (int b = 0; b < NB; ++b) acc[r2][b][0] = acc[r2][b][1] = 0.f;
                    const unsigned seq0 = tile_seq + (unsigned)(blk - b0) * (unsigned)n_chunks;
                    for (int c = 0; c < n_chunks; ++c) {
                        const unsigned seq = seq0 + (unsigned)c;
                        const int lap_no = (int)(seq / (unsigned)NS), slot = (int)(seq - (unsigned)lap_no * (unsigned)NS);
                        const int kc0 = c * KC, kc_len = min(KC, Kd - kc0);
                        // a parity test is only meaningful once every earlier tile of this slot has been consumed
                        // (warps run ahead of one another); then wait for this tile's bytes to land
                        lap(PF_TILES);
                        wait_smem_ge(s_cons + slot, lap_no, P.err, PKE_FULL, dead, P.wait_ns);
                        wait_mbar(full_base + 8 * slot, (uint32_t)(lap_no & 1), P.err, PKE_FULL, dead, P.wait_ns);
                        lap(PF_TWAIT);
                        const unsigned char *tb = ring_mem + (size_t)slot * PK_SLOT_BYTES;
                        for (int k0 = lane * VEC; k0 < kc_len; k0 += 32 * VEC * KSB) {
#pragma unroll
                            for (int rb = 0; rb < ROWS; rb += RB) {
                                uint4 raw[KSB][RB];
#pragma unroll
                                for (int ks = 0; ks < KSB; ++ks)
#pragma unroll
                                    for (int r2 = 0; r2 < RB; ++r2) {
                                        const int k = k0 + ks * 32 * VEC;
                                        const int sg = SHARED ? warp + 8 * r2 : rb + r2;
                                        raw[ks][r2] = k < kc_len ? *reinterpret_cast<const uint4 *>(tb + ((size_t)sg * kc_len + k) * ES)
                                                                 : make_uint4(0u, 0u, 0u, 0u);
                                    }
#pragma unroll
                                for (int ks = 0; ks < KSB; ++ks) {
                                    const int k = min(k0 + ks * 32 * VEC, kc_len - VEC);
                                    float xv[NB][VEC];
#pragma unroll
                                    for (int b = 0; b < NB; ++b) {
                                        // 2-byte weights: column kc0+k starts this lane's 8-column run of its 256-column group
                                        const float *xrow = xs + b * Kpad + (ES == 2 ? ((kc0 + k) & ~255) + lane * 4 : kc0 + k);
#pragma unroll
                                        for (int q = 0; q < VEC / 4; ++q) {
                                            const float4 x4 = *reinterpret_cast<const float4 *>(xrow + q * 128);
                                            xv[b][4 * q + 0] = x4.x; xv[b][4 * q + 1] = x4.y; xv[b][4 * q + 2] = x4.z; xv[b][4 * q + 3] = x4.w;
                                        }
                                    }
#pragma unroll
                                    for (int r2 = 0; r2 < RB; ++r2) {
                                        float f[VEC];
                                        pk_unpack<ES>(raw[ks][r2], f);
#pragma unroll
                                        for (int b = 0; b < NB; ++b)
#pragma unroll
                                            for (int e = 0; e < VEC; ++e) acc[rb + r2][b][e & 1] = fmaf(f[e], xv[b][e], acc[rb + r2][b][e & 1]);
                                    }
                                }
                            }
                        }
                        __syncwarp();
                        if (lane == 0) {
                            // s_cons: "tile lap_no of this slot has landed" (any consumer that saw it may say so)
                            if (!SHARED || warp == 0) s_cons[slot] = lap_no + 1;
                            mbar_arrive(empty_base + 8 * slot, SHARED ? 1u : (uint32_t)PK_CWARPS);
                        }
                        lap(PF_TCOMP);
                    }
                    // reduce across lanes: lane 2i (and 2i+1) ends with the total of the warp's i-th row
                    float tot[NB], oth[NB];
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        if constexpr (SHARED) {
                            float ta = acc[0][b][0] + acc[0][b][1], tb2 = acc[1][b][0] + acc[1][b][1];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) { ta += __shfl_xor_sync(0xffffffffu, ta, o); tb2 += __shfl_xor_sync(0xffffffffu, tb2, o); }
                            tot[b] = (my_i & 1) ? tb2 : ta;
                        } else {
                            float v8[8], v4[4], v2[2];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const bool up = lane & 16;
                                const float lo8 = acc[i % ROWS][b][0] + acc[i % ROWS][b][1], hi8 = acc[(i + 8) % ROWS][b][0] + acc[(i + 8) % ROWS][b][1];
                                v8[i] = (up ? hi8 : lo8) + __shfl_xor_sync(0xffffffffu, up ? lo8 : hi8, 16);
                            }
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const bool up = lane & 8;
                                v4[i] = (up ? v8[i + 4] : v8[i]) + __shfl_xor_sync(0xffffffffu, up ? v8[i] : v8[i + 4], 8);
                            }
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                const bool up = lane & 4;
                                v2[i] = (up ? v4[i + 2] : v4[i]) + __shfl_xor_sync(0xffffffffu, up ? v4[i] : v4[i + 2], 4);
                            }
                            const bool up = lane & 2;
                            tot[b] = (up ? v2[1] : v2[0]) + __shfl_xor_sync(0xffffffffu, up ? v2[0] : v2[1], 2);
                            tot[b] += __shfl_xor_sync(0xffffffffu, tot[b], 1);
                        }
                        tot[b] += eb + xr[b];
                        // partner row (segment ^ 8): the other half of a rotary pair, or the "up" row of a gate row
                        oth[b] = __shfl_xor_sync(0xffffffffu, tot[b], SHARED ? 2 : 16);
                    }
                    if (rv) {
#pragma unroll
                        for (int b = 0; b < NB; ++b) {
                            if (b >= nb) break;
                            float y = tot[b];
                            if (ph.kind == PK_QKV) {
                                if (P.rope && row < qw + kw) y = seg < 8 ? y * rc[b] - oth[b] * rs[b] : y * rc[b] + oth[b] * rs[b];
                                if (row < qw) T.qbuf[(size_t)b * qw + row] = y;
                                else {
                                    const int rk = row - qw, which = rk >= kw, rl = rk - which * kw;
                                    KT *dst = reinterpret_cast<KT *>(T.kv.pool) + page_off[b] +
                                              ((size_t)(which * T.kv.n_kv_head + (rl >> P.hd_shift)) * T.kv.page_tokens + (pos[b] & (T.kv.page_tokens - 1))) * hd + (rl & (hd - 1));
                                    kv_store<KT>(dst, y);
                                }
                            } else if (ph.kind == PK_FC1) {
                                T.hbuf[(size_t)b * ph.n_rows + row] = pk_act(y, P.act);
                            } else if (ph.kind == PK_GATEUP) {
                                if (seg < 8) T.hbuf[(size_t)b * ph.n_rows + row] = pk_silu(y) * oth[b];
                            } else if (ph.kind == PK_OUT || ph.kind == PK_FC2) {
                                x_out[(size_t)b * d + row] = y;
                            } else { // PK_HEAD
                                P.logits[(size_t)slots[b] * ph.n_rows + row] = y;
                                if (y > best_v[b] || (y == best_v[b] && row < best_i[b])) { best_v[b] = y; best_i[b] = row; }
                            }
                        }
                    }
                    lap(PF_TEPI);
                }
            };
            if (b1 - b0 >= 6) run_tiles(std::integral_constant<int, 16>{});
            else run_tiles(std::integral_constant<int, 2>{});
            tile_seq += (unsigned)(b1 - b0) * (unsigned)n_chunks;
            lap(PF_TILES);

            if (ph.kind == PK_HEAD) {
                // per-block argmax partials, then block 0 of the team picks the tokens
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    float bv = best_v[b];
                    int bi = best_i[b];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const float vv = __shfl_xor_sync(0xffffffffu, bv, o);
                        const int ii = __shfl_xor_sync(0xffffffffu, bi, o);
                        if (vv > bv || (vv == bv && ii < bi)) { bv = vv; bi = ii; }
                    }
                    if (lane == 0) { hbest_v[warp * PK_MAXNB + b] = bv; hbest_i[warp * PK_MAXNB + b] = bi; }
                }
                consumer_bar();
                if (tid < NB) {
                    float bv = hbest_v[tid];
                    int bi = hbest_i[tid];
                    for (int w = 1; w < PK_CWARPS; ++w) {
                        const float vv = hbest_v[w * PK_MAXNB + tid];
                        const int ii = hbest_i[w * PK_MAXNB + tid];
                        if (vv > bv || (vv == bv && ii < bi)) { bv = vv; bi = ii; }
                    }
                    P.head_pv[(size_t)tid * T.n_cta + cta] = bv;
                    P.head_pi[(size_t)tid * T.n_cta + cta] = bi;
                }
                team_barrier();
                lap(PF_BARRIER);
                if (cta == 0) {
                    for (int i = warp; i < nb; i += PK_CWARPS) {
                        float bv = -INFINITY;
                        int bi = 0x7fffffff;
                        for (int c2 = lane; c2 < T.n_cta; c2 += 32) {
                            const float vv = __ldcg(P.head_pv + (size_t)i * T.n_cta + c2);
                            const int ii = __ldcg(P.head_pi + (size_t)i * T.n_cta + c2);
                            if (vv > bv || (vv == bv && ii < bi)) { bv = vv; bi = ii; }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            const float vv = __shfl_xor_sync(0xffffffffu, bv, o);
                            const int ii = __shfl_xor_sync(0xffffffffu, bi, o);
                            if (vv > bv || (vv == bv && ii < bi)) { bv = vv; bi = ii; }
                        }
                        if (lane == 0) {
                            const int slot = j + i * G;
                            const int g = P.gen_count[slot];
                            if (g < P.log_stride) P.tok_log[(size_t)slot * P.log_stride + g] = bi;
                            int feed = bi;
                            if (g < P.n_teacher[slot]) feed = P.teacher[(size_t)slot * P.log_stride + g];
                            P.cur_tok[slot] = feed;
                            P.gen_count[slot] = g + 1;
                        }
                    }
                }
                lap(PF_HEADFIN);
            } else {
                team_barrier();
                lap(PF_BARRIER);
            }
        }
        // ---- output edge
        if (cta == 0) {
            consumer_bar();
            if (tid == 0 && P.withhold_partition != p) st_release(T.flag_out + j, r + 1);
        }
    }
    // positions advance by the passes of this launch
    if (cta == 0)
        for (int s = tid; s < P.n_samples; s += PK_CTHREADS) T.pos[s] += P.n_pass;
    if (prof_on)
        for (int i = 0; i < PK_PROF_N; ++i)
            if (i != PF_PROD_WAIT && i != PF_PROD_TOTAL) P.prof[(size_t)blockIdx.x * PK_PROF_N + i] = pf[i];
}

} // namespace mdi
