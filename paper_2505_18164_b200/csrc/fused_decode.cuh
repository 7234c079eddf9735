// Fused-phase persistent decode kernel (GPT block, bf16 weights, fp32 key/value cache).
//
// Like k_persistent_decode this runs the whole recurrent pipeline of one generate call (paper, Section III-C,
// Algorithms 1 and 2) in ONE cooperative launch: one team of thread blocks per partition, flag handoff between
// teams, a producer warp per block that streams weights into a shared-memory ring ahead of the consumers.
// What differs is the cut of a block of the model into phases.  A transformer block costs two team-wide barriers
// here instead of five:
//
//   phase A (per head):  norm 1 -> q, k, v rows of ONE head -> cache append -> attention of that head ->
//                        that head's 64 columns of the output projection, a partial sum over all d_model rows
//   phase B (per slice): norm 2 -> a slice of hidden units of the MLP -> GELU -> those columns of the second
//                        MLP matrix, again a partial sum over all d_model rows
//
// Partial sums meet in a device-wide accumulator of 64-bit fixed-point numbers (red.add on integers is
// associative, so the result does not depend on the order in which blocks arrive), and every block keeps its
// own copy of the residual stream in shared memory, updated identically from the accumulators.
//
// Weights are stored a second time, per thread block, in exactly the order that block consumes them and in the
// register layout of the tensor-core instruction (mma.sync m16n8k16, bf16 x bf16 -> fp32): a "fragment block"
// (FB) of 512 bytes is a 16-row x 16-column tile, 16 bytes per lane.  The producer copies the block's stream
// 64 KB at a time (cp.async.bulk + mbarrier); consumers read a lane's 16 bytes with one shared-memory load
// and issue one MMA per FB.  The activation is the B operand: column 2b holds the high bf16 half of sample
// b's value, column 2b+1 the low half (x = hi + lo to ~16 mantissa bits), so up to 4 samples share a pass.
//
// Every wait is bounded in wall time exactly as in k_persistent_decode.
#pragma once
#include "persistent_decode.cuh"

namespace mdi {

// One bulk copy costs this GPU's copy engine about 0.26 us whatever its size (measured: 8 KB copies stream 31 GB/s per
// SM, 32 KB copies 125 GB/s, 64 KB copies 245 GB/s, however many are in flight), so slots are as large as the ring allows.
constexpr int FZ_SLOT_SHIFT = 7;
constexpr int FZ_SLOT_FB = 1 << FZ_SLOT_SHIFT; // fragment blocks per ring slot (64 KB)
constexpr int FZ_FB_BYTES = 512;
constexpr int FZ_SLOT_BYTES = FZ_SLOT_FB * FZ_FB_BYTES;
constexpr int FZ_MAX_SLOTS = 3;
constexpr int FZ_MAXNB = 4;
constexpr int FZ_CWARPS = 8;          // consumer warps (16 were measured slower: more barrier cost, fewer registers, the same chains)
constexpr int FZ_CTHREADS = FZ_CWARPS * 32;
constexpr int FZ_THREADS = FZ_CTHREADS + 32; // + the producer warp
constexpr int FZ_KREG = 8;           // k-steps per warp and tile in split-K parts (d_model <= 1024: 64 k-steps over 8 warps)
constexpr int FZ_TRACE_N = 128;
constexpr int FZ_MAX_PHASES = 40;    // phases of a team, segments and hidden units of a block kept in shared memory
constexpr int FZ_MAX_SEGS = 16;
constexpr int FZ_MAX_UNITS = 256;
constexpr int FZ_U = 4;              // elements of a d_model vector per consumer thread (d_model <= 1024)

constexpr float FZ_FIX_SCALE = 4294967296.f; // 2^32: accumulator resolution 2.3e-10

enum FzKind { FZ_A = 0, FZ_B = 1, FZ_HEAD = 2 };
enum FzProf { FZP_FLAG = 0, FZP_PROLOGUE = 1, FZP_MMA1 = 2, FZP_REDUCE = 3, FZP_ATTN = 4, FZP_MMA2 = 5, FZP_BARRIER = 8, FZP_FIN = 9 }; // 6, 7: the producer's

struct FzPhase {                 // one per (team, phase)
    int kind, layer_local;
    const float *gamma, *beta;   // norm of this phase's prologue
    const float *bias_in;        // added with the incoming accumulator (null: first phase of a step)
    const float *bias_rows;      // bias of the rows computed first (qkv / mlp up); null for the output layer
};
struct FzWork {                  // one per (block, phase)
    int unit;                    // A: head served by this block in this layer (-1: none)
    int n_tiles;                 // A: row tiles of q,k,v of one head; B: hidden units (16 rows each); HEAD: row tiles
    int tile0;                   // A: first of this block's q,k,v row tiles of the head; B: offset into the block's unit list; HEAD: first row tile
    int row_tile0, row_tiles;    // A: this block's row tiles of the head's output-projection columns
    int fb0, fb1;                // offsets of the two parts of the phase inside their segments
    int seg0, seg1;              // segment of each part
};
// A block's per-step stream is cut into segments: a segment ends after the q,k,v rows of a head, where the
// cache rows of that head follow in the ring (as many slots as the position asks for); every segment starts a new slot.
struct FzSeg {
    int fb_begin, n_fb;          // fragment blocks [fb_begin, fb_begin + n_fb) of the block's stream
    int slots_before;            // ring slots of the earlier segments of a step (cache slots not counted)
    int kv_layer, kv_head;       // the cache rows that follow this segment (-1: none, last segment)
};
struct FzBlock {
    const uint4 *stream;         // this block's weights of one step, in consumption order
    int n_fb, work_begin, seg_begin, n_seg, unit_begin, n_units;
};
struct FzTeam {
    int first_cta, n_cta, phase_begin, n_phases, is_first, is_last;
    KvView kv;
    const float *ring_in;
    float *ring_out;
    const float *bias_final;     // bias that completes the residual stream after the last phase B
    int *pos;
    unsigned *bar, *flag_out;
    const unsigned *flag_in;
    long long *acc;              // [3][gmax_nb][d] rotating accumulators
};
struct FzParams {
    int d, n_head, head_dim, d_ff, vocab, act, K, G, n_samples, gmax, n_pass, n_slots_ring;
    int xb_stride, hb_stride, ob_stride, part_floats, pages_per_seq;
    int kv_pps;                  // cache pages (of one head) per ring slot: cached rows reach the consumers through the ring
    int pair;                    // 1: a head is served by the two blocks of a cluster (q,k,v rows, cache rows of every page and
                                 // output rows split in halves; exchanges through distributed shared memory); 0: by one block
    int kv_rows;                 // rows of a cache page a block handles: page_tokens, or half of it when pair
    float eps, scale;
    const FzTeam *teams;
    const FzPhase *phases;
    const FzWork *works;
    const FzBlock *blocks;
    const FzSeg *segs;
    const int *units;
    const void *wte, *wpe;
    float *logits, *head_pv;
    int *head_pi;
    int *cur_tok, *tok_log, *gen_count;
    const int *teacher, *n_teacher;
    int log_stride;
    int *err;
    unsigned long long wait_ns;
    int withhold_partition;
    unsigned long long *prof;    // optional [grid][PK_PROF_N]
    unsigned long long *trace;   // optional [grid][FZ_TRACE_N]: time stamps of thread 0 at every lap of step trace_step
    int trace_step;
};

// Source of one fragment block, for the repacking kernel.
struct FzFbDesc {
    const void *src; // bf16 matrix, row-major
    int ld, row0, col0, rows; // leading dimension, first row and column, valid rows (<= 16; the rest reads as zero)
};

// One warp per fragment block: gather a 16 x 16 tile into the A-operand register order of mma.m16n8k16
// (lane = 4*g + q holds rows g and g+8, column pairs 2q and 2q+8).
__global__ void k_fz_repack(const FzFbDesc *desc, uint4 *stream, long n_fb) {
    const long fb = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (fb >= n_fb) return;
    const FzFbDesc ds = desc[fb];
    const int lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const uint16_t *W = reinterpret_cast<const uint16_t *>(ds.src);
    auto pair = [&](int r, int c) -> uint32_t {
        if (r >= ds.rows) return 0u;
        return *reinterpret_cast<const uint32_t *>(W + (size_t)(ds.row0 + r) * ds.ld + ds.col0 + c);
    };
    uint4 v;
    v.x = pair(g, 2 * q); v.y = pair(g + 8, 2 * q); v.z = pair(g, 2 * q + 8); v.w = pair(g + 8, 2 * q + 8);
    stream[fb * 32 + lane] = v;
}

__device__ __forceinline__ void fz_mma(float (&c)[4], const uint4 &a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void fz_red_add(long long *p, long long v) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// value -> (hi, lo) bf16 halves with hi + lo = value to about 16 mantissa bits
__device__ __forceinline__ void fz_split(float v, uint16_t &hi, uint16_t &lo) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    const __nv_bfloat16 l = __float2bfloat16_rn(v - __bfloat162float(h));
    hi = __bfloat16_as_ushort(h);
    lo = __bfloat16_as_ushort(l);
}

__device__ __forceinline__ void fz_bar() { asm volatile("bar.sync 1, %0;" ::"n"(FZ_CTHREADS) : "memory"); }
__device__ __forceinline__ void fz_block_sum2(float &a, float &b, float *red /* [2 * FZ_CWARPS] */) { // over the consumer threads
    a = warp_sum(a);
    b = warp_sum(b);
    fz_bar();
    if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = a; red[FZ_CWARPS + (threadIdx.x >> 5)] = b; }
    fz_bar();
    a = b = 0.f;
#pragma unroll
    for (int w = 0; w < FZ_CWARPS; ++w) { a += red[w]; b += red[FZ_CWARPS + w]; }
}

// ---- the two blocks of a cluster (pair mode): remote shared memory and a pair barrier built on mbarriers ----
__device__ __forceinline__ uint32_t fz_cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t fz_mapa(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void fz_st_remote(uint32_t addr, float v) { asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory"); }
__device__ __forceinline__ void fz_arrive_remote(uint32_t bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool fz_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
    return ok != 0;
}
// Bounded wait for the peer's arrivals on this block's pair barrier; true when the wait ran out (or another did).
__device__ __noinline__ bool fz_pair_wait(uint32_t bar, uint32_t parity, int *err, unsigned long long limit_ns) {
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        if (fz_try_wait_cluster(bar, parity)) return false;
        if ((it & 63u) == 63u) {
            if (*(volatile int *)err) return true;
            const unsigned long long now = pk_now();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) break;
        }
    }
    atomicCAS(err, 0, (int)PKE_BARRIER);
    return true;
}
__device__ __forceinline__ void fz_cluster_sync_all() { // every thread of every block of the cluster
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Moves a consumer warp's ring cursor to slot `target` (slots counted from the launch): for every slot on the way,
// arrive on the empty barrier of the slot left behind and wait (bounded) for the next one to be full.  Out of line:
// the kernel calls it from many places and its instruction footprint matters more than the call.
// Cursor state travels by value: x = open slot (0xffffffff: none yet), y = ring index | parity << 8 | dead << 16.
__device__ __noinline__ uint2 fz_advance_slow(uint2 cur, unsigned target, uint32_t full_base, uint32_t empty_base, int NS, int *err,
                                              unsigned long long wait_ns) {
    unsigned open_seq = cur.x;
    int ring_idx = (int)(cur.y & 0xffu);
    uint32_t ring_par = (cur.y >> 8) & 1u;
    bool dead = (cur.y >> 16) & 1u;
    while ((int)(open_seq - target) < 0) {
        if (open_seq != 0xffffffffu) {
            __syncwarp();
            if ((threadIdx.x & 31) == 0) mbar_arrive(empty_base + 8 * ring_idx, 1u);
            if (++ring_idx == NS) { ring_idx = 0; ring_par ^= 1u; }
        }
        ++open_seq;
        wait_mbar(full_base + 8 * ring_idx, ring_par, err, PKE_FULL, dead, wait_ns);
        dead = __any_sync(0xffffffffu, dead);
    }
    return make_uint2(open_seq, (unsigned)ring_idx | (ring_par << 8) | ((unsigned)dead << 16));
}

// Offsets of the kernel's shared-memory regions (bytes from the start of dynamic shared memory); host and
// device call the same function, so the launch size and the carve-up cannot disagree.
struct FzSmem {
    size_t xres, part, qkv, att_o, att_m, att_l, red, hbest_v, hbest_i, s_dead, s_kvdone, s_pilot, s_pt, s_units, xb, hb, ob,
        pairbuf, bars, s_ph, s_wk, s_seg, total;
};
__host__ __device__ inline FzSmem fz_smem_layout(int NB, int NS, int d, int hd, int part_floats, int pages_per_seq, int xbs, int hbs, int obs) {
    FzSmem L;
    size_t o = (size_t)NS * FZ_SLOT_BYTES;
    auto take = [&](size_t bytes, size_t align) { o = (o + align - 1) / align * align; const size_t r = o; o += bytes; return r; };
    L.xres = take((size_t)4 * NB * d, 16);
    L.part = take((size_t)4 * part_floats, 16);
    L.qkv = take((size_t)4 * NB * 3 * hd, 16);
    // attention scratch lives in the split-K buffer (never in use at the same time; the host sizes `part` for both):
    // [groups][hd] with groups * hd = 128 per warp, then up to 8 groups per warp (head_dim 16) of maxima and sums
    L.att_o = L.part;
    L.att_m = L.att_o + 4 * 128 * FZ_CWARPS;
    L.att_l = L.att_m + 4 * 8 * FZ_CWARPS;
    L.red = take(4 * 2 * FZ_CWARPS, 16);
    L.hbest_v = take(4 * FZ_CWARPS * FZ_MAXNB, 16);
    L.hbest_i = take(4 * FZ_CWARPS * FZ_MAXNB, 16);
    L.s_dead = take(8, 8);
    L.s_kvdone = take(8, 8);
    L.s_pilot = take(4 * FZ_MAXNB, 16);
    L.s_pt = take((size_t)4 * NB * pages_per_seq, 16);
    L.s_units = take(4 * FZ_MAX_UNITS, 16);
    L.xb = take((size_t)2 * 2 * NB * xbs, 16);
    L.hb = take((size_t)2 * 2 * NB * hbs, 16);
    L.ob = take((size_t)2 * 2 * NB * obs, 16);
    L.pairbuf = take((size_t)4 * 2 * NB * (hd + 2), 16); // [2 blocks][NB][max, sum, o[hd]] of the halves of a head's attention
    L.bars = take((2 * FZ_MAX_SLOTS + 1) * 8, 16);       // full[NS], empty[NS], then the pair barrier
    L.s_ph = take(sizeof(FzPhase) * FZ_MAX_PHASES, 16);
    L.s_wk = take(sizeof(FzWork) * FZ_MAX_PHASES, 16);
    L.s_seg = take(sizeof(FzSeg) * FZ_MAX_SEGS, 16);
    L.total = o;
    return L;
}

template <int NB>
__global__ void __launch_bounds__(FZ_THREADS, 1) k_fused_decode(const FzParams P) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d = P.d, hd = P.head_dim, NS = P.n_slots_ring, K = P.K, G = P.G;
    const FzSmem L = fz_smem_layout(NB, NS, d, hd, P.part_floats, P.pages_per_seq, P.xb_stride, P.hb_stride, P.ob_stride);
    unsigned char *ring_mem = smem;
    float *xres = reinterpret_cast<float *>(smem + L.xres);       // [NB][d] residual stream
    float *part = reinterpret_cast<float *>(smem + L.part);       // split-K partial sums
    float *qkv = reinterpret_cast<float *>(smem + L.qkv);         // [NB][3 hd]
    float *att_o = reinterpret_cast<float *>(smem + L.att_o);     // [groups][hd], groups * hd = 1024
    float *att_m = reinterpret_cast<float *>(smem + L.att_m);
    float *att_l = reinterpret_cast<float *>(smem + L.att_l);
    float *red = reinterpret_cast<float *>(smem + L.red);
    float *hbest_v = reinterpret_cast<float *>(smem + L.hbest_v);
    int *hbest_i = reinterpret_cast<int *>(smem + L.hbest_i);
    int *s_dead = reinterpret_cast<int *>(smem + L.s_dead);
    volatile int *s_kvdone = reinterpret_cast<volatile int *>(smem + L.s_kvdone); // head units whose cache append is complete
    float *s_pilot = reinterpret_cast<float *>(smem + L.s_pilot);
    int *s_pt = reinterpret_cast<int *>(smem + L.s_pt);           // [NB][pages_per_seq]
    int *s_units = reinterpret_cast<int *>(smem + L.s_units);
    uint16_t *xb = reinterpret_cast<uint16_t *>(smem + L.xb);     // [2 NB][xb_stride] norm output, hi/lo rows
    uint16_t *hb = reinterpret_cast<uint16_t *>(smem + L.hb);     // [2 NB][hb_stride] hidden units, hi/lo rows
    uint16_t *ob = reinterpret_cast<uint16_t *>(smem + L.ob);     // [2 NB][ob_stride] attention output, hi/lo rows
    float *pairbuf = reinterpret_cast<float *>(smem + L.pairbuf);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    FzPhase *s_ph = reinterpret_cast<FzPhase *>(smem + L.s_ph);
    FzWork *s_wk = reinterpret_cast<FzWork *>(smem + L.s_wk);
    FzSeg *s_seg = reinterpret_cast<FzSeg *>(smem + L.s_seg);

    int p = 0;
    while (p + 1 < K && (int)blockIdx.x >= P.teams[p + 1].first_cta) ++p;
    const FzTeam T = P.teams[p];
    const FzBlock B = P.blocks[blockIdx.x];
    const int cta = blockIdx.x - T.first_cta;
    const uint32_t slot_base = smem_u32(ring_mem), full_base = smem_u32(bars), empty_base = smem_u32(bars + NS), pair_bar = smem_u32(bars + 2 * FZ_MAX_SLOTS);
    const uint32_t rank = P.pair ? fz_cluster_rank() : 0u; // this block's half of a head
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full_base + 8 * s, 1);
            mbar_init(empty_base + 8 * s, FZ_CWARPS);
        }
        mbar_init(pair_bar, FZ_CTHREADS); // every consumer thread of the peer arrives
        *s_dead = 0;
        *s_kvdone = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < T.n_phases; i += FZ_THREADS) { s_ph[i] = P.phases[T.phase_begin + i]; s_wk[i] = P.works[B.work_begin + i]; }
    for (int i = tid; i < B.n_seg; i += FZ_THREADS) s_seg[i] = P.segs[B.seg_begin + i];
    for (int i = tid; i < B.n_units; i += FZ_THREADS) s_units[i] = P.units[B.unit_begin + i];
    __syncthreads();
    fz_cluster_sync_all(); // the peer's barriers exist before anything arrives on them (a cluster of one block otherwise)
    bool dead = false;
    const long total_slots = (long)P.n_pass * K;
    const int n_seg = B.n_seg, n_kvu = n_seg - 1; // head units (cache visits) of this block per step
    const int pt = T.kv.page_tokens, pshift = T.kv.page_shift, pps_shift = 31 - __clz(P.kv_pps);
    const int kvr = P.kv_rows, kvr_shift = 31 - __clz(P.kv_rows), kv_row0 = (int)rank * P.kv_rows;
    const uint32_t page_k_bytes = (uint32_t)kvr * hd * 4u; // keys (or values) of this block's rows of one page of one head
    // ring slots one sample's cached rows take
    auto kv_slots_of = [&](int n_old) { return (((n_old + pt - 1) >> pshift) + P.kv_pps - 1) >> pps_shift; };
    const bool prof_on = P.prof != nullptr && lane == 0 && (warp == 0 || warp == FZ_CWARPS);
    unsigned long long pf[PK_PROF_N] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}, pf_t = prof_on ? pk_now() : 0;
    int trace_ev = -1; // >= 0 while the traced step runs (thread 0 only)
    auto lap = [&](int cat) {
        if (prof_on) {
            pk_lap(pf, &pf_t, cat);
            if (trace_ev >= 0 && trace_ev < FZ_TRACE_N) P.trace[(size_t)blockIdx.x * FZ_TRACE_N + trace_ev++] = ((pf_t & 0x0fffffffffffffffull) << 4) | (unsigned)cat;
        }
    };

    if (warp == FZ_CWARPS) {
        // =========================== producer: weight segments and cache rows, slot by slot, step after step ===========================
        unsigned seq = 0;
        int slot = 0;
        uint32_t par = 0;
        long step_idx = 0;
        auto next_slot = [&]() { // lane 0 waits until the slot is free; false once a wait has run out
            lap(PF_PROD_TOTAL);
            if (lane == 0 && seq >= (unsigned)NS) wait_mbar(empty_base + 8 * slot, par ^ 1, P.err, PKE_EMPTY, dead, P.wait_ns);
            dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
            lap(PF_PROD_WAIT);
            return !dead;
        };
        auto bump = [&]() { ++seq; if (++slot == NS) { slot = 0; par ^= 1u; } };
        for (long v = 0; v < total_slots && !dead; ++v) {
            const int j = (int)(v % K);
            if (j >= G) continue;
            const int r = (int)(v / K);
            for (int sg = 0; sg < n_seg && !dead; ++sg) {
                const FzSeg S = s_seg[sg];
                const int nsl = (S.n_fb + FZ_SLOT_FB - 1) / FZ_SLOT_FB;
                for (int k = 0; k < nsl; ++k) {
                    if (!next_slot()) break;
                    if (lane == 0) {
                        const uint32_t bytes = (uint32_t)min(FZ_SLOT_FB, S.n_fb - k * FZ_SLOT_FB) * FZ_FB_BYTES;
                        mbar_expect_tx(full_base + 8 * slot, bytes);
                        bulk_g2s(slot_base + slot * FZ_SLOT_BYTES, B.stream + ((size_t)S.fb_begin + (size_t)k * FZ_SLOT_FB) * (FZ_FB_BYTES / 16), bytes, full_base + 8 * slot);
                    }
                    bump();
                }
                if (dead || S.kv_layer < 0) continue;
                // the row this head appended at the sample's previous visit must be in place before its page is copied
                if (step_idx > 0) {
                    if (lane == 0) wait_smem_ge(s_kvdone, (int)((step_idx - 1) * n_kvu + sg + 1), P.err, PKE_EMPTY, dead, P.wait_ns);
                    dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
                    if (dead) break;
                    __threadfence_block();
                }
                for (int i = 0; i < NB && !dead; ++i) {
                    const int smp = j + i * G;
                    if (smp >= P.n_samples) break;
                    const int n_old = __ldcg(T.pos + smp) + r, pages = (n_old + pt - 1) >> pshift;
                    const int *ptab = T.kv.page_table + ((size_t)smp * T.kv.n_layers_local + S.kv_layer) * T.kv.pages_per_seq;
                    int pg32 = 0; // page ids of 32 consecutive pages, one per lane: one request serves many slots
                    for (int i0 = 0; i0 < pages; i0 += P.kv_pps) {
                        if ((i0 & 31) == 0) pg32 = i0 + lane < pages ? ptab[i0 + lane] : 0;
                        const int cnt = min(P.kv_pps, pages - i0);
                        const int pg = __shfl_sync(0xffffffffu, pg32, (i0 + lane) & 31); // kv_pps divides 32: one chunk of 32 per slot
                        if (!next_slot()) break;
                        if (lane == 0) mbar_expect_tx(full_base + 8 * slot, (uint32_t)cnt * 2u * page_k_bytes);
                        __syncwarp();
                        if (lane < cnt) {
                            const float *kp = reinterpret_cast<const float *>(T.kv.pool) + (size_t)pg * T.kv.page_elems + ((size_t)S.kv_head * pt + kv_row0) * hd;
                            const uint32_t dst = slot_base + slot * FZ_SLOT_BYTES + (uint32_t)lane * 2u * page_k_bytes;
                            bulk_g2s(dst, kp, page_k_bytes, full_base + 8 * slot);
                            bulk_g2s(dst + page_k_bytes, kp + (size_t)T.kv.n_kv_head * pt * hd, page_k_bytes, full_base + 8 * slot);
                        }
                        bump();
                    }
                }
            }
            ++step_idx;
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
    } else {
    // =========================== consumers ===========================
    const int g = lane >> 2, q = lane & 3;
    const uint4 *ring4 = reinterpret_cast<const uint4 *>(ring_mem);
    constexpr int SLOT_U4 = FZ_SLOT_BYTES / 16;
    // Every consumer warp visits every ring slot in order: wait until it is full, use its own fragment blocks,
    // arrive on its empty barrier when moving on (also when it had nothing to read there).
    uint2 cur = make_uint2(0xffffffffu, 0u); // ring cursor (fz_advance_slow); none open yet
    const uint4 *slot4 = ring4;              // start of the open slot
    unsigned step_base = 0;                  // first slot of the current step
    auto advance = [&](unsigned target) {
        if (cur.x != target) {
            const unsigned long long w0 = prof_on ? pk_now() : 0;
            cur = fz_advance_slow(cur, target, full_base, empty_base, NS, P.err, P.wait_ns);
            if (prof_on) pf[11] += pk_now() - w0; // time in ring waits (also counted in the phase part that waited)
            slot4 = ring4 + (size_t)(cur.y & 0xffu) * SLOT_U4;
            if ((cur.y >> 16) & 1u) dead = true;
        }
    };

    // pair mode: arrive on the peer's barrier (after this thread's remote stores), wait for the peer's arrivals on ours
    const uint32_t peer_bar = P.pair ? fz_mapa(pair_bar, rank ^ 1u) : 0u;
    uint32_t pair_parity = 0;
    auto pair_sync = [&]() {
        fz_arrive_remote(peer_bar);
        if (!dead && fz_pair_wait(pair_bar, pair_parity, P.err, P.wait_ns)) dead = true;
        pair_parity ^= 1u;
    };

    unsigned bar_epoch = 0;
    auto team_barrier = [&]() {
        fz_bar();
        if (tid == 0) {
            ++bar_epoch;
            if (T.n_cta > 1) {
                red_release_add(T.bar, 1u);
                wait_ge(T.bar, bar_epoch * (unsigned)T.n_cta, P.err, PKE_BARRIER, dead, P.wait_ns);
            }
            if (dead) *s_dead = 1;
        }
        fz_bar();
        if (*(volatile int *)s_dead) dead = true;
    };

    // Split-K part: n_t row tiles x ks k-steps, fragment blocks in [tile][k-step] order starting at fb0 of the
    // segment whose first slot is slot0; warp w takes k-steps [w ks / 8, (w+1) ks / 8) of every tile (at most
    // FZ_KREG); partial sums go to `part`, to be added up after a block barrier.
    auto split_k = [&](unsigned slot0, int fb0, int n_t, int ks) {
        const int k0 = warp * ks / FZ_CWARPS, k1 = (warp + 1) * ks / FZ_CWARPS, nk = k1 - k0;
        uint32_t bf[FZ_KREG][2];
        const uint16_t *brow = xb + (size_t)g * P.xb_stride + 2 * q;
#pragma unroll
        for (int kk = 0; kk < FZ_KREG; ++kk) {
            const bool on = kk < nk && g < 2 * NB;
            bf[kk][0] = on ? *reinterpret_cast<const uint32_t *>(brow + (k0 + kk) * 16) : 0u;
            bf[kk][1] = on ? *reinterpret_cast<const uint32_t *>(brow + (k0 + kk) * 16 + 8) : 0u;
        }
        for (int t = 0; t < n_t; ++t) {
            float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f};
            const int f0 = fb0 + t * ks + k0;
            advance(slot0 + (unsigned)(f0 >> FZ_SLOT_SHIFT));
            if (nk > 0) {
                const int n1 = min(nk, FZ_SLOT_FB - (f0 & (FZ_SLOT_FB - 1)));
                const uint4 *p1 = slot4 + (f0 & (FZ_SLOT_FB - 1)) * 32 + lane;
                uint4 a[FZ_KREG];
#pragma unroll
                for (int kk = 0; kk < FZ_KREG; ++kk)
                    if (kk < n1) a[kk] = p1[kk * 32];
                if (n1 < nk) { // the warp's run crosses into the next slot
                    advance(slot0 + (unsigned)(f0 >> FZ_SLOT_SHIFT) + 1u);
                    const uint4 *p2 = slot4 + lane;
#pragma unroll
                    for (int kk = 0; kk < FZ_KREG; ++kk)
                        if (kk >= n1 && kk < nk) a[kk] = p2[(kk - n1) * 32];
                }
#pragma unroll
                for (int kk = 0; kk < FZ_KREG; ++kk)
                    if (kk < nk) fz_mma((kk & 1) ? cb : ca, a[kk], bf[kk][0], bf[kk][1]);
            }
            if (q < NB) {
                part[((t * FZ_CWARPS + warp) * 16 + g) * NB + q] = (ca[0] + cb[0]) + (ca[1] + cb[1]);
                part[((t * FZ_CWARPS + warp) * 16 + g + 8) * NB + q] = (ca[2] + cb[2]) + (ca[3] + cb[3]);
            }
        }
    };
    // Tile-split part: n_t row tiles x ks k-steps; warp w takes tiles w, w+8, ...; the fragment blocks of a round
    // of up to 8 tiles are stored [k-step][tile] so that the warps move through the ring together.  B operand rows
    // come from `opnd` (hi/lo rows of `stride` elements).  epi(tile, c) receives the finished accumulators.
    auto tile_split = [&](unsigned slot0, int fb0, int n_t, int ks, const uint16_t *opnd, int stride, auto &&epi) {
        const uint16_t *brow = opnd + (size_t)g * stride + 2 * q;
        const bool bon = g < 2 * NB;
        for (int r0 = 0; r0 < n_t; r0 += FZ_CWARPS) {
            const int n_r = min(FZ_CWARPS, n_t - r0);
            const bool active = warp < n_r;
            const int base = fb0 + r0 * ks + (active ? warp : 0); // idle warps follow warp 0 through the ring
            float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f};
            int k = 0;
            while (k < ks) {
                const int fb = base + k * n_r;
                advance(slot0 + (unsigned)(fb >> FZ_SLOT_SHIFT));
                const int room = FZ_SLOT_FB - (fb & (FZ_SLOT_FB - 1));
                const int k_end = min(ks, k + (n_r == FZ_CWARPS ? (room + FZ_CWARPS - 1) / FZ_CWARPS : (room + n_r - 1) / n_r)); // k-steps in this slot
                const uint4 *ap = slot4 + (fb & (FZ_SLOT_FB - 1)) * 32 + lane;
                const int stp = n_r * 32;
                for (; k + 4 <= k_end; k += 4, ap += 4 * stp) {
                    uint4 a[4];
                    uint32_t b0[4], b1[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        a[u] = ap[u * stp];
                        b0[u] = bon ? *reinterpret_cast<const uint32_t *>(brow + (k + u) * 16) : 0u;
                        b1[u] = bon ? *reinterpret_cast<const uint32_t *>(brow + (k + u) * 16 + 8) : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) fz_mma((u & 1) ? cb : ca, a[u], b0[u], b1[u]);
                }
#pragma unroll 1
                for (; k < k_end; ++k, ap += stp) {
                    const uint4 a = *ap;
                    const uint32_t b0 = bon ? *reinterpret_cast<const uint32_t *>(brow + k * 16) : 0u;
                    const uint32_t b1 = bon ? *reinterpret_cast<const uint32_t *>(brow + k * 16 + 8) : 0u;
                    fz_mma(ca, a, b0, b1);
                }
            }
            if (active) {
                const float c[4] = {ca[0] + cb[0], ca[1] + cb[1], ca[2] + cb[2], ca[3] + cb[3]};
                epi(r0 + warp, c);
            }
        }
    };

    unsigned phase_ctr = 0; // phases this team has run since the launch (selects the rotating accumulators)
    int kv_units_done = 0;  // head units this block has finished since the launch
    const size_t acc_stride = (size_t)NB * d;
    // this thread's elements of the next prologue's vectors, requested before the wait that precedes the prologue
    float gam[FZ_U], bet[FZ_U], bin[FZ_U];
    auto prefetch_vectors = [&](const FzPhase &ph, bool norm) {
#pragma unroll
        for (int u = 0; u < FZ_U; ++u) {
            const int i = tid + u * FZ_CTHREADS;
            gam[u] = (norm && i < d) ? ph.gamma[i] : 0.f;
            bet[u] = (norm && i < d) ? ph.beta[i] : 0.f;
            bin[u] = (ph.bias_in && i < d) ? ph.bias_in[i] : 0.f;
        }
    };
    auto has_work_of = [&](int pi) { return s_ph[pi].kind == FZ_A ? s_wk[pi].unit >= 0 : s_wk[pi].n_tiles > 0; };

    for (long v = 0; v < total_slots; ++v) {
        const int j = (int)(v % K);
        if (j >= G) continue;
        const unsigned r = (unsigned)(v / K);
        trace_ev = (P.trace && tid == 0 && (long)P.trace_step == v) ? 0 : -1;
        int nb = 0;
        int slots[NB], pos[NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const int s = j + i * G;
            slots[i] = s < P.n_samples ? s : j;
            if (s < P.n_samples) nb = i + 1;
        }
        prefetch_vectors(s_ph[0], has_work_of(0));
        // ---- input edge
        if (tid == 0) {
            if (!T.is_first) wait_ge(T.flag_in + j, r + 1, P.err, PKE_FLAG, dead, P.wait_ns);
            else if (r > 0) wait_ge(T.flag_in + j, r, P.err, PKE_FLAG, dead, P.wait_ns);
            if (dead) *s_dead = 1;
        }
        fz_bar();
        if (*(volatile int *)s_dead) dead = true;
        lap(FZP_FLAG);
        int kvs_per_unit = 0; // ring slots the cached rows of one head take in this step (all samples of the group)
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            pos[i] = __ldcg(T.pos + slots[i]) + (int)r;
            if (i < nb) kvs_per_unit += kv_slots_of(pos[i]);
        }
        // ---- the step's input: embedding (partition 0) or the previous partition's ring slot
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (T.is_first) {
                const int tok = b < nb ? min(max(__ldcg(P.cur_tok + slots[b]), 0), P.vocab - 1) : 0;
                const __nv_bfloat16 *te = reinterpret_cast<const __nv_bfloat16 *>(P.wte) + (size_t)tok * d;
                const __nv_bfloat16 *pe = P.wpe ? reinterpret_cast<const __nv_bfloat16 *>(P.wpe) + (size_t)pos[b] * d : nullptr;
                for (int i = tid; i < d; i += FZ_CTHREADS) {
                    float xv = 0.f;
                    if (b < nb) { xv = __bfloat162float(te[i]); if (pe) xv += __bfloat162float(pe[i]); }
                    xres[b * d + i] = xv;
                    if (i == 0) s_pilot[b] = xv;
                }
            } else {
                const float *src = T.ring_in + ((size_t)j * P.gmax + b) * d;
                for (int i = tid; i < d; i += FZ_CTHREADS) {
                    const float xv = b < nb ? __ldcg(src + i) : 0.f;
                    xres[b * d + i] = xv;
                    if (i == 0) s_pilot[b] = xv;
                }
            }
        }
        fz_bar();

        for (int pi = 0; pi < T.n_phases; ++pi, ++phase_ctr) {
            const FzPhase ph = s_ph[pi];
            const FzWork wk = s_wk[pi];
            long long *acc_w = T.acc + (size_t)(phase_ctr % 3u) * acc_stride;
            const long long *acc_r = T.acc + (size_t)((phase_ctr + 2u) % 3u) * acc_stride;
            long long *acc_z = T.acc + (size_t)((phase_ctr + 1u) % 3u) * acc_stride;
            const bool has_work = ph.kind == FZ_A ? wk.unit >= 0 : wk.n_tiles > 0;
            // ---- requests whose answers are needed later in the phase
            long long av[NB][FZ_U];
            if (ph.bias_in) {
#pragma unroll
                for (int b = 0; b < NB; ++b)
#pragma unroll
                    for (int u = 0; u < FZ_U; ++u) {
                        const int i = tid + u * FZ_CTHREADS;
                        av[b][u] = (i < d && b < nb) ? __ldcg(acc_r + (size_t)b * d + i) : 0ll;
                    }
            }
            float brw[4] = {0.f, 0.f, 0.f, 0.f}; // biases of the first four rows this thread finishes after the split-K part
            if (has_work && ph.kind == FZ_A) {
                const int per_a = 16 * wk.n_tiles, n_out = nb * per_a, qw = P.n_head * hd;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int o = tid + u * FZ_CTHREADS;
                    if (o < n_out) { const int rr = wk.tile0 * 16 + o % per_a, which = rr / hd; brw[u] = ph.bias_rows[which * qw + wk.unit * hd + (rr - which * hd)]; }
                }
                // page-table entries of this head's cache rows
                for (int i = tid; i < NB * P.pages_per_seq; i += FZ_CTHREADS) {
                    const int b = i / P.pages_per_seq, pg = i - b * P.pages_per_seq;
                    s_pt[i] = (b < nb && pg <= (pos[b] >> pshift))
                                  ? T.kv.page_table[((size_t)slots[b] * T.kv.n_layers_local + ph.layer_local) * T.kv.pages_per_seq + pg] : 0;
                }
            } else if (has_work && ph.kind == FZ_B) {
                const int n_out = NB * 16 * wk.n_tiles;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int o = tid + u * FZ_CTHREADS;
                    if (o < n_out) { const int rr = o % (16 * wk.n_tiles); brw[u] = ph.bias_rows[s_units[wk.tile0 + (rr >> 4)] * 16 + (rr & 15)]; }
                }
            }
            // ---- prologue: complete the residual stream with the previous phase's sum, then the norm
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                float xv[FZ_U];
#pragma unroll
                for (int u = 0; u < FZ_U; ++u) {
                    const int i = tid + u * FZ_CTHREADS;
                    xv[u] = 0.f;
                    if (i < d) {
                        xv[u] = xres[b * d + i];
                        if (ph.bias_in && b < nb) {
                            xv[u] += bin[u] + (float)((double)av[b][u] * (1.0 / 4294967296.0));
                            xres[b * d + i] = xv[u];
                        }
                    }
                }
                if (!has_work) continue;
                // one reduction for both moments, taken about a pilot value (an element of the step's input) so that
                // the variance does not cancel when the mean is large
                const float pilot = s_pilot[b];
                float s1 = 0.f, s2 = 0.f;
#pragma unroll
                for (int u = 0; u < FZ_U; ++u)
                    if (tid + u * FZ_CTHREADS < d) { const float cv = xv[u] - pilot; s1 += cv; s2 += cv * cv; }
                fz_block_sum2(s1, s2, red);
                const float dm = s1 / (float)d, mean = pilot + dm;
                const float rstd = rsqrtf(fmaxf(s2 / (float)d - dm * dm, 0.f) + P.eps);
#pragma unroll
                for (int u = 0; u < FZ_U; ++u) {
                    const int i = tid + u * FZ_CTHREADS;
                    if (i < d) {
                        const float nv = (xv[u] - mean) * rstd * gam[u] + bet[u];
                        uint16_t hi, lo;
                        fz_split(b < nb ? nv : 0.f, hi, lo);
                        xb[(size_t)(2 * b) * P.xb_stride + i] = hi;
                        xb[(size_t)(2 * b + 1) * P.xb_stride + i] = lo;
                    }
                }
            }
            // accumulator of the phase after next: cleared by one block of the team (all its readers passed the last barrier)
            if ((int)(phase_ctr % (unsigned)T.n_cta) == cta)
                for (int i = tid; i < (int)acc_stride; i += FZ_CTHREADS) acc_z[i] = 0ll;
            fz_bar();
            lap(FZP_PROLOGUE);

            const unsigned seg_slot0 = step_base + (unsigned)s_seg[wk.seg0].slots_before + (unsigned)(wk.seg0 * kvs_per_unit);
            const unsigned seg_slot1 = step_base + (unsigned)s_seg[wk.seg1].slots_before + (unsigned)(wk.seg1 * kvs_per_unit);
            const int ks = d >> 4;
            // ---- first part (not the output layer): rows by split-K, then bias and what follows per row
            if (has_work && ph.kind != FZ_HEAD) {
                const bool is_a = ph.kind == FZ_A;
                const int n_t = wk.n_tiles, h = wk.unit, qw = P.n_head * hd;
                split_k(seg_slot0, wk.fb0, n_t, ks);
                fz_bar();
                lap(FZP_MMA1);
                const int per = 16 * n_t, n_out = (is_a ? nb : NB) * per;
                const uint32_t peer_qkv = (is_a && P.pair) ? fz_mapa(smem_u32(qkv), rank ^ 1u) : 0u;
                auto finish_row = [&](int o, float bias) {
                    const int b = o / per, rr = o - b * per, t = rr >> 4, row = rr & 15;
                    float s = 0.f;
#pragma unroll
                    for (int w = 0; w < FZ_CWARPS; ++w) s += part[((t * FZ_CWARPS + w) * 16 + row) * NB + b];
                    s += bias;
                    if (is_a) {
                        // q, k, v of head h (this block's rows of them; the peer gets a copy); k and v are appended to the cache
                        const int rg = wk.tile0 * 16 + rr, which = rg / hd, e = rg - which * hd;
                        qkv[b * 3 * hd + rg] = s;
                        if (P.pair) fz_st_remote(peer_qkv + (uint32_t)(b * 3 * hd + rg) * 4u, s);
                        if (which > 0) {
                            int pb = pos[0];
#pragma unroll
                            for (int i = 1; i < NB; ++i) if (b == i) pb = pos[i];
                            const int pg = s_pt[b * P.pages_per_seq + (pb >> pshift)];
                            float *dst = reinterpret_cast<float *>(T.kv.pool) + (size_t)pg * T.kv.page_elems +
                                         ((size_t)((which - 1) * T.kv.n_kv_head + h) * pt + (pb & (pt - 1))) * hd + e;
                            *dst = s;
                        }
                    } else {
                        uint16_t hi, lo;
                        fz_split(b < nb ? pk_act(s, P.act) : 0.f, hi, lo);
                        hb[(size_t)(2 * b) * P.hb_stride + rr] = hi;
                        hb[(size_t)(2 * b + 1) * P.hb_stride + rr] = lo;
                    }
                };
#pragma unroll
                for (int u = 0; u < 4; ++u) { const int o = tid + u * FZ_CTHREADS; if (o < n_out) finish_row(o, brw[u]); }
#pragma unroll 1
                for (int o = tid + 4 * FZ_CTHREADS; o < n_out; o += FZ_CTHREADS) {
                    const int rr = o % per;
                    float bias;
                    if (is_a) { const int rg = wk.tile0 * 16 + rr, which = rg / hd; bias = ph.bias_rows[which * qw + h * hd + (rg - which * hd)]; }
                    else bias = ph.bias_rows[s_units[wk.tile0 + (rr >> 4)] * 16 + (rr & 15)];
                    finish_row(o, bias);
                }
                if (is_a) asm volatile("fence.proxy.async.global;" ::: "memory"); // the producers' bulk copies read these rows in later steps
                if (is_a && P.pair) pair_sync(); // both halves of q, k, v are in place, and the peer's cache rows are written
                fz_bar();
                if (is_a) {
                    ++kv_units_done;
                    if (tid == 0) { __threadfence_block(); *s_kvdone = kv_units_done; }
                }
                lap(FZP_REDUCE);
            }
            // ---- attention of head h over cache rows 0..pos-1 (from the ring) and the new row (shared memory)
            if (has_work && ph.kind == FZ_A) {
                const int LPR = hd >> 2, RPW = 32 / LPR, NG = FZ_CWARPS * RPW;
                const int sub = lane & (LPR - 1), grp = warp * RPW + lane / LPR;
                unsigned kv_slot = seg_slot0 + (unsigned)((s_seg[wk.seg0].n_fb + FZ_SLOT_FB - 1) / FZ_SLOT_FB);
                const uint32_t peer_pairbuf = P.pair ? fz_mapa(smem_u32(pairbuf), rank ^ 1u) : 0u;
                float *my_half = pairbuf + (size_t)rank * NB * (hd + 2);
#pragma unroll 1
                for (int b = 0; b < nb; ++b) {
                    const float *qv = qkv + b * 3 * hd;
                    const float4 q4 = make_float4(qv[sub * 4] * P.scale, qv[sub * 4 + 1] * P.scale, qv[sub * 4 + 2] * P.scale, qv[sub * 4 + 3] * P.scale);
                    float m = -INFINITY, l = 0.f;
                    float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    int n_old = pos[0];
#pragma unroll
                    for (int i = 1; i < NB; ++i) if (b == i) n_old = pos[i];
                    // chunks: one per ring slot of cached rows (this block's rows of each page), then one for the new row
                    // (first block of the head, group 0, from shared memory); a group folds four rows per iteration:
                    // four independent dot products, one rescale of the running sums
                    const int n_sl = kv_slots_of(n_old), n_pages = (n_old + pt - 1) >> pshift;
#pragma unroll 1
                    for (int c = 0; c <= n_sl; ++c) {
                        const bool last = c == n_sl;
                        int n_here = rank == 0 ? 1 : 0, page0 = 0;
                        const unsigned char *sp = nullptr;
                        if (!last) {
                            advance(kv_slot++);
                            sp = reinterpret_cast<const unsigned char *>(slot4) + sub * 16;
                            page0 = c << pps_shift;
                            n_here = min(P.kv_pps, n_pages - page0) << kvr_shift;
                        }
#pragma unroll 1
                        for (int jj0 = 0; jj0 < n_here; jj0 += 4 * NG) {
                            float4 kk[4], vv[4];
                            float sc[4];
                            bool live[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const int jj = jj0 + u * NG + grp, pgs = jj >> kvr_shift, row = jj & (kvr - 1);
                                // position of the row: page, this block's first row of a page, row
                                live[u] = jj < n_here && (last || ((page0 + pgs) << pshift) + kv_row0 + row < n_old);
                                kk[u] = vv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                                if (live[u]) {
                                    if (!last) {
                                        const unsigned char *kp = sp + (size_t)pgs * 2u * page_k_bytes + (size_t)row * hd * 4;
                                        kk[u] = *reinterpret_cast<const float4 *>(kp);
                                        vv[u] = *reinterpret_cast<const float4 *>(kp + page_k_bytes);
                                    } else {
                                        kk[u] = *reinterpret_cast<const float4 *>(qv + hd + sub * 4);
                                        vv[u] = *reinterpret_cast<const float4 *>(qv + 2 * hd + sub * 4);
                                    }
                                }
                            }
#pragma unroll
                            for (int u = 0; u < 4; ++u) sc[u] = q4.x * kk[u].x + q4.y * kk[u].y + q4.z * kk[u].z + q4.w * kk[u].w;
                            for (int w = LPR >> 1; w > 0; w >>= 1) {
#pragma unroll
                                for (int u = 0; u < 4; ++u) sc[u] += __shfl_xor_sync(0xffffffffu, sc[u], w);
                            }
                            if (live[0] || live[1] || live[2] || live[3]) {
                                float mn = m;
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    if (!live[u]) sc[u] = -INFINITY;
                                    mn = fmaxf(mn, sc[u]);
                                }
                                const float corr = __expf(m - mn);
                                float pr[4];
#pragma unroll
                                for (int u = 0; u < 4; ++u) pr[u] = __expf(sc[u] - mn);
                                l = l * corr + ((pr[0] + pr[1]) + (pr[2] + pr[3]));
                                o4.x = o4.x * corr + ((pr[0] * vv[0].x + pr[1] * vv[1].x) + (pr[2] * vv[2].x + pr[3] * vv[3].x));
                                o4.y = o4.y * corr + ((pr[0] * vv[0].y + pr[1] * vv[1].y) + (pr[2] * vv[2].y + pr[3] * vv[3].y));
                                o4.z = o4.z * corr + ((pr[0] * vv[0].z + pr[1] * vv[1].z) + (pr[2] * vv[2].z + pr[3] * vv[3].z));
                                o4.w = o4.w * corr + ((pr[0] * vv[0].w + pr[1] * vv[1].w) + (pr[2] * vv[2].w + pr[3] * vv[3].w));
                                m = mn;
                            }
                        }
                    }
                    if (sub == 0) { att_m[grp] = m; att_l[grp] = l; }
                    *reinterpret_cast<float4 *>(att_o + grp * hd + sub * 4) = o4;
                    fz_bar();
                    if (warp == 0) {
                        // this block's maximum, sum and the groups' weights relative to it (NG <= 64: two groups per lane)
                        const float m0 = lane < NG ? att_m[lane] : -INFINITY, m1 = lane + 32 < NG ? att_m[lane + 32] : -INFINITY;
                        float M = fmaxf(m0, m1);
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
                        const float w0 = m0 == -INFINITY ? 0.f : __expf(m0 - M), w1 = m1 == -INFINITY ? 0.f : __expf(m1 - M);
                        const float Ls = warp_sum((lane < NG ? att_l[lane] * w0 : 0.f) + (lane + 32 < NG ? att_l[lane + 32] * w1 : 0.f));
                        __syncwarp();
                        if (lane < NG) att_m[lane] = w0;
                        if (lane + 32 < NG) att_m[lane + 32] = w1;
                        if (lane < 2) {
                            const float hv = lane == 0 ? M : Ls;
                            my_half[b * (hd + 2) + lane] = hv;
                            if (P.pair) fz_st_remote(peer_pairbuf + (uint32_t)((rank * NB + b) * (hd + 2) + lane) * 4u, hv);
                        }
                    }
                    fz_bar();
                    if (tid < hd) {
                        float O0 = 0.f, O1 = 0.f;
                        for (int g2 = 0; g2 + 1 < NG; g2 += 2) {
                            O0 += att_o[g2 * hd + tid] * att_m[g2];
                            O1 += att_o[(g2 + 1) * hd + tid] * att_m[g2 + 1];
                        }
                        if (NG & 1) O0 += att_o[(NG - 1) * hd + tid] * att_m[NG - 1];
                        my_half[b * (hd + 2) + 2 + tid] = O0 + O1;
                        if (P.pair) fz_st_remote(peer_pairbuf + (uint32_t)((rank * NB + b) * (hd + 2) + 2 + tid) * 4u, O0 + O1);
                    }
                    fz_bar();
                }
                // both halves of the head: merged identically by both blocks (first block's half first)
                if (P.pair) pair_sync();
                fz_bar();
                for (int o = tid; o < nb * hd; o += FZ_CTHREADS) {
                    const int b = o / hd, e = o - b * hd;
                    const float *h0 = pairbuf + (size_t)b * (hd + 2), *h1 = pairbuf + (size_t)(NB + b) * (hd + 2);
                    float val;
                    if (P.pair) {
                        const float M = fmaxf(h0[0], h1[0]);
                        const float a0 = h0[0] == -INFINITY ? 0.f : __expf(h0[0] - M), a1 = h1[0] == -INFINITY ? 0.f : __expf(h1[0] - M);
                        val = (a0 * h0[2 + e] + a1 * h1[2 + e]) / (a0 * h0[1] + a1 * h1[1]);
                    } else {
                        val = h0[2 + e] / h0[1];
                    }
                    uint16_t hi, lo;
                    fz_split(val, hi, lo);
                    ob[(size_t)(2 * b) * P.ob_stride + e] = hi;
                    ob[(size_t)(2 * b + 1) * P.ob_stride + e] = lo;
                }
                fz_bar();
                lap(FZP_ATTN);
            }
            // ---- second part: tile-split over all d_model rows (partial sums), or the output layer's rows
            float best_v = -INFINITY;
            int best_i = 0x7fffffff;
            if (has_work) {
                const bool is_head = ph.kind == FZ_HEAD;
                int my_slot = slots[0];
#pragma unroll
                for (int i = 1; i < NB; ++i) if (q == i) my_slot = slots[i];
                const bool is_a2 = ph.kind == FZ_A;
                const int n_t2 = is_head ? wk.n_tiles : (is_a2 ? wk.row_tiles : d >> 4), row_off = is_a2 ? wk.row_tile0 * 16 : 0;
                const int ks2 = is_head ? ks : (ph.kind == FZ_A ? hd >> 4 : wk.n_tiles);
                const uint16_t *opnd = is_head ? xb : (ph.kind == FZ_A ? ob : hb);
                const int stride = is_head ? P.xb_stride : (ph.kind == FZ_A ? P.ob_stride : P.hb_stride);
                tile_split(is_head ? seg_slot0 : seg_slot1, is_head ? wk.fb0 : wk.fb1, n_t2, ks2, opnd, stride, [&](int tile, const float (&c)[4]) {
                    if (q >= nb) return;
                    const float y0 = c[0] + c[1], y1 = c[2] + c[3];
                    if (!is_head) {
                        // partial sums over this block's columns, as 64-bit fixed point into the team's accumulator
                        fz_red_add(acc_w + (size_t)q * d + row_off + tile * 16 + g, __float2ll_rn(y0 * FZ_FIX_SCALE));
                        fz_red_add(acc_w + (size_t)q * d + row_off + tile * 16 + g + 8, __float2ll_rn(y1 * FZ_FIX_SCALE));
                    } else {
                        const int row = (wk.tile0 + tile) * 16 + g;
                        if (row < P.vocab) {
                            P.logits[(size_t)my_slot * P.vocab + row] = y0;
                            if (y0 > best_v || (y0 == best_v && row < best_i)) { best_v = y0; best_i = row; }
                        }
                        if (row + 8 < P.vocab) {
                            P.logits[(size_t)my_slot * P.vocab + row + 8] = y1;
                            if (y1 > best_v || (y1 == best_v && row + 8 < best_i)) { best_v = y1; best_i = row + 8; }
                        }
                    }
                });
                lap(FZP_MMA2);
            }
            if (ph.kind == FZ_HEAD) {
                // lanes with equal q hold candidates of sample q: reduce over g, then over warps, then over blocks
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    const float vv = __shfl_xor_sync(0xffffffffu, best_v, o);
                    const int ii = __shfl_xor_sync(0xffffffffu, best_i, o);
                    if (vv > best_v || (vv == best_v && ii < best_i)) { best_v = vv; best_i = ii; }
                }
                if (lane < FZ_MAXNB) { hbest_v[warp * FZ_MAXNB + lane] = best_v; hbest_i[warp * FZ_MAXNB + lane] = best_i; }
                fz_bar();
                if (tid < NB) {
                    float bv = hbest_v[tid];
                    int bi = hbest_i[tid];
                    for (int w = 1; w < FZ_CWARPS; ++w) {
                        const float vv = hbest_v[w * FZ_MAXNB + tid];
                        const int ii = hbest_i[w * FZ_MAXNB + tid];
                        if (vv > bv || (vv == bv && ii < bi)) { bv = vv; bi = ii; }
                    }
                    P.head_pv[(size_t)tid * T.n_cta + cta] = bv;
                    P.head_pi[(size_t)tid * T.n_cta + cta] = bi;
                }
            }
            if (pi + 1 < T.n_phases) prefetch_vectors(s_ph[pi + 1], has_work_of(pi + 1));
            team_barrier();
            lap(FZP_BARRIER);
        }
        // every slot of this step's stream has been visited by every warp
        {
            const unsigned n_slots_step = (unsigned)s_seg[n_seg - 1].slots_before + (unsigned)((s_seg[n_seg - 1].n_fb + FZ_SLOT_FB - 1) / FZ_SLOT_FB) +
                                          (unsigned)(n_kvu * kvs_per_unit);
            if (n_slots_step > 0) advance(step_base + n_slots_step - 1u);
            step_base += n_slots_step;
        }

        // ---- end of the step
        if (T.is_last) {
            if (cta == 0) {
                for (int i = warp; i < nb; i += FZ_CWARPS) {
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
                        const int gc = P.gen_count[slot];
                        if (gc < P.log_stride) P.tok_log[(size_t)slot * P.log_stride + gc] = bi;
                        int feed = bi;
                        if (gc < P.n_teacher[slot]) feed = P.teacher[(size_t)slot * P.log_stride + gc];
                        P.cur_tok[slot] = feed;
                        P.gen_count[slot] = gc + 1;
                    }
                }
            }
        } else if (cta == 0) {
            // complete the residual stream with the last phase's sum and hand it to the next partition
            const long long *acc_f = T.acc + (size_t)((phase_ctr + 2u) % 3u) * acc_stride;
            for (int b = 0; b < nb; ++b)
                for (int i = tid; i < d; i += FZ_CTHREADS)
                    T.ring_out[((size_t)j * P.gmax + b) * d + i] =
                        xres[b * d + i] + (T.bias_final[i] + (float)((double)__ldcg(acc_f + (size_t)b * d + i) * (1.0 / 4294967296.0)));
        }
        if (cta == 0) {
            fz_bar();
            if (tid == 0 && P.withhold_partition != p) st_release(T.flag_out + j, r + 1);
        }
        lap(FZP_FIN);
    }
    if (cta == 0)
        for (int s = tid; s < P.n_samples; s += FZ_CTHREADS) T.pos[s] += P.n_pass;
    if (prof_on)
        for (int i = 0; i < PK_PROF_N; ++i)
            if (i != PF_PROD_WAIT && i != PF_PROD_TOTAL) P.prof[(size_t)blockIdx.x * PK_PROF_N + i] = pf[i];
    }
    // no block leaves while its peer may still write into its shared memory
    fz_cluster_sync_all();
}

} // namespace mdi
