// Host side of the recurrent-pipeline decoding library: contexts, weights, the paged key/value
// slot allocator, the partition streams with their activation rings and event handoff, and the
// scheduler that rotates sample groups through the partitions (paper, Section III-C, Algorithms 1-2).
#include "mdi.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <tuple>
#include <vector>

#include "fused_decode.cuh"
#include "persistent_decode.cuh"
#include "prefill_kernels.cuh"
#include "step_kernels.cuh"
#include "tc_decode.cuh"
#include "tc_gemm.cuh"

using namespace mdi;

namespace {

std::string g_create_error;

struct LayerW {
    void *wqkv = nullptr, *wo = nullptr, *w1 = nullptr, *w2 = nullptr, *wgate = nullptr, *wup = nullptr, *wdown = nullptr;
    float *ln1g = nullptr, *ln1b = nullptr, *bqkv = nullptr, *bo = nullptr, *ln2g = nullptr, *ln2b = nullptr,
          *b1 = nullptr, *b2 = nullptr;
};

struct TensorSlot {
    void **mat = nullptr;  // destination pointer for matrices (weight dtype on device)
    float **vec = nullptr; // destination pointer for small vectors (fp32 on device)
    size_t elems = 0;
    int partition = 0;
    bool loaded = false;
};

struct Partition {
    int lo = 0, hi = 0;
    cudaStream_t stream = nullptr;
    // key/value pool
    void *kv_pool = nullptr;
    size_t kv_bytes = 0;
    int n_pages = 0;
    std::vector<int> free_pages;
    std::vector<int> pt_host; // [S][L_p][pages_per_seq], -1 = unmapped (uploaded as 0)
    std::vector<int> pages_of_slot; // count per slot (pages per layer)
    int *pt_dev = nullptr;
    int *pos_dev = nullptr;
    std::vector<int> pos_host;
    // scratch (one step at a time runs on the partition's stream)
    float *x_embed = nullptr, *qbuf = nullptr, *obuf = nullptr, *hbuf = nullptr, *part = nullptr, *x_last = nullptr;
    unsigned *attn_ticket = nullptr;
    // output edge: ring of group slots, and two buffers for first-visit (whole prompt) activations
    float *ring = nullptr;
    float *pf_buf[2] = {nullptr, nullptr};
    std::vector<cudaEvent_t> ev_edge, ev_edge_cap;
    cudaEvent_t ev_pf_out[2] = {nullptr, nullptr}, ev_pf_used[2] = {nullptr, nullptr};
    bool pf_used_valid[2] = {false, false};
    cudaEvent_t ev_join = nullptr, ev_join_cap = nullptr;
    // tensor-core first visit: inputs as bf16 hi/lo planes, fp32 intermediates, for up to PF_CHUNK positions
    uint16_t *pf_hi = nullptr, *pf_lo = nullptr;
    float *pf_qkv = nullptr, *pf_q = nullptr, *pf_o = nullptr, *pf_h = nullptr, *pf_u = nullptr, *pf_xa = nullptr, *pf_xb = nullptr,
          *pf_part = nullptr; // split-K partial sums [PF_SPLIT_MAX][PF_CHUNK][d_model]
    int64_t weight_bytes = 0, buffer_bytes = 0;
};

struct GraphEntry {
    cudaGraphExec_t exec = nullptr;
    int64_t launches = 0, steps = 0;
};

} // namespace

struct mdi_ctx {
    mdi_model_shape s{};
    mdi_options o{};
    int K = 0, S = 0, dev = 0;
    int page_tokens = 16, page_shift = 4, pages_per_seq = 0, n_split = 1, gmax = 1, rounds_per_graph = 16;
    size_t page_elems = 0, esize = 2, kv_esize = 4;
    bool kv_f32 = true;
    int kv_kind = 0; // KV_F32 / KV_BF16 / KV_F16
    std::vector<Partition> part;
    std::vector<LayerW> layer;
    void *wte = nullptr, *wpe = nullptr, *lm_head = nullptr;
    float *lnfg = nullptr, *lnfb = nullptr;
    std::map<std::string, TensorSlot> tensors;
    int n_loaded = 0;
    // tensor-core linear layers: every matrix they multiply by also as contiguous 128 x 64 tiles (row-major pointer -> copy)
    std::map<const void *, void *> w_tiled;
    bool tiles_stale = true;
    float *rope_cos = nullptr, *rope_sin = nullptr;
    // output layers
    float *logits = nullptr; // [S][V]
    float *head_pv = nullptr, *head_y = nullptr; // head_y: [MAXB][vocab] logits of a tensor-core output layer, by item
    int *head_pi = nullptr;
    unsigned *head_ticket = nullptr;
    int head_grid = 0;
    // token state
    int *cur_tok = nullptr, *tok_log = nullptr, *gen_count = nullptr, *teacher = nullptr, *n_teacher = nullptr;
    int *prompt_buf = nullptr; // [S][n_ctx]
    std::vector<int> gen_host, returned_host, prefilled;
    int pf_count = 0;
    cudaStream_t main = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_fork_cap = nullptr, ev_t0 = nullptr, ev_t1 = nullptr, ev_pf0 = nullptr, ev_pf1 = nullptr;
    bool pf_open = false; // ev_pf0 recorded by the first prefill since the last generate
    std::map<std::pair<int, int>, GraphEntry> graphs; // (n_samples, window ticks)
    bool capturing = false;
    int64_t cap_launches = 0, cap_steps = 0;
    // tensor-core first visit
    bool pf_tc = false, pdl = true;
    int tc_min_group = 5; // groups with at least this many samples run their linear layers on the tensor cores
    int *tg_err = nullptr;
    std::map<std::tuple<const void *, uint64_t, uint64_t, uint32_t>, CUtensorMap> tmaps;
    // persistent decode kernel
    bool pk_ok = false, pk_prof_on = false, pk_tables_stale = true;
    float temperature = 0.f; // > 0: sample from the pmf (top_k most likely tokens) instead of taking the argmax
    int top_k = 0;
    unsigned long long sample_seed = 0;
    int withhold_once = -1; // partition whose output flags the next persistent launch withholds (time-out test hook)
    int pk_slots = 0, pk_xs_floats = 0, pk_nb = 1, n_sm = 0, scheduler = 0;
    size_t pk_smem = 0;
    std::vector<PkTeam> pk_teams_host;
    std::vector<PkPhase> pk_phases_host;
    std::vector<int> pk_phase_begin, pk_phase_count;
    PkTeam *pk_teams = nullptr;
    PkPhase *pk_phases = nullptr;
    unsigned *pk_sync = nullptr; // [K][64]: word 0 team barrier, words 32.. output-edge flags
    int *pk_err = nullptr;
    unsigned long long *pk_prof = nullptr; // [n_sm][PK_PROF_N]
    // fused-phase persistent kernel (GPT block, bf16 weights): plan made at creation, weight stream built at first use
    bool fz_ok = false, fz_stale = true, fz_prof_on = false;
    int fz_slots = 0, fz_nb = 1, fz_xb_stride = 0, fz_hb_stride = 0, fz_ob_stride = 0, fz_part_floats = 0, fz_grid = 0;
    int last_kernel = 0; // which persistent kernel the last generate call used: 1 phase-per-matrix, 2 fused-phase
    size_t fz_smem = 0;
    std::vector<FzTeam> fz_teams_host;
    std::vector<FzWork> fz_works_host;
    std::vector<FzBlock> fz_blocks_host;
    std::vector<int> fz_units_host, fz_phase_begin, fz_phase_count;
    std::vector<std::vector<int>> fz_unit_lists; // hidden units of (block, phase B), indexed like fz_works_host
    FzTeam *fz_teams = nullptr;
    FzPhase *fz_phases = nullptr;
    FzWork *fz_works = nullptr;
    FzBlock *fz_blocks = nullptr;
    FzSeg *fz_segs = nullptr;
    int *fz_units = nullptr, *fz_err = nullptr;
    int fz_kv_pps = 1, fz_pair = 0, fz_kv_rows = 16;
    uint4 *fz_stream = nullptr;
    long long *fz_acc = nullptr;
    unsigned *fz_sync = nullptr;
    unsigned long long *fz_prof = nullptr, *fz_trace = nullptr;
    int fz_trace_blocks = 0;
    int64_t fz_stream_bytes = 0;
    std::vector<int64_t> fz_team_stream_bytes; // per partition: bytes of its blocks' weight streams
    // persistent tensor-core decode kernel (bf16 weights, groups of up to 8 samples): plan at creation, tables at first use
    bool td_ok = false, td_stale = true;
    int td_grid = 0, td_b_kb = 16;
    size_t td_smem = 0;
    std::vector<TdTeam> td_teams_host;
    std::vector<TdPhase> td_phases_host;
    std::vector<int> td_phase_begin, td_phase_count;
    TdTeam *td_teams = nullptr;
    TdPhase *td_phases = nullptr;
    CUtensorMap *td_maps = nullptr;
    float *td_buf = nullptr;       // all float scratch of the kernel (residual copies, partial and finished sums), one allocation
    int *td_ints = nullptr;        // tickets and argmax candidates
    size_t td_n_ints = 0;
    unsigned *td_sync = nullptr;
    int *td_err = nullptr;
    unsigned long long *td_prof = nullptr;
    int64_t td_buf_bytes = 0;
    mdi_stats st{};
    std::string err;
};

namespace {

int fail(mdi_ctx *c, int code, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (c) c->err = buf; else g_create_error = buf;
    return code;
}

#define CU(call)                                                                                             \
    do {                                                                                                     \
        cudaError_t e_ = (call);                                                                             \
        if (e_ != cudaSuccess)                                                                               \
            return fail(c, e_ == cudaErrorMemoryAllocation ? MDI_ERR_OOM : MDI_ERR_CUDA, "%s: %s", #call,     \
                        cudaGetErrorString(e_));                                                             \
    } while (0)

template <typename T> int dalloc(mdi_ctx *c, T **p, size_t n, int64_t *account = nullptr) {
    size_t bytes = std::max<size_t>(n, 1) * sizeof(T);
    CU(cudaMalloc((void **)p, bytes));
    CU(cudaMemset(*p, 0, bytes));
    if (account) *account += (int64_t)bytes;
    return MDI_OK;
}

inline void count_launch(mdi_ctx *c) {
    if (c->capturing) ++c->cap_launches; else ++c->st.kernel_launches;
}

// Launch with the programmatic-serialization attribute when pdl is set (the kernels of the tensor-core chain
// call griddepcontrol.wait before touching their predecessor's results), else as a plain launch.
template <typename... KArgs, typename... Args>
void launch_k(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- kernel dispatch ------------------------------------------------------------------------------
constexpr size_t LIN_SMEM_MAX = 200 * 1024;

// Element type of the key/value cache: fp32 (always with fp32 weights), or with bf16 weights a 2-byte type on request.
enum { KV_F32 = 0, KV_BF16 = 1, KV_F16 = 2 };
// Runs `call` with KT bound to the cache's element type.
#define KV_DISPATCH(kind, call)                                          \
    do {                                                                 \
        if ((kind) == KV_F32) { using KT = float; call; }                \
        else if ((kind) == KV_F16) { using KT = __half; call; }          \
        else { using KT = __nv_bfloat16; call; }                         \
    } while (0)
template <int NB, typename WT, int MODE> void lin_launch(const LinArgs &a, const Batch &bt, int grid, size_t smem, cudaStream_t st, int kv_kind) {
    if (MODE == LIN_QKV && kv_kind == KV_F32) k_linear<NB, WT, MODE, float><<<grid, LIN_THREADS, smem, st>>>(a, bt);
    else if (MODE == LIN_QKV && kv_kind == KV_F16) k_linear<NB, WT, MODE, __half><<<grid, LIN_THREADS, smem, st>>>(a, bt);
    else k_linear<NB, WT, MODE><<<grid, LIN_THREADS, smem, st>>>(a, bt);
}
template <int NB, typename WT, int MODE> cudaError_t lin_attr() {
    cudaError_t e = cudaFuncSetAttribute(k_linear<NB, WT, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LIN_SMEM_MAX);
    if (e == cudaSuccess && MODE == LIN_QKV)
        e = cudaFuncSetAttribute(k_linear<NB, WT, MODE, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LIN_SMEM_MAX);
    if (e == cudaSuccess && MODE == LIN_QKV)
        e = cudaFuncSetAttribute(k_linear<NB, WT, MODE, __half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LIN_SMEM_MAX);
    return e;
}
template <typename WT, int MODE> void lin_nb(int nb, const LinArgs &a, const Batch &bt, int grid, size_t smem, cudaStream_t st, int kv_kind) {
    switch (nb) {
        case 1: lin_launch<1, WT, MODE>(a, bt, grid, smem, st, kv_kind); break;
        case 2: lin_launch<2, WT, MODE>(a, bt, grid, smem, st, kv_kind); break;
        case 4: lin_launch<4, WT, MODE>(a, bt, grid, smem, st, kv_kind); break;
        default: lin_launch<8, WT, MODE>(a, bt, grid, smem, st, kv_kind); break;
    }
}
template <typename WT> void lin_mode(int mode, int nb, const LinArgs &a, const Batch &bt, int grid, size_t smem, cudaStream_t st, int kv_kind) {
    switch (mode) {
        case LIN_QKV: lin_nb<WT, LIN_QKV>(nb, a, bt, grid, smem, st, kv_kind); break;
        case LIN_ACT: lin_nb<WT, LIN_ACT>(nb, a, bt, grid, smem, st, kv_kind); break;
        case LIN_GATEUP: lin_nb<WT, LIN_GATEUP>(nb, a, bt, grid, smem, st, kv_kind); break;
        case LIN_HEAD: lin_nb<WT, LIN_HEAD>(nb, a, bt, grid, smem, st, kv_kind); break;
        default: lin_nb<WT, LIN_RESID>(nb, a, bt, grid, smem, st, kv_kind); break;
    }
}
template <typename WT, int MODE> cudaError_t lin_attr_nb() {
    cudaError_t e;
    if ((e = lin_attr<1, WT, MODE>()) != cudaSuccess) return e;
    if ((e = lin_attr<2, WT, MODE>()) != cudaSuccess) return e;
    if ((e = lin_attr<4, WT, MODE>()) != cudaSuccess) return e;
    return lin_attr<8, WT, MODE>();
}
template <typename WT> cudaError_t lin_attr_all() {
    cudaError_t e;
    if ((e = lin_attr_nb<WT, LIN_QKV>()) != cudaSuccess) return e;
    if ((e = lin_attr_nb<WT, LIN_ACT>()) != cudaSuccess) return e;
    if ((e = lin_attr_nb<WT, LIN_GATEUP>()) != cudaSuccess) return e;
    if ((e = lin_attr_nb<WT, LIN_HEAD>()) != cudaSuccess) return e;
    return lin_attr_nb<WT, LIN_RESID>();
}

inline int round_nb(int n) { return n <= 1 ? 1 : n <= 2 ? 2 : n <= 4 ? 4 : 8; }

Batch slice(const Batch &bt, int first, int n) {
    Batch r{};
    r.n = n;
    for (int i = 0; i < n; ++i) { r.slot[i] = bt.slot[first + i]; r.off[i] = bt.off[first + i]; r.adv[i] = bt.adv[first + i]; }
    return r;
}

// One linear layer over a batch; splits the batch when its inputs would not fit in shared memory.
int linear(mdi_ctx *c, int mode, LinArgs a, const Batch &bt, cudaStream_t st) {
    const bool f32 = c->s.weight_dtype == MDI_DTYPE_F32;
    int maxb = (int)(LIN_SMEM_MAX / ((size_t)a.in_dim * 4));
    maxb = maxb >= 8 ? 8 : maxb >= 4 ? 4 : maxb >= 2 ? 2 : 1;
    if ((size_t)a.in_dim * 4 > LIN_SMEM_MAX) return fail(c, MDI_ERR_SHAPE, "input width %d too large", a.in_dim);
    const int units = mode == LIN_GATEUP ? a.n_rows : (a.n_rows + 1) / 2;
    const int grid = (units + LIN_WARPS - 1) / LIN_WARPS;
    if (mode == LIN_HEAD && bt.n > maxb) return fail(c, MDI_ERR_SHAPE, "output layer batch does not fit");
    for (int first = 0; first < bt.n; first += maxb) {
        const int n = std::min(maxb, bt.n - first);
        const int nb = round_nb(n);
        Batch sb = slice(bt, first, n);
        LinArgs b = a;
        b.x_in = a.x_in + (size_t)first * a.in_dim;
        if (a.q_out) b.q_out = a.q_out + (size_t)first * a.q_rows;
        if (a.h_out) b.h_out = a.h_out + (size_t)first * a.n_rows;
        if (a.x_res) b.x_res = a.x_res + (size_t)first * a.n_rows;
        if (a.x_out) b.x_out = a.x_out + (size_t)first * a.n_rows;
        const size_t smem = (size_t)nb * a.in_dim * 4;
        if (f32) lin_mode<float>(mode, nb, b, sb, grid, smem, st, KV_F32);
        else lin_mode<__nv_bfloat16>(mode, nb, b, sb, grid, smem, st, c->kv_kind);
        count_launch(c);
    }
    return MDI_OK;
}

template <typename KT> void attn_hd(bool pdl, int hd, const AttnArgs &a, const Batch &bt, dim3 grid, cudaStream_t st) {
    switch (hd) {
        case 16: launch_k(pdl, k_attn_decode<KT, 16>, grid, dim3(ATT_THREADS), 0, st, a, bt); break;
        case 32: launch_k(pdl, k_attn_decode<KT, 32>, grid, dim3(ATT_THREADS), 0, st, a, bt); break;
        case 64: launch_k(pdl, k_attn_decode<KT, 64>, grid, dim3(ATT_THREADS), 0, st, a, bt); break;
        default: launch_k(pdl, k_attn_decode<KT, 128>, grid, dim3(ATT_THREADS), 0, st, a, bt); break;
    }
}

KvView kv_view(const mdi_ctx *c, const Partition &P) {
    KvView v{};
    v.pool = P.kv_pool;
    v.page_table = P.pt_dev;
    v.n_layers_local = P.hi - P.lo;
    v.pages_per_seq = c->pages_per_seq;
    v.page_tokens = c->page_tokens;
    v.page_shift = c->page_shift;
    v.n_kv_head = c->s.n_kv_head;
    v.head_dim = c->s.head_dim;
    v.page_elems = c->page_elems;
    return v;
}

struct HeadReq {
    int item = -1;          // item of the batch whose activation goes through the output layers (-1: all items)
    bool update_state = true; // advance gen_count / cur_tok / tok_log
    int *tok_out = nullptr;
};

// Output layers for the items of hb (final norm, vocabulary projection, greedy argmax); x_rows: [hb.n][d].
int enqueue_head(mdi_ctx *c, const Batch &hb, const float *x_rows, const HeadReq &head, cudaStream_t st) {
    const mdi_model_shape &s = c->s;
    LinArgs a{};
    a.W = s.tied_lm_head ? c->wte : c->lm_head; a.n_rows = s.vocab; a.in_dim = s.d_model;
    a.x_in = x_rows;
    a.norm = s.arch == MDI_ARCH_GPT ? NORM_LAYER : NORM_RMS; a.gamma = c->lnfg; a.beta = c->lnfb; a.eps = s.norm_eps;
    a.logits = c->logits; a.part_val = c->head_pv; a.part_idx = c->head_pi; a.ticket = c->head_ticket;
    a.tok_out = head.tok_out; a.log_stride = s.n_ctx;
    if (head.update_state) {
        a.cur_tok = c->cur_tok; a.tok_log = c->tok_log; a.gen_count = c->gen_count;
        a.teacher = c->teacher; a.n_teacher = c->n_teacher;
        a.temperature = c->temperature; a.top_k = c->top_k; a.sample_seed = c->sample_seed;
    }
    return linear(c, LIN_HEAD, a, hb, st);
}

int tc_partition_step(mdi_ctx *c, int p, const Batch &bt, const float *x_in, float *x_out, cudaStream_t st);
int tc_head(mdi_ctx *c, const Batch &hb, const float *x_rows, const HeadReq &head, cudaStream_t st);

// All kernels of one visit of a batch of items to partition p.
//   x_in:  [n][d] input activations (ignored for p == 0, which embeds tokens from tok_src)
//   x_out: [n][d] where the partition's output activations are written
int enqueue_partition_step(mdi_ctx *c, int p, const Batch &bt, const float *x_in, const int *tok_src, int tok_by_slot,
                           float *x_out, const HeadReq *head, cudaStream_t st) {
    Partition &P = c->part[p];
    const mdi_model_shape &s = c->s;
    const bool f32 = s.weight_dtype == MDI_DTYPE_F32;
    const int d = s.d_model, qw = s.n_head * s.head_dim, kw = s.n_kv_head * s.head_dim;
    const int norm = s.arch == MDI_ARCH_GPT ? NORM_LAYER : NORM_RMS;
    if (p == 0) {
        dim3 g((d + 255) / 256, bt.n);
        if (f32) k_embed<float><<<g, 256, 0, st>>>((const float *)c->wte, (const float *)c->wpe, d, s.vocab, tok_src, tok_by_slot, P.pos_dev, bt, P.x_embed);
        else k_embed<__nv_bfloat16><<<g, 256, 0, st>>>((const __nv_bfloat16 *)c->wte, (const __nv_bfloat16 *)c->wpe, d, s.vocab, tok_src, tok_by_slot, P.pos_dev, bt, P.x_embed);
        count_launch(c);
        x_in = P.x_embed;
    }
    const KvView kv = kv_view(c, P);
    // groups of more than 4 items with bf16 weights: the linear layers run on the tensor cores
    const bool tc = c->pf_tc && bt.n >= c->tc_min_group;
    if (tc) {
        const int rc = tc_partition_step(c, p, bt, x_in, x_out, st);
        if (rc != MDI_OK) return rc;
    }
    for (int l = P.lo; l < P.hi && !tc; ++l) {
        const LayerW &L = c->layer[l];
        const float *xin_l = l == P.lo ? x_in : x_out;
        int rc;
        {   // norm 1 + QKV projection (+ rotary) + cache append
            LinArgs a{};
            a.W = L.wqkv; a.bias = L.bqkv; a.n_rows = qw + 2 * kw; a.in_dim = d;
            a.x_in = xin_l; a.norm = norm; a.gamma = L.ln1g; a.beta = L.ln1b; a.eps = s.norm_eps;
            a.q_out = P.qbuf; a.q_rows = qw; a.kv_rows = kw; a.rope = s.arch == MDI_ARCH_LLAMA;
            a.rope_cos = c->rope_cos; a.rope_sin = c->rope_sin; a.kv = kv; a.layer_local = l - P.lo; a.pos = P.pos_dev;
            if ((rc = linear(c, LIN_QKV, a, bt, st)) != MDI_OK) return rc;
        }
        {   // attention over the slot's cache
            AttnArgs a{};
            a.q = P.qbuf; a.o = P.obuf; a.part = P.part; a.ticket = P.attn_ticket; a.kv = kv;
            a.layer_local = l - P.lo; a.n_head = s.n_head; a.n_split = c->n_split; a.pos = P.pos_dev;
            a.scale = 1.0f / std::sqrt((float)s.head_dim);
            dim3 g(s.n_head, c->n_split, bt.n);
            KV_DISPATCH(c->kv_kind, attn_hd<KT>(false, s.head_dim, a, bt, g, st));
            count_launch(c);
        }
        {   // output projection + residual
            LinArgs a{};
            a.W = L.wo; a.bias = L.bo; a.n_rows = d; a.in_dim = qw; a.x_in = P.obuf; a.norm = NORM_NONE;
            a.x_res = xin_l; a.x_out = x_out;
            if ((rc = linear(c, LIN_RESID, a, bt, st)) != MDI_OK) return rc;
        }
        if (s.act == MDI_ACT_SWIGLU) {
            LinArgs a{};
            a.W = L.wgate; a.W2 = L.wup; a.n_rows = s.d_ff; a.in_dim = d; a.x_in = x_out; a.norm = norm;
            a.gamma = L.ln2g; a.beta = L.ln2b; a.eps = s.norm_eps; a.h_out = P.hbuf;
            if ((rc = linear(c, LIN_GATEUP, a, bt, st)) != MDI_OK) return rc;
        } else {
            LinArgs a{};
            a.W = L.w1; a.bias = L.b1; a.n_rows = s.d_ff; a.in_dim = d; a.x_in = x_out; a.norm = norm;
            a.gamma = L.ln2g; a.beta = L.ln2b; a.eps = s.norm_eps; a.h_out = P.hbuf; a.act = s.act == MDI_ACT_GELU_ERF;
            if ((rc = linear(c, LIN_ACT, a, bt, st)) != MDI_OK) return rc;
        }
        {   // second MLP matrix + residual; the last block also advances the slots' positions
            LinArgs a{};
            a.W = s.act == MDI_ACT_SWIGLU ? L.wdown : L.w2; a.bias = L.b2; a.n_rows = d; a.in_dim = s.d_ff;
            a.x_in = P.hbuf; a.norm = NORM_NONE; a.x_res = x_out; a.x_out = x_out;
            a.pos_adv = l == P.hi - 1 ? P.pos_dev : nullptr;
            if ((rc = linear(c, LIN_RESID, a, bt, st)) != MDI_OK) return rc;
        }
    }
    if (head && p == c->K - 1) {
        const Batch hb = head->item < 0 ? bt : slice(bt, head->item, 1);
        const float *xh = head->item < 0 ? x_out : x_out + (size_t)head->item * d;
        const int rc = (tc && c->head_y) ? tc_head(c, hb, xh, *head, st) : enqueue_head(c, hb, xh, *head, st);
        if (rc != MDI_OK) return rc;
    }
    if (c->capturing) ++c->cap_steps; else ++c->st.stage_steps;
    return MDI_OK;
}


// ---- first visit on tensor cores (bf16 weights): GEMMs of tc_gemm.cuh + helpers of prefill_kernels.cuh ----
constexpr int PF_CHUNK = 128; // positions per pass through a partition (one tile of positions per GEMM block)
constexpr int PF_SPLIT_MAX = 8; // K splits of the GEMMs with few row tiles (output projection, MLP down)

int pf_setup(mdi_ctx *c) {
    const mdi_model_shape &s = c->s;
    c->pf_tc = s.weight_dtype == MDI_DTYPE_BF16 && c->o.prefill_mode != 1;
    // Which decode steps use the tensor-core linear layers (stream scheduler): by default groups of 5 or more
    // samples, and every group when one block's matrices are 48 MB or more (then a step moves enough bytes per
    // kernel for launches not to matter, and TMA-fed GEMM tiles stream faster than the CUDA-core tiles).
    {
        const int d = s.d_model, qw = s.n_head * s.head_dim, kw = s.n_kv_head * s.head_dim;
        const double layer_bytes = 2.0 * ((double)(qw + 2 * kw) * d + (double)d * qw + (double)(s.act == MDI_ACT_SWIGLU ? 3 : 2) * s.d_ff * d);
        c->tc_min_group = c->o.tc_min_group > 0 ? c->o.tc_min_group : (layer_bytes >= 48e6 ? 1 : 5);
    }
    if (!c->pf_tc) return MDI_OK;
    CU(cudaFuncSetAttribute(k_tc_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TG_SMEM));
    const int d = s.d_model, F = s.d_ff, qw = s.n_head * s.head_dim, kw = s.n_kv_head * s.head_dim;
    const size_t maxk = (size_t)std::max(std::max(d, F), qw);
    int rc;
    if ((rc = dalloc(c, &c->tg_err, 1)) != MDI_OK) return rc;
    for (auto &P : c->part) {
        if ((rc = dalloc(c, &P.pf_hi, PF_CHUNK * maxk, &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_lo, PF_CHUNK * maxk, &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_qkv, (size_t)PF_CHUNK * (qw + 2 * kw), &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_q, (size_t)PF_CHUNK * qw, &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_o, (size_t)PF_CHUNK * qw, &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_h, (size_t)PF_CHUNK * F, &P.buffer_bytes)) != MDI_OK) return rc;
        if (s.act == MDI_ACT_SWIGLU && (rc = dalloc(c, &P.pf_u, (size_t)PF_CHUNK * F, &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_xa, (size_t)PF_CHUNK * d, &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_xb, (size_t)PF_CHUNK * d, &P.buffer_bytes)) != MDI_OK) return rc;
        if ((rc = dalloc(c, &P.pf_part, (size_t)PF_SPLIT_MAX * PF_CHUNK * d, &P.buffer_bytes)) != MDI_OK) return rc;
    }
    return MDI_OK;
}

// Tensor maps are cached by (base address, rows, columns, box rows): weights never move, scratch neither.
int pf_map(mdi_ctx *c, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, const CUtensorMap **out) {
    auto key = std::make_tuple(base, rows, cols, box_rows);
    auto it = c->tmaps.find(key);
    if (it == c->tmaps.end()) {
        CUtensorMap m;
        const CUresult r = tg_make_map(&m, base, rows, cols, box_rows);
        if (r != CUDA_SUCCESS) return fail(c, MDI_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) for a %llu x %llu matrix", (int)r,
                                           (unsigned long long)rows, (unsigned long long)cols);
        it = c->tmaps.emplace(key, m).first;
    }
    *out = &it->second;
    return MDI_OK;
}

// A split-K GEMM leaves partial sums behind; they are added up (with bias and residual) by the next norm kernel.
struct PfPending {
    int splits = 0;
    const float *bias = nullptr, *resid = nullptr;
};

// y[t][r] = act(W[r][:] . x[t][:] + bias[r] + resid[t][r]) for T positions whose inputs sit in P.pf_hi / P.pf_lo.
// y may be null when only the bf16 planes out_hi / out_lo are wanted.  When the matrix has few 128-row tiles the
// reduction is split over several blocks: then nothing is written but P.pf_part, and *pending says what is left
// to add (pending must be non-null for matrices with d_model rows).
int pf_gemm(mdi_ctx *c, Partition &P, const void *W, int n_rows, int K, int T, const float *bias, const float *resid, int act,
            float *y, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, PfPending *pending, cudaStream_t st) {
    const int n_tile = T <= TG_NT_PACKED ? TG_NT_PACKED : T <= 16 ? 16 : T <= 32 ? 32 : T <= 64 ? 64 : 128;
    const CUtensorMap *mw, *mhi, *mlo;
    int rc;
    const int grid_x = (n_rows + TG_BM - 1) / TG_BM, n_kb = (K + TG_BK - 1) / TG_BK;
    const auto tiled = c->w_tiled.find(W);
    if (tiled != c->w_tiled.end()) rc = pf_map(c, tiled->second, (uint64_t)grid_x * n_kb * TG_BM, (uint64_t)TG_BK, TG_BM, &mw);
    else rc = pf_map(c, W, (uint64_t)n_rows, (uint64_t)K, TG_BM, &mw);
    if (rc != MDI_OK) return rc;
    if ((rc = pf_map(c, P.pf_hi, PF_CHUNK, (uint64_t)K, (uint32_t)n_tile, &mhi)) != MDI_OK) return rc;
    if ((rc = pf_map(c, P.pf_lo, PF_CHUNK, (uint64_t)K, (uint32_t)n_tile, &mlo)) != MDI_OK) return rc;
    int splits = 1;
    if (pending && 2 * grid_x <= c->n_sm) splits = std::max(1, std::min(std::min(PF_SPLIT_MAX, c->n_sm / grid_x), n_kb / 8));
    TgArgs a{};
    a.n_rows = n_rows; a.K = K; a.T = T; a.n_tile = n_tile; a.bias = bias; a.resid = resid; a.act = act; a.y = y; a.ldy = n_rows;
    a.err = c->tg_err; a.w_tiled = tiled != c->w_tiled.end(); a.partial = P.pf_part; a.out_hi = out_hi; a.out_lo = out_lo;
    launch_k(c->pdl, k_tc_gemm, dim3(grid_x, (T + n_tile - 1) / n_tile, splits), dim3(TG_THREADS), tg_smem_bytes(n_tile), st, *mw, *mhi, *mlo, a);
    count_launch(c);
    if (pending) {
        pending->splits = splits > 1 ? splits : 0;
        pending->bias = bias;
        pending->resid = resid;
    }
    return MDI_OK;
}

template <typename KT> void pf_attn_hd(bool pdl, int hd, dim3 g, cudaStream_t st, const float *q, __nv_bfloat16 *ohi, __nv_bfloat16 *olo,
                                       const KvView &kv, int ll, int n_head, const int *pos, int slot, float scale) {
    switch (hd) {
        case 16: launch_k(pdl, k_pf_attn<KT, 16>, g, dim3(ATT_THREADS), 0, st, q, ohi, olo, kv, ll, n_head, pos, slot, scale); break;
        case 32: launch_k(pdl, k_pf_attn<KT, 32>, g, dim3(ATT_THREADS), 0, st, q, ohi, olo, kv, ll, n_head, pos, slot, scale); break;
        case 64: launch_k(pdl, k_pf_attn<KT, 64>, g, dim3(ATT_THREADS), 0, st, q, ohi, olo, kv, ll, n_head, pos, slot, scale); break;
        default: launch_k(pdl, k_pf_attn<KT, 128>, g, dim3(ATT_THREADS), 0, st, q, ohi, olo, kv, ll, n_head, pos, slot, scale); break;
    }
}

// The blocks of partition p on T rows with the linear layers on the tensor cores.  Two uses:
//  - first visit (bt == null): T (<= PF_CHUNK) consecutive new positions of `slot`; partition 0 embeds tok_dev[0..T);
//  - a group's decode step (bt != null): T = bt->n items of different slots, one new position each.
// x_in: [T][d] (ignored for partition 0 of a first visit); x_out: [T][d].  Cache rows are appended and the
// positions advanced at the end.  Per block: norm+split, QKV GEMM, rotary+append, attention (writes bf16 planes),
// output-projection GEMM, norm+split (adds up split-K partials), MLP up GEMM (writes bf16 planes), MLP down GEMM.
int tc_layers(mdi_ctx *c, int p, const Batch *bt, int slot, const int *tok_dev, int T, const float *x_in, float *x_out, cudaStream_t st) {
    Partition &P = c->part[p];
    const mdi_model_shape &s = c->s;
    const int d = s.d_model, F = s.d_ff, qw = s.n_head * s.head_dim, kw = s.n_kv_head * s.head_dim;
    const int norm = s.arch == MDI_ARCH_GPT ? NORM_LAYER : NORM_RMS, rope = s.arch == MDI_ARCH_LLAMA;
    const KvView kv = kv_view(c, P);
    const float scale = 1.0f / std::sqrt((float)s.head_dim);
    __nv_bfloat16 *hi = (__nv_bfloat16 *)P.pf_hi, *lo = (__nv_bfloat16 *)P.pf_lo;
    int rc;
    const bool pdl = c->pdl;
    // element-wise helpers: few rows (a decode step) are cut into column slices so that their grids are not a handful of blocks
    const int ysl = std::max(1, std::min(16, 2 * c->n_sm / std::max(T, 1) / 4));
    if (!bt && p == 0) {
        launch_k(pdl, k_pf_embed<__nv_bfloat16>, dim3(T), dim3(256), 0, st, (const __nv_bfloat16 *)c->wte, (const __nv_bfloat16 *)c->wpe, d, s.vocab, tok_dev,
                                                    P.pos_dev, slot, P.pf_xa);
        count_launch(c);
        x_in = P.pf_xa;
    }
    PfPending pend; // partial sums of the previous block's MLP-down GEMM, not yet added into x_out
    for (int l = P.lo; l < P.hi; ++l) {
        const LayerW &L = c->layer[l];
        const int ll = l - P.lo;
        const float *xin_l = l == P.lo ? x_in : x_out;
        // norm 1 (first completing the residual stream if the previous GEMM was split)
        launch_k(pdl, k_pf_norm_split, dim3(T), dim3(PF_THREADS), 0, st, pend.splits ? pend.resid : xin_l, d, norm, L.ln1g, L.ln1b, s.norm_eps, hi, lo, P.pf_part,
                                                  pend.splits, T, pend.bias, x_out);
        count_launch(c);
        pend = PfPending();
        if ((rc = pf_gemm(c, P, L.wqkv, qw + 2 * kw, d, T, L.bqkv, nullptr, TG_NONE, P.pf_qkv, nullptr, nullptr, nullptr, st)) != MDI_OK) return rc;
        if (bt) {
            KV_DISPATCH(c->kv_kind, launch_k(pdl, k_bt_rope_append<KT>, dim3(T, ysl), dim3(256), 0, st, P.pf_qkv, qw, kw, s.head_dim, rope, c->rope_cos, c->rope_sin, kv, ll, P.pos_dev, *bt, P.qbuf));
            count_launch(c);
            AttnArgs a{};
            a.q = P.qbuf; a.o = P.obuf; a.part = P.part; a.ticket = P.attn_ticket; a.kv = kv; a.layer_local = ll; a.n_head = s.n_head;
            a.n_split = c->n_split; a.pos = P.pos_dev; a.scale = scale; a.o_hi = hi; a.o_lo = lo;
            const dim3 g(s.n_head, c->n_split, T);
            KV_DISPATCH(c->kv_kind, attn_hd<KT>(pdl, s.head_dim, a, *bt, g, st));
            count_launch(c);
        } else {
            KV_DISPATCH(c->kv_kind, launch_k(pdl, k_pf_rope_append<KT>, dim3(T), dim3(256), 0, st, P.pf_qkv, qw, kw, s.head_dim, rope, c->rope_cos, c->rope_sin, kv, ll, P.pos_dev, slot, P.pf_q));
            count_launch(c);
            KV_DISPATCH(c->kv_kind, pf_attn_hd<KT>(pdl, s.head_dim, dim3(s.n_head, T), st, P.pf_q, hi, lo, kv, ll, s.n_head, P.pos_dev, slot, scale));
            count_launch(c);
        }
        // output projection + residual -> x_out (or partial sums, completed by the next kernel)
        PfPending po;
        if ((rc = pf_gemm(c, P, L.wo, d, qw, T, L.bo, xin_l, TG_NONE, x_out, nullptr, nullptr, &po, st)) != MDI_OK) return rc;
        launch_k(pdl, k_pf_norm_split, dim3(T), dim3(PF_THREADS), 0, st, po.splits ? po.resid : x_out, d, norm, L.ln2g, L.ln2b, s.norm_eps, hi, lo, P.pf_part, po.splits, T,
                                                  po.bias, x_out);
        count_launch(c);
        if (s.act == MDI_ACT_SWIGLU) {
            if ((rc = pf_gemm(c, P, L.wgate, F, d, T, nullptr, nullptr, TG_NONE, P.pf_h, nullptr, nullptr, nullptr, st)) != MDI_OK) return rc;
            if ((rc = pf_gemm(c, P, L.wup, F, d, T, nullptr, nullptr, TG_NONE, P.pf_u, nullptr, nullptr, nullptr, st)) != MDI_OK) return rc;
            launch_k(pdl, k_pf_swiglu_split, dim3(T, ysl), dim3(256), 0, st, P.pf_h, P.pf_u, F, hi, lo);
            count_launch(c);
            if ((rc = pf_gemm(c, P, L.wdown, d, F, T, nullptr, x_out, TG_NONE, x_out, nullptr, nullptr, &pend, st)) != MDI_OK) return rc;
        } else {
            // the GEMM cannot write the planes it is still reading as its input: they go to the other half of the buffers
            if ((rc = pf_gemm(c, P, L.w1, F, d, T, L.b1, nullptr, s.act == MDI_ACT_GELU_ERF ? TG_GELU_ERF : TG_GELU_TANH, P.pf_h, nullptr, nullptr,
                              nullptr, st)) != MDI_OK)
                return rc;
            launch_k(pdl, k_pf_norm_split, dim3(T, ysl), dim3(PF_THREADS), 0, st, P.pf_h, F, NORM_NONE, nullptr, nullptr, 0.f, hi, lo, nullptr, 0, T, nullptr, nullptr);
            count_launch(c);
            if ((rc = pf_gemm(c, P, L.w2, d, F, T, L.b2, x_out, TG_NONE, x_out, nullptr, nullptr, &pend, st)) != MDI_OK) return rc;
        }
    }
    if (pend.splits) { // complete the residual stream after the last block
        launch_k(pdl, k_pf_norm_split, dim3(T), dim3(PF_THREADS), 0, st, pend.resid, d, NORM_NONE, nullptr, nullptr, 0.f, nullptr, nullptr, P.pf_part, pend.splits, T,
                                                  pend.bias, x_out);
        count_launch(c);
    }
    if (bt) launch_k(pdl, k_bt_advance, dim3(1), dim3(32), 0, st, P.pos_dev, *bt);
    else launch_k(pdl, k_pf_advance, dim3(1), dim3(32), 0, st, P.pos_dev, slot, T);
    count_launch(c);
    return MDI_OK;
}

// Output layers of a tensor-core decode step: final norm + hi/lo split, the vocabulary projection as one more GEMM
// (logits of the hb.n items into head_y), then token choice from those logits.
int tc_head(mdi_ctx *c, const Batch &hb, const float *x_rows, const HeadReq &head, cudaStream_t st) {
    const mdi_model_shape &s = c->s;
    Partition &P = c->part[c->K - 1];
    const int d = s.d_model, V = s.vocab, T = hb.n;
    const bool pdl = c->pdl;
    __nv_bfloat16 *hi = (__nv_bfloat16 *)P.pf_hi, *lo = (__nv_bfloat16 *)P.pf_lo;
    launch_k(pdl, k_pf_norm_split, dim3(T), dim3(PF_THREADS), 0, st, x_rows, d, s.arch == MDI_ARCH_GPT ? NORM_LAYER : NORM_RMS, c->lnfg, c->lnfb,
             s.norm_eps, hi, lo, (const float *)nullptr, 0, T, (const float *)nullptr, (float *)nullptr);
    count_launch(c);
    int rc = pf_gemm(c, P, s.tied_lm_head ? c->wte : c->lm_head, V, d, T, nullptr, nullptr, TG_NONE, c->head_y, nullptr, nullptr, nullptr, st);
    if (rc != MDI_OK) return rc;
    LinArgs a{};
    a.n_rows = V; a.in_dim = d;
    a.logits = c->logits; a.part_val = c->head_pv; a.part_idx = c->head_pi; a.ticket = c->head_ticket;
    a.tok_out = head.tok_out; a.log_stride = s.n_ctx;
    if (head.update_state) {
        a.cur_tok = c->cur_tok; a.tok_log = c->tok_log; a.gen_count = c->gen_count;
        a.teacher = c->teacher; a.n_teacher = c->n_teacher;
        a.temperature = c->temperature; a.top_k = c->top_k; a.sample_seed = c->sample_seed;
    }
    launch_k(pdl, k_head_pick, dim3(std::min(1024, std::max(1, (V + 2047) / 2048 * 4))), dim3(LIN_THREADS), 0, st, a, hb, (const float *)c->head_y);
    count_launch(c);
    return MDI_OK;
}

int pf_partition_chunk(mdi_ctx *c, int p, int slot, const int *tok_dev, int T, const float *x_in, float *x_out, cudaStream_t st) {
    const int rc = tc_layers(c, p, nullptr, slot, tok_dev, T, x_in, x_out, st);
    if (rc == MDI_OK) ++c->st.stage_steps;
    return rc;
}

int tc_partition_step(mdi_ctx *c, int p, const Batch &bt, const float *x_in, float *x_out, cudaStream_t st) {
    return tc_layers(c, p, &bt, 0, nullptr, bt.n, x_in, x_out, st);
}

// Did a tensor-core first visit give up on one of its bounded waits?  (Synchronises the partition streams.)
int pf_check(mdi_ctx *c) {
    if (!c->pf_tc) return MDI_OK;
    for (auto &P : c->part) CU(cudaStreamSynchronize(P.stream));
    int e = 0;
    CU(cudaMemcpy(&e, c->tg_err, sizeof(int), cudaMemcpyDeviceToHost));
    if (e) {
        CU(cudaMemset(c->tg_err, 0, sizeof(int)));
        return fail(c, MDI_ERR_TIMEOUT, "a tensor-core first-visit kernel gave up waiting for its operands");
    }
    return MDI_OK;
}

// (Re)build the tiled copies of the matrices of the tensor-core linear layers after weights were loaded.
int pf_tile_weights(mdi_ctx *c) {
    const mdi_model_shape &s = c->s;
    const int d = s.d_model, F = s.d_ff, qw = s.n_head * s.head_dim, kw = s.n_kv_head * s.head_dim;
    struct M { const void *w; int rows, K, part; };
    std::vector<M> ms;
    for (int p = 0; p < c->K; ++p)
        for (int l = c->part[p].lo; l < c->part[p].hi; ++l) {
            const LayerW &L = c->layer[l];
            ms.push_back({L.wqkv, qw + 2 * kw, d, p});
            ms.push_back({L.wo, d, qw, p});
            ms.push_back({L.wgate, F, d, p});
            ms.push_back({L.wup, F, d, p});
            ms.push_back({L.wdown, d, F, p});
            ms.push_back({L.w1, F, d, p});
            ms.push_back({L.w2, d, F, p});
        }
    ms.push_back({s.tied_lm_head ? c->wte : c->lm_head, s.vocab, d, c->K - 1});
    for (const M &m : ms) {
        if (!m.w) continue;
        const size_t n_chunks = (size_t)((m.rows + TG_BM - 1) / TG_BM) * ((m.K + TG_BK - 1) / TG_BK) * (TG_BM * TG_BK / 8);
        void *&t = c->w_tiled[m.w];
        if (!t) {
            CU(cudaMalloc(&t, n_chunks * 16));
            c->part[m.part].buffer_bytes += (int64_t)n_chunks * 16;
        }
        k_tile_weights<<<(unsigned)((n_chunks + 255) / 256), 256, 0, c->main>>>((const __nv_bfloat16 *)m.w, m.rows, m.K, (__nv_bfloat16 *)t, n_chunks);
    }
    CU(cudaStreamSynchronize(c->main));
    CU(cudaGetLastError());
    c->tiles_stale = false;
    return MDI_OK;
}

int check_weights(mdi_ctx *c) {
    if (c->n_loaded != (int)c->tensors.size())
        for (auto &kv : c->tensors)
            if (!kv.second.loaded) return fail(c, MDI_ERR_STATE, "tensor '%s' was never loaded", kv.first.c_str());
    if (c->pf_tc && c->tiles_stale) return pf_tile_weights(c);
    return MDI_OK;
}

// Map pages so that rows [0, rows) of `slot` exist in every local layer of partition p.
int ensure_pages(mdi_ctx *c, int p, int slot, int rows) {
    Partition &P = c->part[p];
    const int Lp = P.hi - P.lo;
    const int need = (rows + c->page_tokens - 1) >> c->page_shift;
    int &have = P.pages_of_slot[slot];
    if (need <= have) return MDI_OK;
    if (need > c->pages_per_seq) return fail(c, MDI_ERR_CONTEXT, "slot %d: %d rows exceed n_ctx", slot, rows);
    if ((size_t)(need - have) * Lp > P.free_pages.size())
        return fail(c, MDI_ERR_OOM, "key/value page pool of partition %d exhausted (%zu free, %d needed)", p,
                    P.free_pages.size(), (need - have) * Lp);
    for (int l = 0; l < Lp; ++l)
        for (int g = have; g < need; ++g) {
            P.pt_host[((size_t)slot * Lp + l) * c->pages_per_seq + g] = P.free_pages.back();
            P.free_pages.pop_back();
        }
    have = need;
    const size_t off = (size_t)slot * Lp * c->pages_per_seq, n = (size_t)Lp * c->pages_per_seq;
    CU(cudaMemcpyAsync(P.pt_dev + off, P.pt_host.data() + off, n * sizeof(int), cudaMemcpyHostToDevice, P.stream));
    return MDI_OK;
}


// ---- persistent decode kernel: tables and launch -----------------------------------------------------
template <typename WT, typename KT> cudaError_t pk_attr(size_t smem) {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(k_persistent_decode<WT, 1, KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_persistent_decode<WT, 2, KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_persistent_decode<WT, 4, KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}
template <typename WT, typename KT> const void *pk_func(int nb) {
    return nb == 1 ? (const void *)k_persistent_decode<WT, 1, KT> : nb == 2 ? (const void *)k_persistent_decode<WT, 2, KT>
                                                                            : (const void *)k_persistent_decode<WT, 4, KT>;
}
const void *pk_func_for(const mdi_ctx *c, int nb) {
    if (c->s.weight_dtype == MDI_DTYPE_F32) return pk_func<float, float>(nb);
    return c->kv_kind == KV_F32 ? pk_func<__nv_bfloat16, float>(nb) : c->kv_kind == KV_F16 ? pk_func<__nv_bfloat16, __half>(nb) : pk_func<__nv_bfloat16, __nv_bfloat16>(nb);
}

// Phase list of every partition, team sizes (blocks per partition, in proportion to the bytes a step
// streams), shared-memory budget.  Leaves pk_ok false when the shape does not fit this kernel
// (groups of more than 4 samples, or too little shared memory for two ring slots).
int pk_setup(mdi_ctx *c) {
    const mdi_model_shape &s = c->s;
    const int K = c->K, d = s.d_model, qw = s.n_head * s.head_dim, kw = s.n_kv_head * s.head_dim;
    cudaDeviceProp prop;
    CU(cudaGetDeviceProperties(&prop, c->dev));
    c->n_sm = prop.multiProcessorCount;
    if (c->scheduler == 1 || c->scheduler == 3 || c->scheduler == 4) return MDI_OK;
    const bool want = c->scheduler == 2;
    if (c->gmax > PK_MAXNB) return want ? fail(c, MDI_ERR_SHAPE, "persistent scheduler: at most %d samples per group", PK_MAXNB) : MDI_OK;
    if (K > 32 || K > c->n_sm) return want ? fail(c, MDI_ERR_SHAPE, "persistent scheduler: too many partitions") : MDI_OK;
    c->pk_nb = c->gmax <= 1 ? 1 : c->gmax <= 2 ? 2 : 4;
    const int max_in = std::max(std::max(d, s.d_ff), qw);
    c->pk_xs_floats = c->pk_nb * ((max_in + 255) & ~255);
    const size_t misc = (size_t)(256 * 8 + 128 + 128 + 16 + 2 * PK_CWARPS * PK_MAXNB + 2 + PK_MAX_SLOTS) * 4 + 2 * PK_MAX_SLOTS * 8 +
                        PK_SMEM_PHASES * sizeof(PkPhase) + 128;
    const size_t fixed = (size_t)c->pk_xs_floats * 4 + misc;
    const size_t budget = (size_t)prop.sharedMemPerBlockOptin;
    if (fixed + 2 * PK_SLOT_BYTES > budget) return want ? fail(c, MDI_ERR_SHAPE, "persistent scheduler: inputs do not fit in shared memory") : MDI_OK;
    c->pk_slots = (int)std::min<size_t>(PK_MAX_SLOTS, (budget - fixed) / PK_SLOT_BYTES);
    c->pk_smem = fixed + (size_t)c->pk_slots * PK_SLOT_BYTES;
    {
        cudaError_t ea;
        if (s.weight_dtype == MDI_DTYPE_F32) ea = pk_attr<float, float>(c->pk_smem);
        else if (c->kv_kind == KV_F32) ea = pk_attr<__nv_bfloat16, float>(c->pk_smem);
        else if (c->kv_kind == KV_F16) ea = pk_attr<__nv_bfloat16, __half>(c->pk_smem);
        else ea = pk_attr<__nv_bfloat16, __nv_bfloat16>(c->pk_smem);
        CU(ea);
    }

    std::vector<PkPhase> &ph = c->pk_phases_host;
    ph.clear();
    c->pk_phase_begin.assign(K, 0);
    c->pk_phase_count.assign(K, 0);
    std::vector<double> bytes(K, 0.0);
    const bool rope = s.arch == MDI_ARCH_LLAMA;
    auto blocks16 = [](int n) { return (n + PK_SEGS - 1) / PK_SEGS; };
    for (int p = 0; p < K; ++p) {
        Partition &P = c->part[p];
        c->pk_phase_begin[p] = (int)ph.size();
        for (int l = P.lo; l < P.hi; ++l) {
            PkPhase q{};
            q.kind = PK_QKV; q.n_rows = qw + 2 * kw; q.in_dim = d; q.layer_local = l - P.lo; q.first_layer = l == P.lo;
            q.n_blocks = rope ? (q.n_rows / 2 + 7) / 8 : blocks16(q.n_rows);
            ph.push_back(q);
            PkPhase a{}; a.kind = PK_ATTN; a.layer_local = l - P.lo; ph.push_back(a);
            PkPhase o{}; o.kind = PK_OUT; o.n_rows = d; o.in_dim = qw; o.n_blocks = blocks16(d); o.layer_local = l - P.lo; o.first_layer = l == P.lo; ph.push_back(o);
            PkPhase f{};
            if (s.act == MDI_ACT_SWIGLU) { f.kind = PK_GATEUP; f.n_rows = s.d_ff; f.in_dim = d; f.n_blocks = (s.d_ff + 7) / 8; }
            else { f.kind = PK_FC1; f.n_rows = s.d_ff; f.in_dim = d; f.n_blocks = blocks16(s.d_ff); }
            f.layer_local = l - P.lo; ph.push_back(f);
            PkPhase g{}; g.kind = PK_FC2; g.n_rows = d; g.in_dim = s.d_ff; g.n_blocks = blocks16(d); g.layer_local = l - P.lo; ph.push_back(g);
            bytes[p] += (double)((size_t)(qw + 2 * kw) * d + (size_t)d * qw + (size_t)(s.act == MDI_ACT_SWIGLU ? 3 : 2) * s.d_ff * d) * c->esize;
        }
        if (p == K - 1) {
            PkPhase h{}; h.kind = PK_HEAD; h.n_rows = s.vocab; h.in_dim = d; h.n_blocks = blocks16(s.vocab); ph.push_back(h);
            bytes[p] += (double)s.vocab * d * c->esize;
        }
        c->pk_phase_count[p] = (int)ph.size() - c->pk_phase_begin[p];
    }
    // team sizes
    std::vector<int> n_cta(K, 1);
    {
        // Proportional to the bytes a step streams, then rounded down to a size that deals the row blocks of
        // the d_model-row matrices (and the attention items) out evenly - uneven shares make every phase wait
        // for the blocks with one more tile - unless that would give up more than 30% of the share.
        const int unit = (blocks16(d) % 2 == 0) ? blocks16(d) / 2 : blocks16(d);
        auto even_size = [&](int share) {
            int best = share;
            if ((share + 1) % unit == 0 || (unit % (share + 1) == 0)) return share + 1; // one block short of an even size
            if (share >= unit) best = share / unit * unit;
            else
                for (int k = 2; k <= unit; ++k)
                    if (unit % k == 0 && unit / k <= share) { best = unit / k; break; }
            return best * 10 >= share * 7 ? best : share;
        };
        double tot = 0;
        for (double b : bytes) tot += b;
        int used = 0, big = 0;
        for (int p = 0; p < K; ++p)
            if (bytes[p] > bytes[big]) big = p;
        for (int p = 0; p < K; ++p) {
            if (p == big) continue;
            n_cta[p] = even_size(std::max(1, (int)std::floor(c->n_sm * bytes[p] / tot)));
            used += n_cta[p];
        }
        if (c->n_sm - used < 1) return want ? fail(c, MDI_ERR_SHAPE, "persistent scheduler: not enough SMs") : MDI_OK;
        n_cta[big] = even_size(c->n_sm - used);
    }
    c->pk_teams_host.assign(K, PkTeam{});
    int first = 0, rcx;
    if ((rcx = dalloc(c, &c->pk_sync, (size_t)K * 64)) != MDI_OK) return rcx;
    if ((rcx = dalloc(c, &c->pk_err, 1)) != MDI_OK) return rcx;
    if ((rcx = dalloc(c, &c->pk_prof, (size_t)c->n_sm * PK_PROF_N)) != MDI_OK) return rcx;
    c->pk_prof_on = c->o.in_kernel_timing != 0;
    for (int p = 0; p < K; ++p) {
        Partition &P = c->part[p];
        PkTeam &T = c->pk_teams_host[p];
        T.first_cta = first; T.n_cta = n_cta[p]; first += n_cta[p];
        T.phase_begin = c->pk_phase_begin[p]; T.n_phases = c->pk_phase_count[p];
        T.is_first = p == 0; T.is_last = p == K - 1;
        T.n_split = std::max(1, std::min(4, n_cta[p] / (c->pk_nb * s.n_head)));
        T.kv = kv_view(c, P);
        T.qbuf = P.qbuf; T.part = P.part; T.hbuf = P.hbuf; T.x_embed = P.x_embed; T.x_last = P.x_last;
        T.ring_in = p > 0 ? c->part[p - 1].ring : nullptr;
        T.ring_out = p < K - 1 ? P.ring : nullptr;
        T.pos = P.pos_dev;
        T.bar = c->pk_sync + (size_t)p * 64;
        T.flag_out = c->pk_sync + (size_t)p * 64 + 32;
        T.flag_in = c->pk_sync + (size_t)((p + K - 1) % K) * 64 + 32;
    }
    if ((rcx = dalloc(c, &c->pk_teams, (size_t)K)) != MDI_OK) return rcx;
    if ((rcx = dalloc(c, &c->pk_phases, ph.size())) != MDI_OK) return rcx;
    CU(cudaMemcpy(c->pk_teams, c->pk_teams_host.data(), sizeof(PkTeam) * K, cudaMemcpyHostToDevice));
    c->pk_ok = true;
    return MDI_OK;
}

// Weight pointers are known once the tensors are loaded: (re)write the device phase table when they changed.
int pk_fill_phases(mdi_ctx *c) {
    if (!c->pk_tables_stale) return MDI_OK;
    const mdi_model_shape &s = c->s;
    std::vector<PkPhase> &ph = c->pk_phases_host;
    for (int p = 0; p < c->K; ++p) {
        Partition &P = c->part[p];
        for (int i = 0; i < c->pk_phase_count[p]; ++i) {
            PkPhase &q = ph[c->pk_phase_begin[p] + i];
            if (q.kind == PK_HEAD) {
                q.W = s.tied_lm_head ? c->wte : c->lm_head; q.gamma = c->lnfg; q.beta = c->lnfb;
                continue;
            }
            const LayerW &L = c->layer[P.lo + q.layer_local];
            switch (q.kind) {
                case PK_QKV: q.W = L.wqkv; q.bias = L.bqkv; q.gamma = L.ln1g; q.beta = L.ln1b; break;
                case PK_OUT: q.W = L.wo; q.bias = L.bo; break;
                case PK_FC1: q.W = L.w1; q.bias = L.b1; q.gamma = L.ln2g; q.beta = L.ln2b; break;
                case PK_GATEUP: q.W = L.wgate; q.W2 = L.wup; q.gamma = L.ln2g; q.beta = L.ln2b; break;
                case PK_FC2: q.W = s.act == MDI_ACT_SWIGLU ? L.wdown : L.w2; q.bias = L.b2; break;
                default: break;
            }
        }
    }
    CU(cudaMemcpy(c->pk_phases, ph.data(), sizeof(PkPhase) * ph.size(), cudaMemcpyHostToDevice));
    c->pk_tables_stale = false;
    return MDI_OK;
}

// The kernel counts the weight tiles a block has consumed in 32 bits: an upper bound for one launch.
bool pk_tile_count_fits(const mdi_ctx *c, int n_pass, int G) {
    double worst = 0;
    for (int p = 0; p < c->K; ++p) {
        double per_step = 0;
        for (int i = 0; i < c->pk_phase_count[p]; ++i) {
            const PkPhase &q = c->pk_phases_host[c->pk_phase_begin[p] + i];
            if (q.kind == PK_ATTN) continue;
            const double chunks = std::ceil((double)q.in_dim * c->esize / (PK_SLOT_BYTES / PK_SEGS));
            per_step += (std::floor((double)q.n_blocks / c->pk_teams_host[p].n_cta) + 1) * chunks;
        }
        worst = std::max(worst, per_step);
    }
    return worst * (double)n_pass * G < 2.0e9;
}

// One cooperative launch that runs n_pass passes of the recurrent pipeline for samples 0..n_samples-1.
int pk_launch(mdi_ctx *c, int n_samples, int G, int n_pass) {
    const mdi_model_shape &s = c->s;
    int rc = pk_fill_phases(c);
    if (rc != MDI_OK) return rc;
    CU(cudaMemsetAsync(c->pk_sync, 0, (size_t)c->K * 64 * sizeof(unsigned), c->main));
    CU(cudaMemsetAsync(c->pk_err, 0, sizeof(int), c->main));
    if (c->pk_prof_on) CU(cudaMemsetAsync(c->pk_prof, 0, (size_t)c->n_sm * PK_PROF_N * 8, c->main));
    PkParams P{};
    P.d = s.d_model; P.n_head = s.n_head; P.n_kv_head = s.n_kv_head; P.head_dim = s.head_dim; P.d_ff = s.d_ff; P.vocab = s.vocab;
    P.norm = s.arch == MDI_ARCH_GPT ? NORM_LAYER : NORM_RMS; P.act = s.act == MDI_ACT_GELU_ERF; P.rope = s.arch == MDI_ARCH_LLAMA;
    P.K = c->K; P.G = G; P.n_samples = n_samples; P.gmax = c->gmax; P.n_pass = n_pass; P.n_slots_ring = c->pk_slots; P.xs_floats = c->pk_xs_floats;
    P.eps = s.norm_eps; P.scale = 1.0f / std::sqrt((float)s.head_dim);
    P.teams = c->pk_teams; P.phases = c->pk_phases; P.wte = c->wte; P.wpe = c->wpe; P.rope_cos = c->rope_cos; P.rope_sin = c->rope_sin;
    P.logits = c->logits; P.head_pv = c->head_pv; P.head_pi = c->head_pi; P.cur_tok = c->cur_tok; P.tok_log = c->tok_log;
    P.gen_count = c->gen_count; P.teacher = c->teacher; P.n_teacher = c->n_teacher; P.log_stride = s.n_ctx; P.err = c->pk_err;
    P.prof = c->pk_prof_on ? c->pk_prof : nullptr;
    P.hd_shift = 0;
    while ((1 << P.hd_shift) < s.head_dim) ++P.hd_shift;
    P.wait_ns = c->o.wait_limit_ms > 0 ? (unsigned long long)c->o.wait_limit_ms * 1000000ull : PK_WAIT_NS;
    P.withhold_partition = c->withhold_once;
    c->withhold_once = -1;
    int grid = 0;
    for (auto &T : c->pk_teams_host) grid += T.n_cta;
    const int nb = (n_samples + G - 1) / G;
    const int tnb = nb <= 1 ? 1 : nb <= 2 ? 2 : 4;
    const void *fn = pk_func_for(c, tnb);
    CU(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->pk_smem)); // per function, not per context
    void *args[] = {&P};
    CU(cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(PK_THREADS), args, c->pk_smem, c->main));
    ++c->st.kernel_launches;
    c->st.stage_steps += (int64_t)c->K * n_pass * G;
    return MDI_OK;
}


// ---- fused-phase persistent kernel: plan, weight stream and launch -------------------------------------
const void *fz_func(int nb) {
    return nb == 1 ? (const void *)k_fused_decode<1> : nb == 2 ? (const void *)k_fused_decode<2> : (const void *)k_fused_decode<4>;
}

// Plan of the fused-phase kernel: team sizes, which block serves which head of which layer, which hidden
// units of the MLP, which rows of the output layer, so that every block streams about the same number of
// bytes per step.  Independent of the weights' addresses.  Leaves fz_ok false when the shape does not fit
// (not the GPT block, weights not bf16, cache not fp32, grouped-query attention, more than 4 samples per
// group, a team smaller than the number of heads).
int fz_setup(mdi_ctx *c) {
    const mdi_model_shape &s = c->s;
    const int K = c->K, d = s.d_model, hd = s.head_dim, H = s.n_head;
    const bool want = c->scheduler == 3;
    auto no = [&](const char *why) { return want ? fail(c, MDI_ERR_SHAPE, "fused-phase scheduler: %s", why) : MDI_OK; };
    if (c->scheduler == 1 || c->scheduler == 2 || c->scheduler == 4) return MDI_OK;
    if (s.arch != MDI_ARCH_GPT || s.weight_dtype != MDI_DTYPE_BF16 || !c->kv_f32) return no("needs the GPT block, bf16 weights and an fp32 cache");
    if (s.n_kv_head != H || H * hd != d) return no("needs n_kv_head = n_head and n_head * head_dim = d_model");
    if (d % 16 || s.d_ff % 16 || hd % 16) return no("widths must be multiples of 16");
    if (d > FZ_U * FZ_CTHREADS) return no("d_model above 1024");
    if (c->gmax > FZ_MAXNB) return no("at most 4 samples per group");
    if (K > 32) return no("too many partitions");
    cudaDeviceProp prop;
    CU(cudaGetDeviceProperties(&prop, c->dev));
    const int n_sm = prop.multiProcessorCount;
    c->fz_nb = c->gmax <= 1 ? 1 : c->gmax <= 2 ? 2 : 4;
    const int NB = c->fz_nb;
    // Pair mode: a head is served by the two blocks of a cluster (halves of its q,k,v rows, of the rows of every cache
    // page and of its output rows).  Needs even tile counts, pages of at least two rows, even team sizes with a cluster
    // per head, and all clusters resident at once.
    bool pair = c->o.fused_blocks_per_head != 1 && c->page_tokens >= 2 && (3 * hd / 16) % 2 == 0 && (d / 16) % 2 == 0 && n_sm >= 2;
    if (pair) {
        for (int nb : {1, 2, 4}) CU(cudaFuncSetAttribute(fz_func(nb), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)prop.sharedMemPerBlockOptin));
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(n_sm & ~1); cfg.blockDim = dim3(FZ_THREADS); cfg.dynamicSmemBytes = prop.sharedMemPerBlockOptin;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&n_clusters, fz_func(c->fz_nb), &cfg) != cudaSuccess) { cudaGetLastError(); n_clusters = 0; }
        if (n_clusters < (n_sm & ~1) / 2) pair = false;
    }
    // team sizes in proportion to the bytes a step streams
    std::vector<double> bytes(K, 0.0);
    const double layer_bytes = 2.0 * (4.0 * d * d + 2.0 * (double)s.d_ff * d);
    for (int p = 0; p < K; ++p) {
        bytes[p] = layer_bytes * (c->part[p].hi - c->part[p].lo);
        if (p == K - 1) bytes[p] += 2.0 * (double)s.vocab * d;
    }
    std::vector<int> n_cta(K, 0);
    auto team_sizes = [&](bool even) {
        double tot = 0;
        for (double b : bytes) tot += b;
        int used = 0, big = 0;
        for (int p = 0; p < K; ++p) if (bytes[p] > bytes[big]) big = p;
        for (int p = 0; p < K; ++p) {
            if (p == big) continue;
            n_cta[p] = std::max(1, (int)std::floor(n_sm * bytes[p] / tot));
            if (even) n_cta[p] = std::max(2, n_cta[p] & ~1);
            used += n_cta[p];
        }
        n_cta[big] = even ? (n_sm - used) & ~1 : n_sm - used;
        // pair mode wants a cluster per head in every team: a team that is short of 2 * n_head blocks by at most a
        // quarter takes the difference from the largest team (measured on the GPT-2-medium shape: +20% tokens/s)
        for (int p = 0; p < K && even; ++p) {
            const int need = 2 * H - n_cta[p];
            if (p != big && need > 0 && need * 4 <= n_cta[p] && n_cta[big] - need >= 2 * H) { n_cta[p] += need; n_cta[big] -= need; }
        }
    };
    team_sizes(pair);
    for (int p = 0; p < K && pair; ++p)
        if (n_cta[p] / 2 < H) { pair = false; team_sizes(false); } // not a cluster per head in every team: one block per head
    for (int p = 0; p < K; ++p)
        if (n_cta[p] < H) return no("a team has fewer blocks than the model has heads");
    c->fz_pair = pair;
    const int pr = pair ? 2 : 1, qkv_tiles = 3 * hd / 16 / pr, out_tiles = d / 16 / pr;

    // per team: phases; per block: work items
    c->fz_teams_host.assign(K, FzTeam{});
    c->fz_phase_begin.assign(K, 0);
    c->fz_phase_count.assign(K, 0);
    c->fz_works_host.clear();
    c->fz_unit_lists.clear();
    c->fz_blocks_host.clear();
    int n_phases_total = 0, first = 0, m_max = 1;
    for (int p = 0; p < K; ++p) {
        const int n = n_cta[p], Lp = c->part[p].hi - c->part[p].lo, np = 2 * Lp + (p == K - 1 ? 1 : 0);
        c->fz_phase_begin[p] = n_phases_total;
        c->fz_phase_count[p] = np;
        n_phases_total += np;
        // Phases end in a team barrier, so what counts is the slowest block of each phase: hidden units and output
        // rows are dealt out evenly within their own phase; heads rotate over the blocks from layer to layer so
        // that the same blocks do not wait (with full rings) through every attention phase.
        std::vector<std::vector<FzWork>> wk(n, std::vector<FzWork>(np, FzWork{-1, 0, 0, 0, 0, 0, 0}));
        std::vector<std::vector<std::vector<int>>> ul(n, std::vector<std::vector<int>>(np));
        int next_head_block = 0;
        for (int l = 0; l < Lp; ++l) {
            for (int h = 0; h < H; ++h) {
                for (int r = 0; r < pr; ++r) {
                    FzWork &a = wk[next_head_block + r][2 * l];
                    a.unit = h;
                    a.n_tiles = qkv_tiles; a.tile0 = r * qkv_tiles;
                    a.row_tiles = out_tiles; a.row_tile0 = r * out_tiles;
                }
                next_head_block = (next_head_block + pr) % (n / pr * pr);
            }
            // blocks without a head in this layer come first: their rings had the attention phase to fill up
            const int n_units = s.d_ff / 16;
            for (int u = 0; u < n_units; ++u) ul[(next_head_block + u) % n][2 * l + 1].push_back(u);
            for (int b = 0; b < n; ++b) {
                wk[b][2 * l + 1].n_tiles = (int)ul[b][2 * l + 1].size();
                m_max = std::max(m_max, wk[b][2 * l + 1].n_tiles);
            }
        }
        if (p == K - 1) {
            const int NT = (s.vocab + 15) / 16;
            int t0 = 0;
            for (int b = 0; b < n; ++b) {
                const int give = NT / n + (b < NT % n ? 1 : 0);
                wk[b][np - 1].n_tiles = give; wk[b][np - 1].tile0 = t0; t0 += give;
            }
        }
        for (int b = 0; b < n; ++b) {
            FzBlock fb{};
            fb.work_begin = (int)c->fz_works_host.size();
            c->fz_blocks_host.push_back(fb);
            for (int i = 0; i < np; ++i) { c->fz_works_host.push_back(wk[b][i]); c->fz_unit_lists.push_back(ul[b][i]); }
        }
        FzTeam &T = c->fz_teams_host[p];
        T.first_cta = first; T.n_cta = n; first += n;
        T.phase_begin = c->fz_phase_begin[p]; T.n_phases = np;
        T.is_first = p == 0; T.is_last = p == K - 1;
    }
    c->fz_grid = first;
    for (int p = 0; p < K; ++p) {
        if (c->fz_phase_count[p] > FZ_MAX_PHASES) return no("too many blocks of the model in one partition");
        // a block serves at most one head per layer, so it has at most Lp + 1 segments
        if (c->part[p].hi - c->part[p].lo + 1 > FZ_MAX_SEGS) return no("too many blocks of the model in one partition");
    }
    for (size_t b = 0; b < c->fz_blocks_host.size(); ++b) {
        size_t nu = 0;
        const size_t w0 = c->fz_blocks_host[b].work_begin, w1 = b + 1 < c->fz_blocks_host.size() ? c->fz_blocks_host[b + 1].work_begin : c->fz_unit_lists.size();
        for (size_t i = w0; i < w1; ++i) nu += c->fz_unit_lists[i].size();
        if (nu > FZ_MAX_UNITS) return no("too many hidden units per thread block");
    }
    // cache rows through the ring: whole pages of one head, as many as fit a slot
    {
        c->fz_kv_rows = c->page_tokens / pr;
        const size_t page_kv_bytes = (size_t)2 * c->fz_kv_rows * hd * 4; // keys and values of a block's rows of one page of one head
        if (page_kv_bytes > (size_t)FZ_SLOT_BYTES) return no("one head's rows of a cache page exceed a ring slot");
        c->fz_kv_pps = std::min<int>(32, (int)(FZ_SLOT_BYTES / page_kv_bytes));
    }
    // shared memory
    m_max = (m_max + 3) & ~3;
    const int max_tiles = std::max(qkv_tiles, m_max);
    c->fz_xb_stride = d + 8; c->fz_hb_stride = 16 * m_max + 8; c->fz_ob_stride = hd + 8;
    c->fz_part_floats = std::max(max_tiles * FZ_CWARPS * 16 * NB, (128 + 16) * FZ_CWARPS); // also the attention scratch
    const size_t fixed = fz_smem_layout(NB, 0, d, hd, c->fz_part_floats, c->pages_per_seq, c->fz_xb_stride, c->fz_hb_stride, c->fz_ob_stride).total;
    const size_t budget = (size_t)prop.sharedMemPerBlockOptin;
    if (fixed + 2 * (size_t)FZ_SLOT_BYTES > budget) return no("activations do not fit in shared memory");
    c->fz_slots = (int)std::min<size_t>(FZ_MAX_SLOTS, (budget - fixed) / FZ_SLOT_BYTES);
    c->fz_smem = fz_smem_layout(NB, c->fz_slots, d, hd, c->fz_part_floats, c->pages_per_seq, c->fz_xb_stride, c->fz_hb_stride, c->fz_ob_stride).total;
    for (int nb : {1, 2, 4}) CU(cudaFuncSetAttribute(fz_func(nb), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->fz_smem));
    int rc;
    if ((rc = dalloc(c, &c->fz_sync, (size_t)K * 64)) != MDI_OK) return rc;
    if ((rc = dalloc(c, &c->fz_err, 1)) != MDI_OK) return rc;
    if ((rc = dalloc(c, &c->fz_acc, (size_t)K * 3 * FZ_MAXNB * d)) != MDI_OK) return rc;
    c->fz_prof_on = c->o.in_kernel_timing != 0;
    if (c->fz_prof_on && (rc = dalloc(c, &c->fz_prof, (size_t)c->fz_grid * PK_PROF_N)) != MDI_OK) return rc;
    c->fz_ok = true;
    return MDI_OK;
}

// The weights in the order the plan consumes them: one descriptor per fragment block, gathered on the device.
// Runs before the first fused launch and again after weights were replaced.
int fz_build(mdi_ctx *c) {
    if (!c->fz_stale) return MDI_OK;
    const mdi_model_shape &s = c->s;
    const int K = c->K, d = s.d_model, hd = s.head_dim, H = s.n_head, qw = H * hd, ks = d / 16;
    void *old[] = {c->fz_teams, c->fz_phases, c->fz_works, c->fz_blocks, c->fz_segs, c->fz_units, c->fz_stream};
    for (void *q : old) if (q) cudaFree(q);
    c->fz_teams = nullptr; c->fz_phases = nullptr; c->fz_works = nullptr; c->fz_blocks = nullptr; c->fz_segs = nullptr; c->fz_units = nullptr; c->fz_stream = nullptr;
    std::vector<FzPhase> phases;
    std::vector<FzFbDesc> desc;
    std::vector<FzSeg> segs;
    c->fz_units_host.clear();
    const void *head_w = s.tied_lm_head ? c->wte : c->lm_head;
    auto rounds = [&](const void *W, int ld, int n_t, int n_k, auto &&row_of, auto &&col_of, int row_limit) {
        for (int r0 = 0; r0 < n_t; r0 += FZ_CWARPS) {
            const int n_r = std::min(FZ_CWARPS, n_t - r0);
            for (int k = 0; k < n_k; ++k)
                for (int w = 0; w < n_r; ++w) {
                    const int row0 = row_of(r0 + w);
                    desc.push_back(FzFbDesc{W, ld, row0, col_of(k), std::max(0, std::min(16, row_limit - row0))});
                }
        }
    };
    for (int p = 0; p < K; ++p) {
        Partition &P = c->part[p];
        FzTeam &T = c->fz_teams_host[p];
        const int Lp = P.hi - P.lo, np = T.n_phases;
        for (int l = 0; l < Lp; ++l) {
            const LayerW &L = c->layer[P.lo + l];
            FzPhase a{}; a.kind = FZ_A; a.layer_local = l; a.gamma = L.ln1g; a.beta = L.ln1b;
            a.bias_in = l > 0 ? c->layer[P.lo + l - 1].b2 : nullptr; a.bias_rows = L.bqkv;
            phases.push_back(a);
            FzPhase b{}; b.kind = FZ_B; b.layer_local = l; b.gamma = L.ln2g; b.beta = L.ln2b; b.bias_in = L.bo; b.bias_rows = L.b1;
            phases.push_back(b);
        }
        if (p == K - 1) {
            FzPhase h{}; h.kind = FZ_HEAD; h.gamma = c->lnfg; h.beta = c->lnfb; h.bias_in = c->layer[P.hi - 1].b2;
            phases.push_back(h);
        }
        T.kv = kv_view(c, P);
        T.ring_in = p > 0 ? c->part[p - 1].ring : nullptr;
        T.ring_out = p < K - 1 ? P.ring : nullptr;
        T.bias_final = c->layer[P.hi - 1].b2;
        T.pos = P.pos_dev;
        T.bar = c->fz_sync + (size_t)p * 64;
        T.flag_out = c->fz_sync + (size_t)p * 64 + 32;
        T.flag_in = c->fz_sync + (size_t)((p + K - 1) % K) * 64 + 32;
        T.acc = c->fz_acc + (size_t)p * 3 * FZ_MAXNB * d;
        for (int b = 0; b < T.n_cta; ++b) {
            FzBlock &FB = c->fz_blocks_host[T.first_cta + b];
            const size_t fb_begin = desc.size();
            FB.seg_begin = (int)segs.size();
            FB.unit_begin = (int)c->fz_units_host.size();
            size_t seg_fb0 = fb_begin; // first fragment block of the open segment
            int slots_before = 0;
            auto close_segment = [&](int kv_layer, int kv_head) {
                FzSeg sg{};
                sg.fb_begin = (int)(seg_fb0 - fb_begin); sg.n_fb = (int)(desc.size() - seg_fb0); sg.slots_before = slots_before;
                sg.kv_layer = kv_layer; sg.kv_head = kv_head;
                segs.push_back(sg);
                slots_before += (sg.n_fb + FZ_SLOT_FB - 1) / FZ_SLOT_FB;
                seg_fb0 = desc.size();
            };
            for (int i = 0; i < np; ++i) {
                FzWork &wk = c->fz_works_host[FB.work_begin + i];
                const std::vector<int> &ul = c->fz_unit_lists[FB.work_begin + i];
                const bool is_head = p == K - 1 && i == np - 1;
                const LayerW &L = c->layer[P.lo + std::min(i / 2, Lp - 1)];
                wk.seg0 = wk.seg1 = (int)segs.size() - FB.seg_begin;
                wk.fb0 = wk.fb1 = (int)(desc.size() - seg_fb0);
                if (is_head) {
                    const int t0 = wk.tile0;
                    rounds(head_w, d, wk.n_tiles, ks, [&](int t) { return (t0 + t) * 16; }, [&](int k) { return 16 * k; }, s.vocab);
                } else if (i % 2 == 0) {
                    if (wk.unit < 0) continue;
                    const int h = wk.unit, tph = hd / 16;
                    for (int tt = 0; tt < wk.n_tiles; ++tt)
                        for (int k = 0; k < ks; ++k) {
                            const int t = wk.tile0 + tt; // row tile of the head's q, k, v rows
                            desc.push_back(FzFbDesc{L.wqkv, d, (t / tph) * qw + h * hd + (t % tph) * 16, 16 * k, 16});
                        }
                    close_segment(i / 2, h); // this head's cache rows follow in the ring
                    wk.seg1 = (int)segs.size() - FB.seg_begin;
                    wk.fb1 = 0;
                    const int rt0 = wk.row_tile0;
                    rounds(L.wo, qw, wk.row_tiles, hd / 16, [&](int t) { return (rt0 + t) * 16; }, [&](int k) { return h * hd + 16 * k; }, d);
                } else {
                    wk.tile0 = (int)c->fz_units_host.size() - FB.unit_begin;
                    for (int u : ul) c->fz_units_host.push_back(u);
                    if (ul.empty()) continue;
                    for (int u : ul)
                        for (int k = 0; k < ks; ++k) desc.push_back(FzFbDesc{L.w1, d, u * 16, 16 * k, 16});
                    wk.fb1 = (int)(desc.size() - seg_fb0);
                    rounds(L.w2, s.d_ff, d / 16, (int)ul.size(), [&](int t) { return t * 16; }, [&](int k) { return ul[k] * 16; }, d);
                }
            }
            close_segment(-1, -1);
            FB.n_seg = (int)segs.size() - FB.seg_begin;
            FB.n_units = (int)c->fz_units_host.size() - FB.unit_begin;
            FB.n_fb = (int)(desc.size() - fb_begin);
            FB.stream = reinterpret_cast<const uint4 *>(fb_begin); // fragment-block index for now; the address follows
        }
    }
    const size_t n_fb = desc.size();
    c->fz_stream_bytes = (int64_t)n_fb * FZ_FB_BYTES;
    c->fz_team_stream_bytes.assign(K, 0);
    for (int p = 0; p < K; ++p)
        for (int b = 0; b < c->fz_teams_host[p].n_cta; ++b)
            c->fz_team_stream_bytes[p] += (int64_t)c->fz_blocks_host[c->fz_teams_host[p].first_cta + b].n_fb * FZ_FB_BYTES;
    CU(cudaMalloc((void **)&c->fz_stream, std::max<size_t>(n_fb, 1) * FZ_FB_BYTES));
    for (auto &FB : c->fz_blocks_host) FB.stream = c->fz_stream + reinterpret_cast<size_t>(FB.stream) * (FZ_FB_BYTES / 16);
    {
        FzFbDesc *ddesc = nullptr;
        CU(cudaMalloc((void **)&ddesc, std::max<size_t>(n_fb, 1) * sizeof(FzFbDesc)));
        cudaError_t e = cudaMemcpy(ddesc, desc.data(), n_fb * sizeof(FzFbDesc), cudaMemcpyHostToDevice);
        if (e == cudaSuccess && n_fb) {
            k_fz_repack<<<(unsigned)((n_fb + 7) / 8), 256, 0, c->main>>>(ddesc, c->fz_stream, (long)n_fb);
            ++c->st.kernel_launches;
            e = cudaStreamSynchronize(c->main);
        }
        cudaFree(ddesc);
        CU(e);
    }
    auto up = [&](auto **dst, const auto &v) -> cudaError_t {
        using E = typename std::remove_reference<decltype(v[0])>::type;
        cudaError_t e = cudaMalloc((void **)dst, std::max<size_t>(v.size(), 1) * sizeof(E));
        if (e != cudaSuccess) return e;
        return cudaMemcpy(*dst, v.data(), v.size() * sizeof(E), cudaMemcpyHostToDevice);
    };
    CU(up(&c->fz_teams, c->fz_teams_host));
    CU(up(&c->fz_phases, phases));
    CU(up(&c->fz_works, c->fz_works_host));
    CU(up(&c->fz_blocks, c->fz_blocks_host));
    CU(up(&c->fz_segs, segs));
    CU(up(&c->fz_units, c->fz_units_host));
    c->fz_stale = false;
    return MDI_OK;
}

// The kernel counts ring slots in 32 bits per launch.
bool fz_slot_count_fits(const mdi_ctx *c, int n_pass, int G) {
    double worst = 0;
    // static slots of a step plus, per head unit and sample, the slots of a full context of cache rows
    const double kv = (double)FZ_MAXNB * (c->pages_per_seq / (double)c->fz_kv_pps + 1.0);
    for (const auto &FB : c->fz_blocks_host) worst = std::max(worst, std::ceil((double)FB.n_fb / FZ_SLOT_FB) + FB.n_seg * (1.0 + kv));
    return worst * (double)n_pass * G < 2.0e9;
}

int fz_launch(mdi_ctx *c, int n_samples, int G, int n_pass) {
    const mdi_model_shape &s = c->s;
    int rc = fz_build(c);
    if (rc != MDI_OK) return rc;
    CU(cudaMemsetAsync(c->fz_sync, 0, (size_t)c->K * 64 * sizeof(unsigned), c->main));
    CU(cudaMemsetAsync(c->fz_err, 0, sizeof(int), c->main));
    CU(cudaMemsetAsync(c->fz_acc, 0, (size_t)c->K * 3 * FZ_MAXNB * s.d_model * sizeof(long long), c->main));
    if (c->fz_prof_on) CU(cudaMemsetAsync(c->fz_prof, 0, (size_t)c->fz_grid * PK_PROF_N * 8, c->main));
    FzParams P{};
    P.d = s.d_model; P.n_head = s.n_head; P.head_dim = s.head_dim; P.d_ff = s.d_ff; P.vocab = s.vocab; P.act = s.act == MDI_ACT_GELU_ERF;
    P.K = c->K; P.G = G; P.n_samples = n_samples; P.gmax = c->gmax; P.n_pass = n_pass; P.n_slots_ring = c->fz_slots;
    P.xb_stride = c->fz_xb_stride; P.hb_stride = c->fz_hb_stride; P.ob_stride = c->fz_ob_stride; P.part_floats = c->fz_part_floats;
    P.pages_per_seq = c->pages_per_seq; P.kv_pps = c->fz_kv_pps; P.pair = c->fz_pair; P.kv_rows = c->fz_kv_rows; P.segs = c->fz_segs;
    P.eps = s.norm_eps; P.scale = 1.0f / std::sqrt((float)s.head_dim);
    P.teams = c->fz_teams; P.phases = c->fz_phases; P.works = c->fz_works; P.blocks = c->fz_blocks; P.units = c->fz_units;
    P.wte = c->wte; P.wpe = c->wpe; P.logits = c->logits; P.head_pv = c->head_pv; P.head_pi = c->head_pi;
    P.cur_tok = c->cur_tok; P.tok_log = c->tok_log; P.gen_count = c->gen_count; P.teacher = c->teacher; P.n_teacher = c->n_teacher;
    P.log_stride = s.n_ctx; P.err = c->fz_err;
    P.wait_ns = c->o.wait_limit_ms > 0 ? (unsigned long long)c->o.wait_limit_ms * 1000000ull : PK_WAIT_NS;
    P.withhold_partition = c->withhold_once;
    c->withhold_once = -1;
    P.prof = c->fz_prof_on ? c->fz_prof : nullptr;
    // trace_slot: with in-kernel timing on, thread 0 of every block also records a time stamp at every category
    // change while it serves that schedule slot (read back with mdi_get_trace)
    if (c->fz_prof_on && c->o.trace_slot > 0) {
        if (!c->fz_trace || c->fz_trace_blocks != c->fz_grid) {
            if (c->fz_trace) cudaFree(c->fz_trace);
            c->fz_trace = nullptr;
            CU(cudaMalloc((void **)&c->fz_trace, (size_t)c->fz_grid * FZ_TRACE_N * 8));
            c->fz_trace_blocks = c->fz_grid;
        }
        CU(cudaMemsetAsync(c->fz_trace, 0, (size_t)c->fz_grid * FZ_TRACE_N * 8, c->main));
        P.trace = c->fz_trace;
        P.trace_step = c->o.trace_slot - 1;
    }
    // the template parameter fixes the accumulator stride, so it is the context's group size, not this call's
    const void *fn = fz_func(c->fz_nb);
    CU(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->fz_smem)); // per function, not per context
    void *args[] = {&P};
    if (c->fz_pair) {
        // cooperative (all blocks resident: teams wait on one another) and in clusters of two (the halves of a head)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(c->fz_grid); cfg.blockDim = dim3(FZ_THREADS); cfg.dynamicSmemBytes = c->fz_smem; cfg.stream = c->main;
        cudaLaunchAttribute at[2];
        at[0].id = cudaLaunchAttributeCooperative; at[0].val.cooperative = 1;
        at[1].id = cudaLaunchAttributeClusterDimension;
        at[1].val.clusterDim.x = 2; at[1].val.clusterDim.y = 1; at[1].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 2;
        const cudaError_t le = cudaLaunchKernelExC(&cfg, fn, args);
        if (le != cudaSuccess) {
            cudaGetLastError();
            return fail(c, MDI_ERR_CUDA, "the runtime refused the cooperative launch in clusters of two (%s): create the context with "
                        "fused_blocks_per_head = 1 (one block per head, no clusters)", cudaGetErrorString(le));
        }
    } else {
        CU(cudaLaunchCooperativeKernel(fn, dim3(c->fz_grid), dim3(FZ_THREADS), args, c->fz_smem, c->main));
    }
    ++c->st.kernel_launches;
    c->st.stage_steps += (int64_t)c->K * n_pass * G;
    return MDI_OK;
}


// ---- persistent tensor-core decode kernel: plan, tables and launch ----------------------------------------
template <typename KT> cudaError_t td_attr(size_t smem) {
    return cudaFuncSetAttribute(k_tc_decode<KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}
const void *td_func(const mdi_ctx *c) {
    return c->kv_kind == KV_F32 ? (const void *)k_tc_decode<float> : c->kv_kind == KV_F16 ? (const void *)k_tc_decode<__half> : (const void *)k_tc_decode<__nv_bfloat16>;
}

// How many ranges of k-blocks a contraction with `tiles` row tiles (all its matrices together) and n_kb k-blocks is
// cut into for a team of n_cta blocks: at least so many that a range fits the resident B operand; beyond that the
// count that minimises the estimated time of the busiest block (a phase ends in a team barrier).  Units (range-major,
// the last range possibly shorter) go to the blocks in contiguous runs; a unit costs its k-blocks plus about four
// k-blocks' worth of fixed work (accumulator read-back, ticket, partial sums written and re-read), and every further
// range of a block another prologue.
void td_choose_split(int tiles, int n_kb, int n_cta, int b_kb, int *n_split, int *kb_per_split) {
    int best_s = 0, best_k = 0;
    double best = 1e30;
    const int s_min = (n_kb + b_kb - 1) / b_kb;
    for (int s0 = s_min; s0 <= std::min(n_kb, 32); ++s0) {
        const int kbps = (n_kb + s0 - 1) / s0, s = (n_kb + kbps - 1) / kbps;
        if (kbps < 8 && s0 > s_min) break; // units of at least 128 KB of weights
        const long units = (long)s * tiles;
        double worst = 0;
        for (int b = 0; b < n_cta; ++b) {
            const long u0 = (long)b * units / n_cta, u1 = (long)(b + 1) * units / n_cta;
            double load = 0;
            int last_ks = -1;
            for (long u = u0; u < u1; ++u) {
                const int ks = (int)(u / tiles);
                load += std::min(n_kb, (ks + 1) * kbps) - ks * kbps + (s > 1 ? 4.0 : 1.0);
                if (ks != last_ks) { load += 24.0; last_ks = ks; }
            }
            worst = std::max(worst, load);
        }
        if (worst < best * 0.985) { best = worst; best_s = s; best_k = kbps; }
    }
    *n_split = best_s;
    *kb_per_split = best_k;
}

int td_setup(mdi_ctx *c) {
    const mdi_model_shape &s = c->s;
    const int K = c->K, d = s.d_model, hd = s.head_dim, H = s.n_head, qw = H * hd, kw = s.n_kv_head * hd, F = s.d_ff, V = s.vocab;
    const bool want = c->scheduler == 4;
    auto no = [&](const char *why) { return want ? fail(c, MDI_ERR_SHAPE, "tensor-core persistent scheduler: %s", why) : MDI_OK; };
    if (c->scheduler != 4) return MDI_OK;
    if (s.weight_dtype != MDI_DTYPE_BF16) return no("needs bf16 weights");
    if (c->gmax > TD_MAXB) return no("at most 8 samples per group");
    if (d % 64 || qw % 64 || F % 64) return no("d_model, n_head * head_dim and d_ff must be multiples of 64");
    if (hd != 32 && hd != 64 && hd != 128) return no("head_dim must be 32, 64 or 128");
    if (K > 32) return no("too many partitions");
    if (!tg_encoder()) return no("no tensor-map encoder (driver too old)");
    cudaDeviceProp prop;
    CU(cudaGetDeviceProperties(&prop, c->dev));
    const int n_sm = prop.multiProcessorCount;
    if (n_sm < K) return no("fewer SMs than partitions");
    // resident B operand: 32 k-blocks (2048 columns; 7 ring stages) for wide models, whose matrices then need fewer
    // ranges, else 16 (9 ring stages)
    c->td_b_kb = c->o.td_b_kblocks > 0 ? c->o.td_b_kblocks : (d >= 2048 ? 32 : 16);
    if (c->td_b_kb < 4 || c->td_b_kb > 48) return no("td_b_kblocks must be between 4 and 48");
    c->td_smem = td_smem_layout().total;
    if (c->td_smem > (size_t)prop.sharedMemPerBlockOptin) return no("not enough shared memory per block");
    {
        cudaError_t ea = c->kv_kind == KV_F32 ? td_attr<float>(c->td_smem) : c->kv_kind == KV_F16 ? td_attr<__half>(c->td_smem) : td_attr<__nv_bfloat16>(c->td_smem);
        CU(ea);
    }
    for (int p = 0; p < K; ++p)
        if (5 * (c->part[p].hi - c->part[p].lo) + 1 > TD_MAX_PHASES) return no("too many blocks of the model in one partition");
    // a warp hands out the page-table entries of its sequence split by shuffles: a split may span at most 32 pages
    int min_att_split = 1;
    while (min_att_split < TD_MAX_SPLITS && (c->pages_per_seq + min_att_split - 1) / min_att_split + 2 > 32) min_att_split *= 2;
    if ((c->pages_per_seq + min_att_split - 1) / min_att_split + 2 > 32) return no("too many cache pages per sequence (use larger pages)");
    // team sizes in proportion to the bytes a partition step streams
    const double layer_bytes = 2.0 * ((double)(qw + 2 * kw) * d + (double)d * qw + (double)(s.act == MDI_ACT_SWIGLU ? 3 : 2) * F * d);
    std::vector<double> bytes(K);
    double tot = 0;
    for (int p = 0; p < K; ++p) {
        bytes[p] = layer_bytes * (c->part[p].hi - c->part[p].lo) + (p == K - 1 ? 2.0 * V * d : 0.0);
        tot += bytes[p];
    }
    std::vector<int> n_cta(K);
    int used = 0, big = 0;
    for (int p = 0; p < K; ++p) if (bytes[p] > bytes[big]) big = p;
    for (int p = 0; p < K; ++p) {
        if (p == big) continue;
        n_cta[p] = std::max(1, (int)std::floor(n_sm * bytes[p] / tot));
        used += n_cta[p];
    }
    if (n_sm - used < 1) return no("not enough SMs");
    n_cta[big] = n_sm - used;
    // phases (addresses follow in td_build)
    c->td_phases_host.clear();
    c->td_teams_host.assign(K, TdTeam{});
    c->td_phase_begin.assign(K, 0);
    c->td_phase_count.assign(K, 0);
    int first = 0;
    bool too_wide = false;
    for (int p = 0; p < K; ++p) {
        const int n = n_cta[p], Lp = c->part[p].hi - c->part[p].lo;
        c->td_phase_begin[p] = (int)c->td_phases_host.size();
        auto gemm = [&](int kind, int ll, int n_mat, int rows, int Kd, int pro) {
            TdPhase q{};
            q.kind = kind; q.layer_local = ll; q.n_mat = n_mat; q.n_rows = rows; q.K = Kd; q.pro = pro;
            q.n_tiles = (rows + TG_BM - 1) / TG_BM; q.n_kb = Kd / TG_BK;
            td_choose_split(n_mat * q.n_tiles, q.n_kb, n, c->td_b_kb, &q.n_split, &q.kb_per_split);
            if (q.n_split < 1) too_wide = true;
            q.n_units = q.n_split * n_mat * q.n_tiles;
            c->td_phases_host.push_back(q);
        };
        for (int l = 0; l < Lp; ++l) {
            gemm(TD_QKV, l, 1, qw + 2 * kw, d, TDP_NORM);
            c->td_phases_host.back().first_of_step = l == 0;
            TdPhase a{}; a.kind = TD_ATTN; a.layer_local = l; c->td_phases_host.push_back(a);
            gemm(TD_OUT, l, 1, d, qw, TDP_COPY);
            gemm(TD_UP, l, s.act == MDI_ACT_SWIGLU ? 2 : 1, F, d, TDP_NORM);
            gemm(TD_DOWN, l, 1, d, F, TDP_ACT);
        }
        if (p == K - 1) gemm(TD_HEAD, Lp, 1, V, d, TDP_NORM);
        c->td_phase_count[p] = (int)c->td_phases_host.size() - c->td_phase_begin[p];
        TdTeam &T = c->td_teams_host[p];
        T.first_cta = first; T.n_cta = n; first += n;
        T.phase_begin = c->td_phase_begin[p]; T.n_phases = c->td_phase_count[p];
        T.is_first = p == 0; T.is_last = p == K - 1;
        // attention units (sample, head, split) over the team's warps: the split count that deals them out most evenly
        {
            // estimated time of the phase: units of the busiest warp x (fixed cost of a unit: its q/k/v rows, page-table
            // entries, ticket, about four round trips to memory + a round trip per 16 cached rows), at a quarter of n_ctx
            const int warps = n * TD_CWARPS, pairs = c->gmax * H;
            int best_s = min_att_split;
            double best = 1e30;
            for (int sp = min_att_split; sp <= TD_MAX_SPLITS; sp *= 2) {
                const long units = (long)pairs * sp, most = (units + warps - 1) / warps;
                const double cost = (double)most * (4.0 + (double)(s.n_ctx / 4) / sp / 16.0);
                if (cost < best * 0.97) { best = cost; best_s = sp; }
            }
            T.n_att_split = best_s;
        }
    }
    c->td_grid = first;
    if (too_wide) return no("a matrix has more columns than 32 ranges of the resident B operand cover");
    int rc;
    if ((rc = dalloc(c, &c->td_sync, (size_t)K * 64)) != MDI_OK) return rc;
    if ((rc = dalloc(c, &c->td_err, 1)) != MDI_OK) return rc;
    if (c->o.in_kernel_timing && (rc = dalloc(c, &c->td_prof, (size_t)c->td_grid * PK_PROF_N)) != MDI_OK) return rc;
    c->td_ok = true;
    return MDI_OK;
}

// Scratch, tensor maps and phase tables; runs before the first launch and again after weights were replaced.
int td_build(mdi_ctx *c) {
    if (!c->td_stale) return MDI_OK;
    const mdi_model_shape &s = c->s;
    const int K = c->K, d = s.d_model, hd = s.head_dim, H = s.n_head, qw = H * hd, kw = s.n_kv_head * hd, F = s.d_ff, V = s.vocab;
    void *old[] = {c->td_teams, c->td_phases, c->td_maps, c->td_buf, c->td_ints};
    for (void *q : old) if (q) cudaFree(q);
    c->td_teams = nullptr; c->td_phases = nullptr; c->td_maps = nullptr; c->td_buf = nullptr; c->td_ints = nullptr;
    // one allocation for all float scratch and one for all integers: first count, then carve
    std::vector<CUtensorMap> maps;
    size_t floats = 0, ints = 0;
    auto take = [&](size_t n) { const size_t r = floats; floats += (n + 3) & ~(size_t)3; return r; };
    auto take_i = [&](size_t n) { const size_t r = ints; ints += (n + 3) & ~(size_t)3; return r; };
    struct Off { size_t x0, x1, qkv, u, att_part, att_out, att_ticket, head_pv, head_pi; std::vector<size_t> part, ticket; };
    std::vector<Off> offs(K);
    for (int p = 0; p < K; ++p) {
        Off &o = offs[p];
        const TdTeam &T = c->td_teams_host[p];
        o.x0 = take((size_t)TD_MAXB * d);
        o.x1 = take((size_t)TD_MAXB * d);
        o.qkv = take((size_t)TD_MAXB * (qw + 2 * kw));
        o.u = take((size_t)2 * TD_MAXB * F);
        o.att_part = take((size_t)TD_MAXB * H * T.n_att_split * (hd + 4));
        o.att_out = take((size_t)TD_MAXB * qw);
        o.att_ticket = take_i((size_t)TD_MAXB * H);
        o.head_pv = o.head_pi = 0;
        for (int i = 0; i < c->td_phase_count[p]; ++i) {
            const TdPhase &q = c->td_phases_host[c->td_phase_begin[p] + i];
            const bool split = td_is_gemm(q.kind) && q.n_split > 1;
            o.part.push_back(split ? take((size_t)q.n_mat * q.n_split * TD_MAXB * q.n_rows) : 0);
            o.ticket.push_back(split ? take_i((size_t)q.n_mat * q.n_tiles * 4) : 0);
            if (q.kind == TD_HEAD) { o.head_pv = take((size_t)TD_MAXB * 4 * q.n_tiles); o.head_pi = take_i((size_t)TD_MAXB * 4 * q.n_tiles); }
        }
    }
    c->td_buf_bytes = (int64_t)floats * 4 + (int64_t)ints * 4;
    c->td_n_ints = ints;
    CU(cudaMalloc((void **)&c->td_buf, std::max<size_t>(floats, 4) * 4));
    CU(cudaMemset(c->td_buf, 0, std::max<size_t>(floats, 4) * 4));
    CU(cudaMalloc((void **)&c->td_ints, std::max<size_t>(ints, 4) * 4));
    CU(cudaMemset(c->td_ints, 0, std::max<size_t>(ints, 4) * 4));
    auto add_map = [&](const void *W, int rows, int cols, int *idx) -> int {
        CUtensorMap m;
        const CUresult r = tg_make_map(&m, W, (uint64_t)rows, (uint64_t)cols, TG_BM);
        if (r != CUDA_SUCCESS) return fail(c, MDI_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) for a %d x %d matrix", (int)r, rows, cols);
        *idx = (int)maps.size();
        maps.push_back(m);
        return MDI_OK;
    };
    std::vector<std::pair<int, int>> map_idx(c->td_phases_host.size(), {-1, -1});
    for (int p = 0; p < K; ++p) {
        Partition &P = c->part[p];
        for (int i = 0; i < c->td_phase_count[p]; ++i) {
            const int gi = c->td_phase_begin[p] + i;
            TdPhase &q = c->td_phases_host[gi];
            if (!td_is_gemm(q.kind)) continue;
            int rc = MDI_OK;
            if (q.kind == TD_HEAD) rc = add_map(s.tied_lm_head ? c->wte : c->lm_head, V, d, &map_idx[gi].first);
            else {
                const LayerW &L = c->layer[P.lo + q.layer_local];
                if (q.kind == TD_QKV) rc = add_map(L.wqkv, qw + 2 * kw, d, &map_idx[gi].first);
                else if (q.kind == TD_OUT) rc = add_map(L.wo, d, qw, &map_idx[gi].first);
                else if (q.kind == TD_UP && s.act == MDI_ACT_SWIGLU) {
                    rc = add_map(L.wgate, F, d, &map_idx[gi].first);
                    if (rc == MDI_OK) rc = add_map(L.wup, F, d, &map_idx[gi].second);
                } else if (q.kind == TD_UP) rc = add_map(L.w1, F, d, &map_idx[gi].first);
                else rc = add_map(s.act == MDI_ACT_SWIGLU ? L.wdown : L.w2, d, F, &map_idx[gi].first);
            }
            if (rc != MDI_OK) return rc;
        }
    }
    CU(cudaMalloc((void **)&c->td_maps, std::max<size_t>(maps.size(), 1) * sizeof(CUtensorMap)));
    CU(cudaMemcpy(c->td_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice));
    for (int p = 0; p < K; ++p) {
        Partition &P = c->part[p];
        const Off &o = offs[p];
        float *x0 = c->td_buf + o.x0, *x1 = c->td_buf + o.x1, *qkv = c->td_buf + o.qkv, *u = c->td_buf + o.u;
        const int Lp = P.hi - P.lo;
        for (int i = 0; i < c->td_phase_count[p]; ++i) {
            const int gi = c->td_phase_begin[p] + i;
            TdPhase &q = c->td_phases_host[gi];
            const int ll = q.layer_local;
            if (td_is_gemm(q.kind)) {
                q.wmap[0] = map_idx[gi].first >= 0 ? c->td_maps + map_idx[gi].first : nullptr;
                q.wmap[1] = map_idx[gi].second >= 0 ? c->td_maps + map_idx[gi].second : nullptr;
                q.part = q.n_split > 1 ? c->td_buf + o.part[i] : nullptr;
                q.ticket = q.n_split > 1 ? c->td_ints + o.ticket[i] : nullptr;
            }
            const LayerW *L = ll < Lp ? &c->layer[P.lo + ll] : nullptr;
            switch (q.kind) {
                case TD_QKV:   // input: the residual stream entering the block (ring slot or embedding for the first block)
                    q.src = x0; q.dst = (p == 0 && ll == 0) ? x0 : nullptr; q.gamma = L->ln1g; q.beta = L->ln1b;
                    q.fin = qkv; q.fin_bias = s.has_bias ? L->bqkv : nullptr;
                    break;
                case TD_ATTN:
                    q.src = qkv;
                    break;
                case TD_OUT:   // x1 = x0 + bo + Wo . attention
                    q.src = c->td_buf + o.att_out;
                    q.fin = x1; q.fin_bias = s.has_bias ? L->bo : nullptr;
                    q.fin_resid = x0; q.fin_resid_ring = (ll == 0 && p > 0) ? 1 : 0;
                    break;
                case TD_UP:
                    q.src = x1; q.gamma = L->ln2g; q.beta = L->ln2b;
                    q.fin = u; q.fin_bias = s.has_bias ? L->b1 : nullptr;
                    break;
                case TD_DOWN:  // x0 (or the ring slot after the partition's last block) = x1 + b2 + W2 . hidden
                    q.src = u;
                    q.fin = x0; q.fin_bias = s.has_bias ? L->b2 : nullptr; q.fin_resid = x1;
                    q.fin_ring = (ll == Lp - 1 && p < K - 1) ? 1 : 0;
                    break;
                default:       // TD_HEAD
                    q.src = x0; q.gamma = c->lnfg; q.beta = c->lnfb;
                    break;
            }
        }
        TdTeam &T = c->td_teams_host[p];
        T.kv = kv_view(c, P);
        T.ring_in = p > 0 ? c->part[p - 1].ring : nullptr;
        T.ring_out = p < K - 1 ? P.ring : nullptr;
        T.att_part = c->td_buf + o.att_part;
        T.att_out = c->td_buf + o.att_out;
        T.att_ticket = c->td_ints + o.att_ticket;
        T.head_pv = p == K - 1 ? c->td_buf + o.head_pv : nullptr;
        T.head_pi = p == K - 1 ? c->td_ints + o.head_pi : nullptr;
        T.pos = P.pos_dev;
        T.bar = c->td_sync + (size_t)p * 64;
        T.flag_out = c->td_sync + (size_t)p * 64 + 32;
        T.flag_in = c->td_sync + (size_t)((p + K - 1) % K) * 64 + 32;
    }
    CU(cudaMalloc((void **)&c->td_teams, sizeof(TdTeam) * K));
    CU(cudaMemcpy(c->td_teams, c->td_teams_host.data(), sizeof(TdTeam) * K, cudaMemcpyHostToDevice));
    CU(cudaMalloc((void **)&c->td_phases, sizeof(TdPhase) * c->td_phases_host.size()));
    CU(cudaMemcpy(c->td_phases, c->td_phases_host.data(), sizeof(TdPhase) * c->td_phases_host.size(), cudaMemcpyHostToDevice));
    c->td_stale = false;
    return MDI_OK;
}

int td_launch(mdi_ctx *c, int n_samples, int G, int n_pass) {
    const mdi_model_shape &s = c->s;
    int rc = td_build(c);
    if (rc != MDI_OK) return rc;
    CU(cudaMemsetAsync(c->td_sync, 0, (size_t)c->K * 64 * sizeof(unsigned), c->main));
    CU(cudaMemsetAsync(c->td_err, 0, sizeof(int), c->main));
    CU(cudaMemsetAsync(c->td_ints, 0, std::max<size_t>(c->td_n_ints, 4) * 4, c->main)); // tickets start at zero (a timed-out call may have left some)
    if (c->td_prof) CU(cudaMemsetAsync(c->td_prof, 0, (size_t)c->td_grid * PK_PROF_N * 8, c->main));
    TdParams P{};
    P.d = s.d_model; P.n_head = s.n_head; P.n_kv_head = s.n_kv_head; P.head_dim = s.head_dim; P.d_ff = s.d_ff; P.vocab = s.vocab;
    P.norm = s.arch == MDI_ARCH_GPT ? NORM_LAYER : NORM_RMS; P.act = s.act; P.rope = s.arch == MDI_ARCH_LLAMA;
    P.K = c->K; P.G = G; P.n_samples = n_samples; P.gmax = c->gmax; P.n_pass = n_pass; P.b_kb = c->td_b_kb;
    P.eps = s.norm_eps; P.scale = 1.0f / std::sqrt((float)s.head_dim);
    P.teams = c->td_teams; P.phases = c->td_phases; P.wte = c->wte; P.wpe = c->wpe; P.rope_cos = c->rope_cos; P.rope_sin = c->rope_sin;
    P.logits = c->logits; P.cur_tok = c->cur_tok; P.tok_log = c->tok_log;
    P.gen_count = c->gen_count; P.teacher = c->teacher; P.n_teacher = c->n_teacher; P.log_stride = s.n_ctx; P.err = c->td_err;
    P.wait_ns = c->o.wait_limit_ms > 0 ? (unsigned long long)c->o.wait_limit_ms * 1000000ull : PK_WAIT_NS;
    P.withhold_partition = c->withhold_once;
    c->withhold_once = -1;
    P.prof = c->td_prof;
    void *args[] = {&P};
    CU(cudaFuncSetAttribute(td_func(c), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->td_smem)); // per function, not per context
    CU(cudaLaunchCooperativeKernel(td_func(c), dim3(c->td_grid), dim3(TD_THREADS), args, c->td_smem, c->main));
    ++c->st.kernel_launches;
    c->st.stage_steps += (int64_t)c->K * n_pass * G;
    return MDI_OK;
}

} // namespace

// Used by entry points that take no context (other files of the library): text for mdi_last_error(NULL).
void mdi_internal_set_error(const char *text) { g_create_error = text ? text : ""; }

// ====================================================================================================
extern "C" {

const char *mdi_last_error(mdi_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

void mdi_destroy(mdi_ctx *c) {
    if (!c) return;
    cudaSetDevice(c->dev);
    cudaDeviceSynchronize();
    for (auto &g : c->graphs) if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
    for (auto &t : c->w_tiled) if (t.second) cudaFree(t.second);
    for (auto &t : c->tensors) {
        if (t.second.mat && *t.second.mat) cudaFree(*t.second.mat);
        if (t.second.vec && *t.second.vec) cudaFree(*t.second.vec);
    }
    for (auto &P : c->part) {
        void *ptrs[] = {P.kv_pool, P.pt_dev, P.pos_dev, P.x_embed, P.qbuf, P.obuf, P.hbuf, P.part, P.x_last, P.attn_ticket,
                        P.ring, P.pf_buf[0], P.pf_buf[1], P.pf_hi, P.pf_lo, P.pf_qkv, P.pf_q, P.pf_o, P.pf_h, P.pf_u, P.pf_xa, P.pf_xb, P.pf_part};
        for (void *q : ptrs) if (q) cudaFree(q);
        for (auto e : P.ev_edge) cudaEventDestroy(e);
        for (auto e : P.ev_edge_cap) cudaEventDestroy(e);
        for (int i = 0; i < 2; ++i) { if (P.ev_pf_out[i]) cudaEventDestroy(P.ev_pf_out[i]); if (P.ev_pf_used[i]) cudaEventDestroy(P.ev_pf_used[i]); }
        if (P.ev_join) cudaEventDestroy(P.ev_join);
        if (P.ev_join_cap) cudaEventDestroy(P.ev_join_cap);
        if (P.stream) cudaStreamDestroy(P.stream);
    }
    void *ptrs[] = {c->rope_cos, c->rope_sin, c->logits, c->head_pv, c->head_y, c->head_pi, c->head_ticket, c->cur_tok, c->tok_log,
                    c->gen_count, c->teacher, c->n_teacher, c->prompt_buf, c->pk_teams, c->pk_phases, c->pk_sync, c->pk_err, c->pk_prof, c->tg_err,
                    c->fz_teams, c->fz_phases, c->fz_works, c->fz_blocks, c->fz_segs, c->fz_units, c->fz_err, c->fz_stream, c->fz_acc, c->fz_sync, c->fz_prof, c->fz_trace,
                    c->td_teams, c->td_phases, c->td_maps, c->td_buf, c->td_ints, c->td_sync, c->td_err, c->td_prof};
    for (void *q : ptrs) if (q) cudaFree(q);
    cudaEvent_t evs[] = {c->ev_fork, c->ev_fork_cap, c->ev_t0, c->ev_t1, c->ev_pf0, c->ev_pf1};
    for (auto e : evs) if (e) cudaEventDestroy(e);
    if (c->main) cudaStreamDestroy(c->main);
    delete c;
}

int mdi_create(const mdi_model_shape *shape, const int *part_bounds, int K, int n_samples, const mdi_options *opts,
               mdi_ctx **out) {
    mdi_ctx *c = nullptr;
    if (!shape || !part_bounds || !out) return fail(c, MDI_ERR_ARG, "null argument");
    *out = nullptr;
    const mdi_model_shape &s = *shape;
    if (K < 1 || n_samples < 1) return fail(c, MDI_ERR_ARG, "K and n_samples must be positive");
    if (part_bounds[0] != 0 || part_bounds[K] != s.n_layer) return fail(c, MDI_ERR_ARG, "partition bounds must run from 0 to n_layer");
    for (int p = 0; p < K; ++p)
        if (part_bounds[p + 1] <= part_bounds[p]) return fail(c, MDI_ERR_ARG, "partition bounds must be strictly ascending");
    if (s.arch != MDI_ARCH_GPT && s.arch != MDI_ARCH_LLAMA) return fail(c, MDI_ERR_ARG, "unknown arch");
    if (s.weight_dtype != MDI_DTYPE_F32 && s.weight_dtype != MDI_DTYPE_BF16) return fail(c, MDI_ERR_ARG, "unknown weight dtype");
    if (s.act < 0 || s.act > 2) return fail(c, MDI_ERR_ARG, "unknown activation");
    if (s.n_layer < 1 || s.d_model < 1 || s.n_head < 1 || s.n_kv_head < 1 || s.d_ff < 1 || s.vocab < 1 || s.n_ctx < 1)
        return fail(c, MDI_ERR_ARG, "non-positive dimension");
    if ((s.arch == MDI_ARCH_LLAMA) != (s.act == MDI_ACT_SWIGLU)) return fail(c, MDI_ERR_SHAPE, "SwiGLU goes with the Llama block, GELU with the GPT block");
    if (s.arch == MDI_ARCH_LLAMA && (s.has_bias || s.tied_lm_head)) return fail(c, MDI_ERR_SHAPE, "Llama block: no biases, untied output layer");
    if (s.arch == MDI_ARCH_GPT && !s.has_bias) return fail(c, MDI_ERR_SHAPE, "GPT block: biases required");
    const int vec = s.weight_dtype == MDI_DTYPE_F32 ? 4 : 8;
    if (s.head_dim != 16 && s.head_dim != 32 && s.head_dim != 64 && s.head_dim != 128)
        return fail(c, MDI_ERR_SHAPE, "head_dim must be 16, 32, 64 or 128");
    if (s.n_head % s.n_kv_head) return fail(c, MDI_ERR_SHAPE, "n_head must be a multiple of n_kv_head");
    if (s.d_model % vec || s.d_ff % vec || (s.n_head * s.head_dim) % vec)
        return fail(c, MDI_ERR_SHAPE, "d_model, d_ff and n_head*head_dim must be multiples of %d", vec);
    if ((size_t)std::max(s.d_model, s.d_ff) * 4 > LIN_SMEM_MAX) return fail(c, MDI_ERR_SHAPE, "layer width too large");

    c = new mdi_ctx();
    c->s = s;
    if (opts) c->o = *opts;
    c->K = K;
    c->S = n_samples;
    cudaError_t e = cudaGetDevice(&c->dev);
    if (e != cudaSuccess) { int rc = fail(nullptr, MDI_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(e)); delete c; return rc; }
    auto bail = [&](int rc) { g_create_error = c->err; mdi_destroy(c); return rc; };
    int rc;
#define TRY(x) do { if ((rc = (x)) != MDI_OK) return bail(rc); } while (0)
#define CUB(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return bail(fail(c, e_ == cudaErrorMemoryAllocation ? MDI_ERR_OOM : MDI_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_))); } while (0)

    // default page: 16 rows; 128 rows where the fused-phase kernel can run (GPT block, bf16 weights, fp32 cache), which
    // copies one head's rows of a page with one bulk copy each for keys and values and wants those copies large
    {
        const bool fused_candidate = s.arch == MDI_ARCH_GPT && s.weight_dtype == MDI_DTYPE_BF16 &&
                                     (c->o.kv_cache_dtype == MDI_KV_DEFAULT || c->o.kv_cache_dtype == MDI_KV_F32) &&
                                     s.n_kv_head == s.n_head && c->o.scheduler != 1 && c->o.scheduler != 2 && c->o.scheduler != 4 && s.head_dim <= 64;
        // ... and 64 rows where the tensor-core persistent kernel may run (a warp hands out the page-table entries of
        // its sequence split by shuffles: fewer, larger pages)
        const bool td_candidate = s.weight_dtype == MDI_DTYPE_BF16 && c->o.scheduler == 4;
        c->page_tokens = c->o.page_tokens > 0 ? c->o.page_tokens : (fused_candidate ? 128 : td_candidate ? 64 : 16);
    }
    if (c->page_tokens & (c->page_tokens - 1)) return bail(fail(c, MDI_ERR_ARG, "page_tokens must be a power of two"));
    c->page_shift = 0;
    while ((1 << c->page_shift) < c->page_tokens) ++c->page_shift;
    c->pages_per_seq = (s.n_ctx + c->page_tokens - 1) / c->page_tokens;
    c->esize = s.weight_dtype == MDI_DTYPE_F32 ? 4 : 2;
    if (c->o.kv_cache_dtype < 0 || c->o.kv_cache_dtype > 3) return bail(fail(c, MDI_ERR_ARG, "kv_cache_dtype must be one of MDI_KV_*"));
    {
        // default: fp16 for bf16 models outside the fused-phase kernel's reach (that kernel reads fp32 pages), else fp32
        const bool fused_shape = s.arch == MDI_ARCH_GPT && s.n_kv_head == s.n_head && s.d_model <= 1024 && s.head_dim <= 64;
        const int want = c->o.kv_cache_dtype != MDI_KV_DEFAULT ? c->o.kv_cache_dtype : (fused_shape ? MDI_KV_F32 : MDI_KV_F16);
        c->kv_kind = s.weight_dtype != MDI_DTYPE_BF16 ? KV_F32 : want == MDI_KV_BF16 ? KV_BF16 : want == MDI_KV_F16 ? KV_F16 : KV_F32;
    }
    c->kv_f32 = c->kv_kind == KV_F32;
    c->kv_esize = c->kv_f32 ? 4 : 2;
    c->page_elems = (size_t)2 * s.n_kv_head * c->page_tokens * s.head_dim;
    c->n_split = c->o.attn_splits > 0 ? c->o.attn_splits : std::max(1, std::min(16, s.n_ctx / 128));
    c->rounds_per_graph = c->o.rounds_per_graph != 0 ? c->o.rounds_per_graph : 16;
    if (c->o.prefill_mode < 0 || c->o.prefill_mode > 1) return bail(fail(c, MDI_ERR_ARG, "prefill_mode must be 0 or 1"));
    if (c->o.debug_withhold_handoff < 0 || c->o.debug_withhold_handoff > K) return bail(fail(c, MDI_ERR_ARG, "debug_withhold_handoff must name a partition (1-based) or be 0"));
    c->withhold_once = c->o.debug_withhold_handoff - 1;
    c->scheduler = c->o.scheduler;
    if (c->scheduler < 0 || c->scheduler > 4) return bail(fail(c, MDI_ERR_ARG, "scheduler must be 0, 1, 2, 3 or 4"));
    const int G = std::min(n_samples, K);
    c->gmax = (n_samples + G - 1) / G;
    const long pool_tokens = c->o.kv_pool_tokens > 0 ? c->o.kv_pool_tokens : (long)n_samples * s.n_ctx;

    CUB((lin_attr_all<float>()));
    CUB((lin_attr_all<__nv_bfloat16>()));
    CUB(cudaStreamCreateWithFlags(&c->main, cudaStreamNonBlocking));
    cudaEvent_t *evs[] = {&c->ev_fork, &c->ev_fork_cap};
    for (auto ev : evs) CUB(cudaEventCreateWithFlags(ev, cudaEventDisableTiming));
    cudaEvent_t *tevs[] = {&c->ev_t0, &c->ev_t1, &c->ev_pf0, &c->ev_pf1};
    for (auto ev : tevs) CUB(cudaEventCreate(ev));

    // tensors
    c->layer.resize(s.n_layer);
    const int d = s.d_model, F = s.d_ff, V = s.vocab, qw = s.n_head * s.head_dim, kw = s.n_kv_head * s.head_dim;
    auto part_of = [&](int l) { int p = 0; while (l >= part_bounds[p + 1]) ++p; return p; };
    auto mat = [&](const std::string &n, void **dst, size_t el, int p) { TensorSlot t; t.mat = dst; t.elems = el; t.partition = p; c->tensors[n] = t; };
    auto vecr = [&](const std::string &n, float **dst, size_t el, int p) { TensorSlot t; t.vec = dst; t.elems = el; t.partition = p; c->tensors[n] = t; };
    mat("wte", &c->wte, (size_t)V * d, 0);
    if (s.arch == MDI_ARCH_GPT) mat("wpe", &c->wpe, (size_t)s.n_ctx * d, 0);
    for (int i = 0; i < s.n_layer; ++i) {
        LayerW &L = c->layer[i];
        const std::string pfx = "h." + std::to_string(i) + ".";
        const int p = part_of(i);
        vecr(pfx + "ln1.g", &L.ln1g, d, p);
        if (s.arch == MDI_ARCH_GPT) vecr(pfx + "ln1.b", &L.ln1b, d, p);
        mat(pfx + "attn.wqkv", &L.wqkv, (size_t)(qw + 2 * kw) * d, p);
        if (s.has_bias) vecr(pfx + "attn.bqkv", &L.bqkv, qw + 2 * kw, p);
        mat(pfx + "attn.wo", &L.wo, (size_t)d * qw, p);
        if (s.has_bias) vecr(pfx + "attn.bo", &L.bo, d, p);
        vecr(pfx + "ln2.g", &L.ln2g, d, p);
        if (s.arch == MDI_ARCH_GPT) vecr(pfx + "ln2.b", &L.ln2b, d, p);
        if (s.act == MDI_ACT_SWIGLU) {
            mat(pfx + "mlp.wgate", &L.wgate, (size_t)F * d, p);
            mat(pfx + "mlp.wup", &L.wup, (size_t)F * d, p);
            mat(pfx + "mlp.wdown", &L.wdown, (size_t)d * F, p);
        } else {
            mat(pfx + "mlp.w1", &L.w1, (size_t)F * d, p);
            vecr(pfx + "mlp.b1", &L.b1, F, p);
            mat(pfx + "mlp.w2", &L.w2, (size_t)d * F, p);
            vecr(pfx + "mlp.b2", &L.b2, d, p);
        }
    }
    vecr("lnf.g", &c->lnfg, d, K - 1);
    if (s.arch == MDI_ARCH_GPT) vecr("lnf.b", &c->lnfb, d, K - 1);
    if (!s.tied_lm_head) mat("lm_head", &c->lm_head, (size_t)V * d, K - 1);

    // rotary tables, evaluated in fp64 on the host
    if (s.arch == MDI_ARCH_LLAMA) {
        const int half = s.head_dim / 2;
        std::vector<float> hc((size_t)s.n_ctx * half), hs((size_t)s.n_ctx * half);
        for (int pos = 0; pos < s.n_ctx; ++pos)
            for (int i = 0; i < half; ++i) {
                const double ang = (double)pos * std::pow((double)s.rope_theta, -2.0 * i / (double)s.head_dim);
                hc[(size_t)pos * half + i] = (float)std::cos(ang);
                hs[(size_t)pos * half + i] = (float)std::sin(ang);
            }
        TRY(dalloc(c, &c->rope_cos, hc.size()));
        TRY(dalloc(c, &c->rope_sin, hs.size()));
        CUB(cudaMemcpy(c->rope_cos, hc.data(), hc.size() * 4, cudaMemcpyHostToDevice));
        CUB(cudaMemcpy(c->rope_sin, hs.data(), hs.size() * 4, cudaMemcpyHostToDevice));
    }

    // partitions
    c->part.resize(K);
    for (int p = 0; p < K; ++p) {
        Partition &P = c->part[p];
        P.lo = part_bounds[p];
        P.hi = part_bounds[p + 1];
        const int Lp = P.hi - P.lo;
        CUB(cudaStreamCreateWithFlags(&P.stream, cudaStreamNonBlocking));
        // every sample may leave one page partly filled: with pages above 16 rows that slack is added to the pool
        const long pages_per_layer = (pool_tokens + c->page_tokens - 1) / c->page_tokens + (c->page_tokens > 16 ? n_samples : 0);
        P.n_pages = (int)(pages_per_layer * Lp);
        P.kv_bytes = (size_t)P.n_pages * c->page_elems * c->kv_esize;
        CUB(cudaMalloc(&P.kv_pool, std::max<size_t>(P.kv_bytes, 16)));
        CUB(cudaMemset(P.kv_pool, 0, std::max<size_t>(P.kv_bytes, 16)));
        P.free_pages.resize(P.n_pages);
        for (int i = 0; i < P.n_pages; ++i) P.free_pages[i] = P.n_pages - 1 - i;
        P.pt_host.assign((size_t)n_samples * Lp * c->pages_per_seq, 0);
        P.pages_of_slot.assign(n_samples, 0);
        P.pos_host.assign(n_samples, 0);
        TRY(dalloc(c, &P.pt_dev, P.pt_host.size(), &P.buffer_bytes));
        TRY(dalloc(c, &P.pos_dev, (size_t)n_samples, &P.buffer_bytes));
        if (p == 0) TRY(dalloc(c, &P.x_embed, (size_t)MAXB * d, &P.buffer_bytes));
        TRY(dalloc(c, &P.qbuf, (size_t)MAXB * qw, &P.buffer_bytes));
        TRY(dalloc(c, &P.obuf, (size_t)MAXB * qw, &P.buffer_bytes));
        TRY(dalloc(c, &P.hbuf, (size_t)MAXB * F, &P.buffer_bytes));
        TRY(dalloc(c, &P.part, (size_t)MAXB * s.n_head * std::max(c->n_split, 16) * (s.head_dim + 2), &P.buffer_bytes));
        TRY(dalloc(c, &P.attn_ticket, (size_t)MAXB * s.n_head, &P.buffer_bytes));
        TRY(dalloc(c, &P.x_last, (size_t)std::max(MAXB, c->gmax) * d, &P.buffer_bytes));
        if (p < K - 1) {
            TRY(dalloc(c, &P.ring, (size_t)G * c->gmax * d, &P.buffer_bytes));
            for (int i = 0; i < 2; ++i) TRY(dalloc(c, &P.pf_buf[i], (size_t)s.n_ctx * d, &P.buffer_bytes));
        }
        P.ev_edge.resize(G);
        P.ev_edge_cap.resize(G);
        for (int j = 0; j < G; ++j) {
            CUB(cudaEventCreateWithFlags(&P.ev_edge[j], cudaEventDisableTiming));
            CUB(cudaEventCreateWithFlags(&P.ev_edge_cap[j], cudaEventDisableTiming));
        }
        for (int i = 0; i < 2; ++i) {
            CUB(cudaEventCreateWithFlags(&P.ev_pf_out[i], cudaEventDisableTiming));
            CUB(cudaEventCreateWithFlags(&P.ev_pf_used[i], cudaEventDisableTiming));
        }
        CUB(cudaEventCreateWithFlags(&P.ev_join, cudaEventDisableTiming));
        CUB(cudaEventCreateWithFlags(&P.ev_join_cap, cudaEventDisableTiming));
    }
    for (auto &t : c->tensors) c->part[t.second.partition].weight_bytes += (int64_t)t.second.elems * (t.second.mat ? c->esize : 4);

    // output layers and token state
    const int head_units = (V + 1) / 2;
    c->head_grid = (head_units + LIN_WARPS - 1) / LIN_WARPS;
    int64_t *acc = &c->part[K - 1].buffer_bytes;
    TRY(dalloc(c, &c->logits, (size_t)n_samples * V, acc));
    TRY(dalloc(c, &c->head_pv, (size_t)MAXB * std::max(c->head_grid, 1024), acc));
    TRY(dalloc(c, &c->head_pi, (size_t)MAXB * std::max(c->head_grid, 1024), acc));
    TRY(dalloc(c, &c->head_ticket, 1, acc));
    if (s.weight_dtype == MDI_DTYPE_BF16 && c->o.prefill_mode != 1) TRY(dalloc(c, &c->head_y, (size_t)MAXB * V, acc));
    TRY(dalloc(c, &c->cur_tok, (size_t)n_samples));
    TRY(dalloc(c, &c->gen_count, (size_t)n_samples));
    TRY(dalloc(c, &c->n_teacher, (size_t)n_samples));
    TRY(dalloc(c, &c->tok_log, (size_t)n_samples * s.n_ctx));
    TRY(dalloc(c, &c->teacher, (size_t)n_samples * s.n_ctx));
    TRY(dalloc(c, &c->prompt_buf, (size_t)n_samples * s.n_ctx));
    c->gen_host.assign(n_samples, 0);
    c->returned_host.assign(n_samples, 0);
    c->prefilled.assign(n_samples, 0);
    TRY(pk_setup(c));
    TRY(pf_setup(c));
    TRY(fz_setup(c));
    TRY(td_setup(c));
    CUB(cudaDeviceSynchronize());
#undef TRY
#undef CUB
    *out = c;
    return MDI_OK;
}

int mdi_load_weights(mdi_ctx *c, const char *name, const void *host, size_t nbytes) {
    if (!c || !name || !host) return fail(c, MDI_ERR_ARG, "null argument");
    auto it = c->tensors.find(name);
    if (it == c->tensors.end()) return fail(c, MDI_ERR_ARG, "unknown tensor '%s'", name);
    TensorSlot &t = it->second;
    if (nbytes != t.elems * c->esize) return fail(c, MDI_ERR_SHAPE, "tensor '%s': %zu bytes given, %zu expected", name, nbytes, t.elems * c->esize);
    CU(cudaSetDevice(c->dev));
    if (t.mat) {
        if (!*t.mat) CU(cudaMalloc(t.mat, nbytes));
        CU(cudaMemcpy(*t.mat, host, nbytes, cudaMemcpyHostToDevice));
    } else {
        std::vector<float> f(t.elems);
        if (c->s.weight_dtype == MDI_DTYPE_F32) memcpy(f.data(), host, nbytes);
        else {
            const uint16_t *h = (const uint16_t *)host;
            for (size_t i = 0; i < t.elems; ++i) { uint32_t u = (uint32_t)h[i] << 16; memcpy(&f[i], &u, 4); }
        }
        if (!*t.vec) CU(cudaMalloc((void **)t.vec, t.elems * 4));
        CU(cudaMemcpy(*t.vec, f.data(), t.elems * 4, cudaMemcpyHostToDevice));
    }
    if (!t.loaded) { t.loaded = true; ++c->n_loaded; }
    c->pk_tables_stale = true;
    c->fz_stale = true;
    c->td_stale = true;
    c->tiles_stale = true;
    return MDI_OK;
}

int mdi_reset_sample(mdi_ctx *c, int sample) {
    if (!c) return MDI_ERR_ARG;
    if (sample < 0 || sample >= c->S) return fail(c, MDI_ERR_ARG, "sample %d out of range", sample);
    CU(cudaSetDevice(c->dev));
    // No device-wide wait: mdi_generate returns only when its work is done, and whatever a first visit or mdi_step
    // has left on a partition's stream precedes, on that same stream, both the clearing below and any later work
    // that could take over the pages given back here (a partition's pool is only ever touched from its stream, or
    // from a persistent launch that waits for all partition streams).
    const int K = c->K;
    for (auto &P : c->part) {
        const int Lp = P.hi - P.lo;
        for (int l = 0; l < Lp; ++l)
            for (int g = 0; g < P.pages_of_slot[sample]; ++g) {
                int &pg = P.pt_host[((size_t)sample * Lp + l) * c->pages_per_seq + g];
                P.free_pages.push_back(pg);
                pg = 0;
            }
        P.pages_of_slot[sample] = 0;
        P.pos_host[sample] = 0;
        CU(cudaMemsetAsync(P.pos_dev + sample, 0, 4, P.stream));
    }
    // counters of the output layers: written by kernels of the last partition's stream
    CU(cudaMemsetAsync(c->gen_count + sample, 0, 4, c->part[K - 1].stream));
    CU(cudaMemsetAsync(c->n_teacher + sample, 0, 4, c->part[K - 1].stream));
    c->gen_host[sample] = c->returned_host[sample] = c->prefilled[sample] = 0;
    return MDI_OK;
}

int mdi_set_teacher_tokens(mdi_ctx *c, int sample, const int32_t *tok, int n) {
    if (!c) return MDI_ERR_ARG;
    if (sample < 0 || sample >= c->S || n < 0 || (n > 0 && !tok)) return fail(c, MDI_ERR_ARG, "bad argument");
    if (n > c->s.n_ctx) return fail(c, MDI_ERR_CONTEXT, "more teacher tokens than n_ctx");
    if (c->prefilled[sample]) return fail(c, MDI_ERR_STATE, "set teacher tokens before the sample's prefill");
    CU(cudaSetDevice(c->dev));
    // on the stream whose kernels read them (and after a preceding mdi_reset_sample's clearing on that stream)
    cudaStream_t st = c->part[c->K - 1].stream;
    if (n) CU(cudaMemcpyAsync(c->teacher + (size_t)sample * c->s.n_ctx, tok, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(c->n_teacher + sample, &n, 4, cudaMemcpyHostToDevice, st));
    CU(cudaStreamSynchronize(st));
    return MDI_OK;
}

static int prefill_impl(mdi_ctx *c, int sample, const int32_t *prompt, int n, bool on_device) {
    if (!c || !prompt) return fail(c, MDI_ERR_ARG, "null argument");
    if (sample < 0 || sample >= c->S || n < 1) return fail(c, MDI_ERR_ARG, "bad sample or prompt length");
    if (n > c->s.n_ctx) return fail(c, MDI_ERR_CONTEXT, "prompt of %d tokens exceeds n_ctx %d", n, c->s.n_ctx);
    if (c->prefilled[sample]) return fail(c, MDI_ERR_STATE, "sample %d already holds tokens", sample);
    for (auto &P : c->part) if (P.pos_host[sample]) return fail(c, MDI_ERR_STATE, "sample %d already holds tokens", sample);
    int rc = check_weights(c);
    if (rc != MDI_OK) return rc;
    CU(cudaSetDevice(c->dev));
    if (!on_device)
        for (int i = 0; i < n; ++i)
            if (prompt[i] < 0 || prompt[i] >= c->s.vocab) return fail(c, MDI_ERR_ARG, "token id %d out of range", prompt[i]);
    for (int p = 0; p < c->K; ++p) if ((rc = ensure_pages(c, p, sample, n)) != MDI_OK) return rc;
    const int d = c->s.d_model, K = c->K;
    int *pbuf = c->prompt_buf + (size_t)sample * c->s.n_ctx;
    CU(cudaMemcpyAsync(pbuf, prompt, (size_t)n * 4, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->part[0].stream));
    const int par = c->pf_count & 1;
    if (!c->pf_open) { CU(cudaEventRecord(c->ev_pf0, c->part[0].stream)); c->pf_open = true; }
    for (int p = 0; p < K; ++p) {
        Partition &P = c->part[p];
        if (p > 0) CU(cudaStreamWaitEvent(P.stream, c->part[p - 1].ev_pf_out[par], 0));
        if (p < K - 1 && c->part[p + 1].pf_used_valid[par]) CU(cudaStreamWaitEvent(P.stream, c->part[p + 1].ev_pf_used[par], 0));
        for (int c0 = 0; c->pf_tc && c0 < n; c0 += PF_CHUNK) {
            const int m = std::min(PF_CHUNK, n - c0);
            const float *x_in = p > 0 ? c->part[p - 1].pf_buf[par] + (size_t)c0 * d : nullptr;
            float *x_out = p < K - 1 ? P.pf_buf[par] + (size_t)c0 * d : P.pf_xb;
            if ((rc = pf_partition_chunk(c, p, sample, pbuf + c0, m, x_in, x_out, P.stream)) != MDI_OK) return rc;
            if (p == K - 1 && c0 + m == n) {
                Batch hb{};
                hb.n = 1; hb.slot[0] = sample;
                HeadReq hr;
                if ((rc = enqueue_head(c, hb, x_out + (size_t)(m - 1) * d, hr, P.stream)) != MDI_OK) return rc;
            }
        }
        for (int c0 = 0; !c->pf_tc && c0 < n; c0 += MAXB) {
            const int m = std::min(MAXB, n - c0);
            Batch bt{};
            bt.n = m;
            for (int i = 0; i < m; ++i) { bt.slot[i] = sample; bt.off[i] = i; bt.adv[i] = i == 0 ? m : 0; }
            const float *x_in = p > 0 ? c->part[p - 1].pf_buf[par] + (size_t)c0 * d : nullptr;
            float *x_out = p < K - 1 ? P.pf_buf[par] + (size_t)c0 * d : P.x_last;
            HeadReq hr;
            hr.item = m - 1;
            const bool last_chunk = c0 + m == n;
            rc = enqueue_partition_step(c, p, bt, x_in, pbuf + c0, 0, x_out, last_chunk ? &hr : nullptr, P.stream);
            if (rc != MDI_OK) return rc;
        }
        CU(cudaEventRecord(P.ev_pf_out[par], P.stream));
        if (p > 0) { CU(cudaEventRecord(P.ev_pf_used[par], P.stream)); P.pf_used_valid[par] = true; }
        P.pos_host[sample] += n;
    }
    CU(cudaEventRecord(c->ev_pf1, c->part[K - 1].stream));
    CU(cudaGetLastError());
    ++c->pf_count;
    c->prefilled[sample] = 1;
    c->gen_host[sample] = 1;
    c->returned_host[sample] = 0;
    ++c->st.tokens_generated;
    return MDI_OK;
}

int mdi_prefill(mdi_ctx *c, int sample, const int32_t *prompt_host, int n) { return prefill_impl(c, sample, prompt_host, n, false); }
int mdi_prefill_dev(mdi_ctx *c, int sample, const int32_t *prompt_dev, int n) { return prefill_impl(c, sample, prompt_dev, n, true); }

int mdi_step(mdi_ctx *c, int p, int slot, const void *act_in, void *act_out) {
    if (!c || !act_in || !act_out) return fail(c, MDI_ERR_ARG, "null argument");
    if (p < 0 || p >= c->K || slot < 0 || slot >= c->S) return fail(c, MDI_ERR_ARG, "partition or slot out of range");
    int rc = check_weights(c);
    if (rc != MDI_OK) return rc;
    CU(cudaSetDevice(c->dev));
    Partition &P = c->part[p];
    if (P.pos_host[slot] + 1 > c->s.n_ctx) return fail(c, MDI_ERR_CONTEXT, "slot %d is full (%d rows)", slot, P.pos_host[slot]);
    if ((rc = ensure_pages(c, p, slot, P.pos_host[slot] + 1)) != MDI_OK) return rc;
    Batch bt{};
    bt.n = 1; bt.slot[0] = slot; bt.off[0] = 0; bt.adv[0] = 1;
    HeadReq hr;
    hr.item = 0; hr.update_state = false; hr.tok_out = (int *)act_out;
    const bool last = p == c->K - 1;
    rc = enqueue_partition_step(c, p, bt, (const float *)act_in, (const int *)act_in, 0, last ? P.x_last : (float *)act_out,
                                last ? &hr : nullptr, P.stream);
    if (rc != MDI_OK) return rc;
    CU(cudaGetLastError());
    ++P.pos_host[slot];
    return MDI_OK;
}

// Enqueue ticks [t_begin, t_end) of the recurrent schedule.  The ring has K phase slots: at tick t
// partition p serves phase (t - p) mod K, pass (t - p) / K; phases 0..G-1 carry the G sample groups and
// the others are idle (fewer samples than partitions).  Handoffs whose producer lies before t_begin are
// already ordered by the fork at the start of the segment.
static int enqueue_ticks(mdi_ctx *c, int n_samples, int G, long t_begin, long t_end, long total_slots) {
    const int K = c->K, d = c->s.d_model;
    const bool cap = c->capturing;
    cudaEvent_t fork = cap ? c->ev_fork_cap : c->ev_fork;
    CU(cudaEventRecord(fork, c->main));
    for (int p = 0; p < K; ++p) CU(cudaStreamWaitEvent(c->part[p].stream, fork, 0));
    for (long t = t_begin; t < t_end; ++t)
        for (int p = 0; p < K; ++p) {
            const long v = t - p;
            if (v < 0 || v >= total_slots) continue;
            const int j = (int)(v % K);
            if (j >= G) continue;
            Partition &P = c->part[p];
            const int prev = (p + K - 1) % K;
            // producer of this step's input: partition p-1 one tick earlier (for p = 0: the last partition,
            // which chose the token; none on a group's first pass of this call)
            const bool has_producer = p > 0 || v >= K;
            if (has_producer && t - 1 >= t_begin && K > 1)
                CU(cudaStreamWaitEvent(P.stream, cap ? c->part[prev].ev_edge_cap[j] : c->part[prev].ev_edge[j], 0));
            // the group's samples, in sub-batches of at most MAXB
            std::vector<int> members;
            for (int smp = j; smp < n_samples; smp += G) members.push_back(smp);
            for (size_t first = 0; first < members.size(); first += MAXB) {
                const int m = (int)std::min<size_t>(MAXB, members.size() - first);
                Batch bt{};
                bt.n = m;
                for (int i = 0; i < m; ++i) { bt.slot[i] = members[first + i]; bt.off[i] = 0; bt.adv[i] = 1; }
                const float *x_in = p > 0 ? c->part[p - 1].ring + ((size_t)j * c->gmax + first) * d : nullptr;
                float *x_out = p < K - 1 ? P.ring + ((size_t)j * c->gmax + first) * d : P.x_last;
                HeadReq hr;
                int rc = enqueue_partition_step(c, p, bt, x_in, c->cur_tok, 1, x_out, &hr, P.stream);
                if (rc != MDI_OK) return rc;
            }
            CU(cudaEventRecord(cap ? P.ev_edge_cap[j] : P.ev_edge[j], P.stream));
        }
    for (int p = 0; p < K; ++p) {
        cudaEvent_t ej = cap ? c->part[p].ev_join_cap : c->part[p].ev_join;
        CU(cudaEventRecord(ej, c->part[p].stream));
        CU(cudaStreamWaitEvent(c->main, ej, 0));
    }
    return MDI_OK;
}

static int generate_impl(mdi_ctx *c, int n_samples, int n_new, int32_t *out, bool on_device) {
    if (!c || !out) return fail(c, MDI_ERR_ARG, "null argument");
    if (n_samples < 1 || n_samples > c->S || n_new < 0) return fail(c, MDI_ERR_ARG, "bad n_samples or n_new_tokens");
    int rc = check_weights(c);
    if (rc != MDI_OK) return rc;
    CU(cudaSetDevice(c->dev));
    const int K = c->K, G = std::min(n_samples, K);
    if ((n_samples + G - 1) / G > c->gmax) return fail(c, MDI_ERR_ARG, "group size exceeds what the context was created for");
    const int pending = c->gen_host[0] - c->returned_host[0];
    for (int smp = 0; smp < n_samples; ++smp) {
        if (!c->prefilled[smp]) return fail(c, MDI_ERR_STATE, "sample %d has not been prefilled", smp);
        if (c->gen_host[smp] - c->returned_host[smp] != pending) return fail(c, MDI_ERR_STATE, "samples are at different points of generation");
    }
    const int n_pass = std::max(0, n_new - pending);
    for (int smp = 0; smp < n_samples; ++smp) {
        if (c->part[0].pos_host[smp] + n_pass > c->s.n_ctx)
            return fail(c, MDI_ERR_CONTEXT, "sample %d: %d cached + %d new positions exceed n_ctx %d", smp, c->part[0].pos_host[smp], n_pass, c->s.n_ctx);
        if (c->gen_host[smp] + n_pass > c->s.n_ctx) return fail(c, MDI_ERR_CONTEXT, "token log full");
    }
    for (int p = 0; p < K; ++p)
        for (int smp = 0; smp < n_samples; ++smp)
            if ((rc = ensure_pages(c, p, smp, c->part[p].pos_host[smp] + n_pass)) != MDI_OK) return rc;

    // everything enqueued so far (prefills, page tables) precedes the schedule
    for (int p = 0; p < K; ++p) {
        CU(cudaEventRecord(c->part[p].ev_join, c->part[p].stream));
        CU(cudaStreamWaitEvent(c->main, c->part[p].ev_join, 0));
    }
    CU(cudaEventRecord(c->ev_t0, c->main));
    if ((rc = pf_check(c)) != MDI_OK) return rc;
    const long total = (long)n_pass * K;        // phase slots per partition
    const long t_total = total ? total + K - 1 : 0;
    // fused-phase kernel where the shape fits it, else the phase-per-matrix kernel, else streams
    const bool small_groups = c->temperature <= 0.f && (n_samples + G - 1) / G <= PK_MAXNB &&
                              !(c->pf_tc && c->scheduler == 0 && (n_samples + G - 1) / G >= c->tc_min_group);
    const bool use_fz = c->fz_ok && (c->scheduler == 0 || c->scheduler == 3) && small_groups && fz_slot_count_fits(c, n_pass, G);
    const bool use_pk = !use_fz && c->pk_ok && c->scheduler != 1 && c->scheduler != 3 && c->scheduler != 4 && small_groups && pk_tile_count_fits(c, n_pass, G);
    // the tensor-core persistent kernel: on request only (measured on the two large workloads it does not beat the
    // stream scheduler's tensor-core steps: its teams run their phases in lock-step, so the weight stream stops
    // during attention, prologues and barriers), greedy token choice
    const bool use_td = c->td_ok && c->scheduler == 4 && c->temperature <= 0.f && (n_samples + G - 1) / G <= TD_MAXB;
    if (c->scheduler == 2 && !use_pk) return fail(c, MDI_ERR_SHAPE, "persistent scheduler unavailable for this call");
    if (c->scheduler == 3 && !use_fz) return fail(c, MDI_ERR_SHAPE, "fused-phase scheduler unavailable for this call");
    if (c->scheduler == 4 && !use_td) return fail(c, MDI_ERR_SHAPE, "tensor-core persistent scheduler unavailable for this call");
    // From here on work is queued that advances positions and counters on the device; the host's copies follow only
    // once all of it has run.  A failure half-way leaves the two out of step, so it forgets every sample.
    auto enqueue_all = [&]() -> int {
        int rc = MDI_OK;
        long t = 0;
        if (t_total && use_fz) {
            if ((rc = fz_launch(c, n_samples, G, n_pass)) != MDI_OK) return rc;
            c->last_kernel = 2;
        } else if (t_total && use_pk) {
            if ((rc = pk_launch(c, n_samples, G, n_pass)) != MDI_OK) return rc;
            c->last_kernel = 1;
        } else if (t_total && use_td) {
            if ((rc = td_launch(c, n_samples, G, n_pass)) != MDI_OK) return rc;
            c->last_kernel = 3;
        } else if (t_total) {
            const int R = c->rounds_per_graph;
            const long t_steady = K > 1 ? K : 0; // first tick, multiple of K, from which every partition is in steady state
            // Steady-state windows are replayed from CUDA graphs: first windows of R rounds, then windows of one round
            // for what is left, so that at most a round (plus fill and drain) is launched kernel by kernel.
            bool started = false;
            for (int pass = 0; pass < 2 && R > 0; ++pass) {
                const long W = pass == 0 ? (long)R * K : (long)K;
                if (pass == 1 && R == 1) break;
                if ((started ? t : t_steady) + (pass == 0 ? 2 * W : W) > total) continue;
                if (!started) {
                    if ((rc = enqueue_ticks(c, n_samples, G, 0, t_steady, total)) != MDI_OK) return rc;
                    t = t_steady;
                    started = true;
                }
                auto key = std::make_pair(n_samples, (int)W);
                GraphEntry &ge = c->graphs[key];
                if (!ge.exec) {
                    cudaGraph_t graph = nullptr;
                    CU(cudaStreamBeginCapture(c->main, cudaStreamCaptureModeThreadLocal));
                    c->capturing = true;
                    c->cap_launches = c->cap_steps = 0;
                    rc = enqueue_ticks(c, n_samples, G, t_steady, t_steady + W, 1L << 60);
                    c->capturing = false;
                    cudaError_t e = cudaStreamEndCapture(c->main, &graph);
                    if (rc != MDI_OK) { if (graph) cudaGraphDestroy(graph); c->graphs.erase(key); return rc; }
                    if (e != cudaSuccess) { c->graphs.erase(key); return fail(c, MDI_ERR_CUDA, "graph capture: %s", cudaGetErrorString(e)); }
                    e = cudaGraphInstantiate(&ge.exec, graph, 0);
                    cudaGraphDestroy(graph);
                    if (e != cudaSuccess) { c->graphs.erase(key); return fail(c, MDI_ERR_CUDA, "graph instantiate: %s", cudaGetErrorString(e)); }
                    ge.launches = c->cap_launches;
                    ge.steps = c->cap_steps;
                }
                while (t + W <= total) {
                    CU(cudaGraphLaunch(ge.exec, c->main));
                    c->st.kernel_launches += ge.launches;
                    c->st.stage_steps += ge.steps;
                    t += W;
                }
            }
            if ((rc = enqueue_ticks(c, n_samples, G, t, t_total, total)) != MDI_OK) return rc;
        }
        CU(cudaEventRecord(c->ev_t1, c->main));
        CU(cudaGetLastError());
        // tokens: entries [returned, returned + n_new) of each sample's log
        for (int smp = 0; smp < n_samples && n_new; ++smp)
            CU(cudaMemcpyAsync(out + (size_t)smp * n_new, c->tok_log + (size_t)smp * c->s.n_ctx + c->returned_host[smp], (size_t)n_new * 4,
                               on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, c->main));
        CU(cudaStreamSynchronize(c->main));
        return MDI_OK;
    };
    auto forget_all = [&]() {
        cudaDeviceSynchronize();
        cudaGetLastError();
        for (int smp = 0; smp < c->S; ++smp) mdi_reset_sample(c, smp);
    };
    if ((rc = enqueue_all()) != MDI_OK) {
        const std::string why = c->err;
        forget_all();
        return fail(c, rc, "%s; all samples were reset", why.c_str());
    }
    if (t_total && (use_pk || use_fz || use_td)) {
        int kerr = 0;
        CU(cudaMemcpy(&kerr, use_fz ? c->fz_err : use_td ? c->td_err : c->pk_err, sizeof(int), cudaMemcpyDeviceToHost));
        if (kerr) {
            // the pipeline stopped half-way: positions, caches and counters no longer agree
            forget_all();
            return fail(c, MDI_ERR_TIMEOUT, "persistent decode kernel gave up waiting (code %d: 1 edge flag, 2 team barrier, 3 weight tile, 4 ring slot); all samples were reset", kerr);
        }
    }
    for (int smp = 0; smp < n_samples; ++smp) {
        for (int p = 0; p < K; ++p) c->part[p].pos_host[smp] += n_pass;
        c->gen_host[smp] += n_pass;
        c->returned_host[smp] += n_new;
        c->st.tokens_generated += n_pass;
    }
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->ev_t0, c->ev_t1) == cudaSuccess) c->st.last_generate_ms = ms;
    if (c->pf_open) {
        if (cudaEventElapsedTime(&ms, c->ev_pf0, c->ev_pf1) == cudaSuccess) c->st.last_prefill_ms = ms;
        if (cudaEventElapsedTime(&ms, c->ev_pf0, c->ev_t1) == cudaSuccess) c->st.last_run_ms = ms;
        c->pf_open = false;
    }
    return MDI_OK;
}

int mdi_generate(mdi_ctx *c, int n_samples, int n_new, int32_t *out_host) { return generate_impl(c, n_samples, n_new, out_host, false); }
int mdi_generate_dev(mdi_ctx *c, int n_samples, int n_new, int32_t *out_dev) { return generate_impl(c, n_samples, n_new, out_dev, true); }

int mdi_set_sampling(mdi_ctx *c, float temperature, int top_k, uint64_t seed) {
    if (!c) return MDI_ERR_ARG;
    if (temperature > 0.f && (top_k < 1 || top_k > 64)) return fail(c, MDI_ERR_ARG, "top_k must be between 1 and 64 when sampling");
    if (!(temperature == temperature)) return fail(c, MDI_ERR_ARG, "temperature is not a number");
    CU(cudaSetDevice(c->dev));
    CU(cudaDeviceSynchronize());
    // the captured windows of the stream scheduler carry the token-choice parameters in their kernel arguments
    for (auto &g : c->graphs) if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
    c->graphs.clear();
    c->temperature = temperature > 0.f ? temperature : 0.f;
    c->top_k = top_k;
    c->sample_seed = seed;
    return MDI_OK;
}

int mdi_get_logits(mdi_ctx *c, int sample, float *out_host) {
    if (!c || !out_host) return fail(c, MDI_ERR_ARG, "null argument");
    if (sample < 0 || sample >= c->S) return fail(c, MDI_ERR_ARG, "sample out of range");
    CU(cudaSetDevice(c->dev));
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(out_host, c->logits + (size_t)sample * c->s.vocab, (size_t)c->s.vocab * 4, cudaMemcpyDeviceToHost));
    return MDI_OK;
}

int mdi_sync(mdi_ctx *c) {
    if (!c) return MDI_ERR_ARG;
    CU(cudaSetDevice(c->dev));
    for (auto &P : c->part) CU(cudaStreamSynchronize(P.stream));
    CU(cudaStreamSynchronize(c->main));
    return pf_check(c);
}

int mdi_get_stats(mdi_ctx *c, mdi_stats *out) {
    if (!c || !out) return fail(c, MDI_ERR_ARG, "null argument");
    int rc = mdi_sync(c);
    if (rc != MDI_OK) return rc;
    if (c->pf_open) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->ev_pf0, c->ev_pf1) == cudaSuccess) c->st.last_prefill_ms = ms;
    }
    c->st.n_partitions = c->K;
    c->st.n_samples = c->S;
    c->st.n_groups = std::min(c->S, c->K);
    c->st.kv_element_bytes = (int)c->kv_esize;
    for (int p = 0; p < c->K && p < 16; ++p) {
        c->st.weight_bytes[p] = c->part[p].weight_bytes;
        c->st.kv_pool_bytes[p] = (int64_t)c->part[p].kv_bytes;
        c->st.kv_pages_in_use[p] = c->part[p].n_pages - (int64_t)c->part[p].free_pages.size();
    }
    *out = c->st;
    return MDI_OK;
}

int mdi_get_partition_times(mdi_ctx *c, int p, double *out_ms, int n) {
    if (!c || !out_ms) return fail(c, MDI_ERR_ARG, "null argument");
    if (p < 0 || p >= c->K || n < 1) return fail(c, MDI_ERR_ARG, "partition out of range");
    const bool fz = c->last_kernel == 2, td = c->last_kernel == 3;
    if (td ? !(c->td_ok && c->td_prof) : fz ? !(c->fz_ok && c->fz_prof_on) : !(c->pk_ok && c->pk_prof_on))
        return fail(c, MDI_ERR_STATE, "in-kernel timing is off (options.in_kernel_timing at mdi_create; persistent schedulers only)");
    CU(cudaSetDevice(c->dev));
    CU(cudaDeviceSynchronize());
    const int first_cta = td ? c->td_teams_host[p].first_cta : fz ? c->fz_teams_host[p].first_cta : c->pk_teams_host[p].first_cta;
    const int n_cta = td ? c->td_teams_host[p].n_cta : fz ? c->fz_teams_host[p].n_cta : c->pk_teams_host[p].n_cta;
    std::vector<unsigned long long> h((size_t)n_cta * PK_PROF_N);
    CU(cudaMemcpy(h.data(), (td ? c->td_prof : fz ? c->fz_prof : c->pk_prof) + (size_t)first_cta * PK_PROF_N, h.size() * 8, cudaMemcpyDeviceToHost));
    for (int i = 0; i < n; ++i) {
        double acc = 0;
        for (int k = 0; k < n_cta && i < PK_PROF_N; ++k) acc += (double)h[(size_t)k * PK_PROF_N + i];
        out_ms[i] = acc / n_cta * 1e-6;
    }
    return n_cta;
}

int mdi_get_trace(mdi_ctx *c, uint64_t *out_host, int n_words) {
    if (!c || !out_host || n_words < 1) return fail(c, MDI_ERR_ARG, "null argument");
    static_assert(FZ_TRACE_N == MDI_TRACE_WORDS, "trace record size");
    if (!c->fz_trace || c->last_kernel != 2) return fail(c, MDI_ERR_STATE, "no trace was taken (in_kernel_timing and trace_slot at mdi_create; fused-phase kernel only)");
    CU(cudaSetDevice(c->dev));
    CU(cudaDeviceSynchronize());
    const size_t n = std::min<size_t>((size_t)n_words, (size_t)c->fz_trace_blocks * FZ_TRACE_N);
    CU(cudaMemcpy(out_host, c->fz_trace, n * 8, cudaMemcpyDeviceToHost));
    return c->fz_trace_blocks;
}

int64_t mdi_memory_bytes(mdi_ctx *c, int p) {
    if (!c || p < 0 || p >= c->K) return MDI_ERR_ARG;
    return c->part[p].weight_bytes + (int64_t)c->part[p].kv_bytes + c->part[p].buffer_bytes +
           (p < (int)c->fz_team_stream_bytes.size() ? c->fz_team_stream_bytes[p] : 0) + (c->K ? c->td_buf_bytes / c->K : 0);
}

} // extern "C"
