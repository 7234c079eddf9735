/* mdi.h - C ABI of the recurrent-pipeline decoding library (MDI-LLM hot path on one GPU).
 *
 * The method (paper, Section III): a decoder-only transformer is cut into K contiguous
 * chunks of blocks ("nodes"); several text samples are kept in flight; each node
 * repeatedly takes the next sample's activation from its input queue, selects that
 * sample's key/value cache (Section III-D), runs its blocks, and hands the result to the
 * next node; the last result returns to the first node, which produces a token and feeds
 * it back (Section III-C, Algorithms 1 and 2).  Here the K nodes are K CUDA streams of one
 * GPU, the links between nodes are device-resident activation ring buffers handed over
 * with events, and every sample owns a slot of a paged key/value pool.
 *
 * Conventions
 *  - Every function returns MDI_OK (0) or a negative MDI_ERR_* code; nothing aborts.
 *    mdi_last_error() gives the text of the last failure on that context.
 *  - "host" pointers are ordinary CPU memory owned by the caller; the library copies
 *    what it needs before returning.  "dev" pointers are CUDA device memory owned by the
 *    caller.  All other device memory (weights, caches, rings, logits) belongs to the
 *    context and is released by mdi_destroy().
 *  - A context is bound to the CUDA device current at mdi_create() and is not
 *    thread-safe.  The library never falls back to the CPU.
 *  - slot == sample index in [0, n_samples).
 */
#ifndef MDI_H_
#define MDI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    MDI_OK = 0,
    MDI_ERR_ARG = -1,     /* null pointer, index out of range, bad enum value */
    MDI_ERR_SHAPE = -2,   /* model shape or tensor size the kernels do not support */
    MDI_ERR_OOM = -3,     /* device allocation failed or key/value page pool exhausted */
    MDI_ERR_CONTEXT = -4, /* prompt + new tokens would exceed n_ctx */
    MDI_ERR_STATE = -5,   /* call out of order: missing weights, sample not prefilled, ... */
    MDI_ERR_TIMEOUT = -6, /* a bounded wait ran out */
    MDI_ERR_CUDA = -7     /* a CUDA runtime call failed */
};

enum { MDI_ARCH_GPT = 0, MDI_ARCH_LLAMA = 1 };
enum { MDI_DTYPE_F32 = 0, MDI_DTYPE_BF16 = 1 };
enum { MDI_ACT_GELU_TANH = 0, MDI_ACT_GELU_ERF = 1, MDI_ACT_SWIGLU = 2 };
enum { MDI_KV_DEFAULT = 0, MDI_KV_BF16 = 1, MDI_KV_F16 = 2, MDI_KV_F32 = 3 };

typedef struct mdi_ctx mdi_ctx;

/* Shape of the decoder (the block of Section III-B: attention + fully connected layer,
 * each with a residual connection; equal input and output width d_model). */
typedef struct {
    int arch;         /* MDI_ARCH_GPT: LayerNorm, learned positions, biases, GELU MLP;
                         MDI_ARCH_LLAMA: RMSNorm, rotary positions (split-halves pairing), SwiGLU, no biases */
    int n_layer, d_model, n_head, head_dim, n_kv_head, d_ff, vocab, n_ctx;
    int weight_dtype; /* MDI_DTYPE_*: element type of every tensor given to mdi_load_weights; activations,
                         accumulation and (by default) the key/value cache are fp32 */
    int tied_lm_head; /* 1: the output projection reuses "wte" */
    int has_bias;     /* 1: linear layers carry biases (GPT) */
    int act;          /* MDI_ACT_* */
    float norm_eps, rope_theta;
} mdi_model_shape;

/* Optional tuning; zero means "default". */
typedef struct {
    int page_tokens;   /* rows per key/value page (power of two; default 16, or 128 for shapes the fused-phase
                          scheduler covers, whose bulk copies of cache rows want large pages) */
    int kv_pool_tokens;/* tokens of cache each partition's pool can hold over all samples
                          (default n_samples * n_ctx, rounded up to pages) */
    int attn_splits;   /* sequence splits of decode attention (default: chosen from n_ctx) */
    int rounds_per_graph; /* stream scheduler: rounds of the recurrent schedule captured per CUDA graph
                             (default 16; <0: no graphs) */
    int kv_cache_dtype; /* MDI_KV_*: element type of the key/value cache when the weights are bf16 (fp32 weights always
                          keep an fp32 cache).  DEFAULT: F16 for models the fused-phase scheduler cannot cover (Llama block,
                          grouped-query heads, d_model > 1024 or head_dim > 64), F32 for those it can (it reads fp32 pages).
                          F16 halves the cache bytes at 1.6e-2 worst absolute logit error on the 32-block Llama-7B shape and
                          6e-4 on the 48-block GPT-2-XL shape (measured over whole generations; fp32: 1.2e-3 and 3e-5); keys
                          and values of these models are far inside its range.  BF16 costs eight times the F16 error, which
                          on the 32-block model exceeds a 3e-2 absolute logit tolerance */
    int prefill_mode;  /* first visits (whole prompt): 0 (default) tensor-core GEMMs (tcgen05, bf16 x bf16 -> fp32, inputs split
                          into two bf16 planes) when the weights are bf16, else the CUDA-core step kernels in chunks of 8
                          positions; 1: always the CUDA-core kernels */
    int tc_min_group;  /* decode steps of groups with at least this many samples run their linear layers as tensor-core
                          GEMMs (bf16 weights, prefill_mode 0; such calls use the stream scheduler).  0 (default): 5,
                          or 1 when the matrices of one block hold 48 MB or more */
    int wait_limit_ms; /* limit of every wait inside the persistent kernel (input edge, team barrier, weight tile); when
                          one runs out mdi_generate returns MDI_ERR_TIMEOUT, every sample is reset and the context stays
                          usable.  0 (default): 2000 ms */
    int debug_withhold_handoff; /* failure-detection check: p > 0 makes partition p-1 withhold its output handoff during
                          the first persistent mdi_generate after creation, so that the next partition's wait runs out */
    int scheduler;     /* how mdi_generate runs the recurrent pipeline.
                          0: a persistent kernel when the shape fits one (one cooperative launch for the whole call,
                             one team of thread blocks per partition, flag handoff between teams), else the stream
                             scheduler.  Two persistent kernels exist: the fused-phase kernel (GPT block, bf16 weights,
                             fp32 cache, n_kv_head = n_head, d_model <= 1024, groups of at most 4 samples, every team
                             at least n_head blocks: two team barriers per block of the model, weights re-stored per
                             thread block in tensor-core fragment order, a head shared by the two blocks of a
                             cluster where every team has 2 n_head blocks) is preferred; the phase-per-matrix kernel
                             (groups of at most 4 samples, any block type) comes next;
                          1: always the stream scheduler (one stream per partition, event handoff);
                          2: the phase-per-matrix persistent kernel, or fail;
                          3: the fused-phase persistent kernel, or fail;
                          4: the tensor-core persistent kernel, or fail (bf16 weights, groups of at most 8 samples, widths
                             that are multiples of 64, greedy token choice: one cooperative launch, a team per partition,
                             every linear layer a tcgen05 contraction fed by a TMA weight ring).  Never picked by
                             scheduler 0: on the large workloads it measures at or below the stream scheduler */
    int in_kernel_timing; /* 1: the persistent kernels time themselves (mdi_get_partition_times); costs a few percent */
    int fused_blocks_per_head; /* fused-phase kernel: 0 (default) two thread blocks of a cluster share a head where every
                          team has a cluster per head, else one block per head; 1: always one block per head (plain
                          cooperative launch, no clusters: the choice for a runtime or tool that refuses cooperative launches
                          in clusters, which otherwise fail with MDI_ERR_CUDA) */
    int reserved0;     /* must be 0 */
    int trace_slot;    /* with in_kernel_timing: s > 0 makes thread 0 of every block of the fused-phase kernel record a
                          time stamp at every change of timing category while it serves schedule slot s - 1
                          (mdi_get_trace) */
    int td_b_kblocks;  /* tensor-core persistent kernel: 64-column blocks of the activation operand kept in shared memory
                          (the weight ring gets the rest); 0 (default): 32 for d_model >= 2048, else 16 */
} mdi_options;

typedef struct {
    int n_partitions, n_samples, n_groups;
    int64_t weight_bytes[16];   /* per partition, device bytes of parameters (first 16 partitions) */
    int64_t kv_pool_bytes[16];  /* per partition, device bytes of the key/value pool */
    int64_t kv_pages_in_use[16];
    int64_t tokens_generated;   /* head evaluations since creation */
    int64_t stage_steps;        /* partition steps launched since creation */
    int64_t kernel_launches;    /* kernels of this library launched (or replayed in graphs) since creation */
    float last_prefill_ms;      /* device time from the first mdi_prefill after the previous mdi_generate to the
                                   end of the last one (events on the partition streams) */
    float last_generate_ms;     /* device time of the last mdi_generate, first to last partition step */
    float last_run_ms;          /* device time from that first mdi_prefill to the end of the last mdi_generate */
    int kv_element_bytes;       /* bytes per element of the key/value cache (4, or 2 for a bf16 / fp16 cache) */
} mdi_stats;

/* Set-up of the nodes (Section III-A: the starter assigns each node its chunk).
 * part_bounds: K+1 ascending layer indices, part_bounds[0] = 0, part_bounds[K] = n_layer;
 * partition p holds blocks [part_bounds[p], part_bounds[p+1]).  Partition 0 also holds the
 * input layers (embeddings); partition K-1 also holds the output layers (final norm and
 * vocabulary projection) - the paper keeps them on the starter, which changes only where
 * the work runs.  n_samples = samples in flight (slots).  opts may be NULL.
 * Errors: ARG (nulls, K < 1, bounds not ascending), SHAPE (unsupported sizes), OOM. */
int mdi_create(const mdi_model_shape *shape, const int *part_bounds, int K, int n_samples,
               const mdi_options *opts, mdi_ctx **out);
void mdi_destroy(mdi_ctx *ctx);

/* Giving a node its chunk of the model (the loading step that opens Algorithms 1 and 2).  One call per tensor; host_data is row-major
 * [out_features][in_features] for matrices, element type shape.weight_dtype, nbytes its
 * exact size.  Names: "wte" [vocab][d], "wpe" [n_ctx][d] (GPT), "lnf.g", "lnf.b" (GPT),
 * "lm_head" [vocab][d] (untied), and per block i: "h.<i>.ln1.g", "h.<i>.ln1.b" (GPT),
 * "h.<i>.attn.wqkv" [(n_head+2 n_kv_head) head_dim][d] (q rows, then k, then v),
 * "h.<i>.attn.bqkv", "h.<i>.attn.wo" [d][n_head head_dim], "h.<i>.attn.bo", "h.<i>.ln2.g",
 * "h.<i>.ln2.b", GPT: "h.<i>.mlp.w1" [d_ff][d], ".b1", ".w2" [d][d_ff], ".b2";
 * Llama: "h.<i>.mlp.wgate" [d_ff][d], ".wup" [d_ff][d], ".wdown" [d][d_ff].
 * The data is copied to the device before the call returns.  With bf16 weights (and prefill_mode != 1)
 * the first mdi_prefill / mdi_step / mdi_generate after a load also builds, on the device, a second copy
 * of every matrix of the blocks and of the output layer as contiguous 128 x 64 tiles for the tensor-core
 * linear layers (device memory of those matrices doubles; counted by mdi_memory_bytes among the buffers of the
 * partition that owns the matrix).
 * Errors: ARG (unknown name), SHAPE (nbytes mismatch), CUDA. */
int mdi_load_weights(mdi_ctx *ctx, const char *tensor_name, const void *host_data, size_t nbytes);

/* First visit of a sample (the branch of Algorithm 1 taken on a sample's first iteration, and of Algorithm 2 taken
 * while the node holds no cache for the sample yet):
 * the whole prompt goes through every partition in turn, filling cache rows 0..n_prompt-1 of
 * the sample's slot; only the last position reaches the output layers, whose result is the
 * sample's first new token (kept pending until mdi_generate returns it).  Work is enqueued
 * on the partition streams with event handoff, so consecutive calls for different samples
 * overlap like the paper's start-up phase; it completes by the next mdi_sync/mdi_generate.
 * prompt_host: n_prompt token ids in [0, vocab).  The _dev form reads them from device memory.
 * Errors: ARG, STATE (slot already holds tokens: mdi_reset_sample first; weights missing),
 * CONTEXT (n_prompt > n_ctx), OOM (page pool). */
int mdi_prefill(mdi_ctx *ctx, int sample, const int32_t *prompt_host, int n_prompt);
int mdi_prefill_dev(mdi_ctx *ctx, int sample, const int32_t *prompt_dev, int n_prompt);

/* One visit of one sample to one node (body of the loop of Algorithm 2; for partition 0 the
 * "forward through input layers" of Algorithm 1): select the slot's cache, run the partition's
 * blocks on one new position, append its keys and values.
 * act_in_dev:  partition 0: one int32 token id; otherwise fp32[d_model].
 * act_out_dev: last partition: one int32 token id (greedy argmax, lowest id on ties; the logits
 * are kept for mdi_get_logits); otherwise fp32[d_model].  Both in device memory.
 * Advances the slot's position in that partition by one.  Enqueued on the partition's stream;
 * mdi_sync() waits.  Errors: ARG, STATE, CONTEXT (slot full), OOM. */
int mdi_step(mdi_ctx *ctx, int partition, int slot, const void *act_in_dev, void *act_out_dev);

/* Recurrent pipeline (Section III-C; Algorithm 1's loop over n_samples x n_tokens): returns the
 * next n_new_tokens greedy tokens of samples 0..n_samples-1, which must all have been
 * prefilled.  Samples are dealt into G = min(n_samples, K) groups (sample s in group s mod G);
 * at tick t partition p serves group (t - p) mod K (an idle tick if that is >= G, i.e. fewer
 * samples than partitions); a group's samples share one pass over the partition's weights.  A token produced by the last partition is fed to partition 0 one tick
 * later; the last token of the call is produced but not fed (it is fed first by a later call).
 * out_tokens: [n_samples][n_new_tokens] int32, host (or device for the _dev form).
 * Blocks until the tokens are there.  Errors: ARG, STATE, CONTEXT, OOM, TIMEOUT (a bounded wait of the
 * persistent kernel ran out: all samples are then reset, prefill them again). */
int mdi_generate(mdi_ctx *ctx, int n_samples, int n_new_tokens, int32_t *out_tokens_host);
int mdi_generate_dev(mdi_ctx *ctx, int n_samples, int n_new_tokens, int32_t *out_tokens_dev);

/* Token choice.  The paper samples the next token from the probability mass function given by the logits
 * (Section III-B); the default here is the greedy argmax.  temperature > 0 switches to sampling: the top_k
 * (1..64) most likely tokens are kept (larger logit first, lower id first on ties), p_j = exp((l_j - l_0) /
 * temperature) in fp64, and token j is chosen when the running sum in that order first exceeds u * sum(p),
 * where u in [0,1) is a counter-based uniform of (seed, sample, index of the output-layer evaluation counted
 * from the prefill): u = (h >> 11) / 2^53, h = mix(mix(seed ^ (sample << 32)) + index), mix = the splitmix64
 * output function.  The same (seed, sample, index) always gives the same u, so a run can be reproduced.
 * temperature <= 0 returns to greedy.  Sampling calls run on the stream scheduler.  mdi_step keeps the argmax.
 * Errors: ARG (top_k out of range). */
int mdi_set_sampling(mdi_ctx *ctx, float temperature, int top_k, uint64_t seed);

/* Logits (fp32[vocab]) of the sample's most recent output-layer evaluation, copied to host. */
int mdi_get_logits(mdi_ctx *ctx, int sample, float *out_host);

/* Checking aid: the i-th output-layer evaluation of the sample (counted from its prefill)
 * still reports its own argmax, but tokens_host[i] is what gets fed back for i < n.
 * Must be set after mdi_reset_sample/creation and before the sample's prefill. */
int mdi_set_teacher_tokens(mdi_ctx *ctx, int sample, const int32_t *tokens_host, int n);

/* Forget a sample: its pages go back to the pools, its position and counters to zero. */
int mdi_reset_sample(mdi_ctx *ctx, int sample);

int mdi_get_stats(mdi_ctx *ctx, mdi_stats *out);
/* Device bytes held by one partition (parameters + key/value pool + buffers, and once the fused-phase kernel has run its
 * per-thread-block copy of the partition's matrices), cf. Tables I-II. */
int64_t mdi_memory_bytes(mdi_ctx *ctx, int partition);
/* Tracing aid (the paper times token arrival on the starter; here each partition's team of thread
 * blocks times itself).  With in_kernel_timing set at mdi_create, the persistent kernel accumulates, per
 * thread block, the nanoseconds spent in: [0] waiting for the input edge, [1] staging
 * and normalising inputs, [2] streaming weight tiles, [3] team barriers, [4] attention, [5] choosing
 * tokens, [6] producer warp waiting for a free ring slot, [7] producer warp total, and within [2]:
 * [8] waiting for a tile to land, [9] multiply-accumulate, [10] reduction and epilogue.  When the last call ran the
 * fused-phase kernel the categories are: [0] input edge, [1] norm prologues, [2] row parts (split along k; for the
 * output layer: unused), [3] bias / activation / cache append after a row part, [4] attention, [5] column parts and the
 * output layer's rows, [6] and [7] as above, [8] team barriers, [9] end of step (token choice or handoff), [11] time
 * inside [2], [4], [5] spent waiting for ring slots.  This call averages
 * them over the partition's blocks for the last mdi_generate, in milliseconds, into out_ms[0..n).
 * Returns the number of blocks of the partition (> 0) or a negative error (STATE when timing is off). */
int mdi_get_partition_times(mdi_ctx *ctx, int partition, double *out_ms, int n);
/* Time stamps of the traced schedule slot (options.trace_slot) of the last mdi_generate that ran the fused-phase
 * kernel: per thread block MDI_TRACE_WORDS 64-bit words, each (nanoseconds << 4) | category in the order the
 * block went through them, 0 = unused.  Copies min(n_words, blocks * MDI_TRACE_WORDS) words to out_host and returns
 * the number of blocks (> 0), or a negative error (STATE when no trace was taken). */
#define MDI_TRACE_WORDS 128
int mdi_get_trace(mdi_ctx *ctx, uint64_t *out_host, int n_words);
/* Wait for everything enqueued on the context's streams. */
int mdi_sync(mdi_ctx *ctx);
/* Greedy token choice for callers that must not allocate.  (The paper has no counterpart: this is a
 * convenience of this library, not part of the method.)
 * Some users of the library cannot call cudaMalloc where they pick tokens: a serving loop that has
 * given the whole device to its own memory pool, a latency-critical section that cannot afford the
 * device synchronisation an allocation or a free may bring, or code that runs where another component
 * owns the allocator.  They already hold the logits; this call returns, per row, the index of the largest
 * value (the lowest index on ties, like the output layer of mdi_generate) and allocates nothing: its
 * working memory is a fixed array inside the library (about 128 KB on every GPU that loads the library,
 * held until the process exits).
 *   logits_dev: [n_rows][n_cols] fp32, row-major, device memory of the current device (read only);
 *   out_dev:    [n_rows] int32, device memory; stream: a cudaStream_t (NULL = default stream).
 * Limits: n_rows <= 64 and n_cols <= 262144; larger sizes return MDI_ERR_SHAPE and touch nothing.
 * The work is enqueued on `stream`; the result is there once the stream has reached it.
 * The first call on each device looks up the array's device address (one extra runtime query): make
 * that first call outside any stream capture.  All calls on a device share the one array, which keeps
 * what the previous call left in it (the call clears the counters it needs): two calls that overlap on
 * the GPU - different streams without an ordering between them - race on it and give wrong tokens, so
 * order them (same stream, or events).  Errors: ARG (null pointer, non-positive size), SHAPE, CUDA; the
 * text is available from mdi_last_error(NULL). */
int mdi_greedy_argmax_static(const float *logits_dev, int n_rows, int n_cols, int32_t *out_dev, void *stream);

/* Text of the last error of this context; with ctx NULL, of the last failed call that takes no context
 * (mdi_create, mdi_greedy_argmax_static). */
const char *mdi_last_error(mdi_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* MDI_H_ */
