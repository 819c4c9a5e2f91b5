/*
 * skipdecode.h - C ABI of the SkipDecode decode path for NVIDIA B200 (sm_100a).
 *
 * The library runs the batched autoregressive decode step of an OPT-style
 * decoder in which every token of the batch at one sequence position uses the
 * same set of layers (Section 2.1 of the paper), the number of layers follows
 * a monotonically non-increasing per-position budget between a maximum and a
 * minimum (Sections 2.2 and 2.3), and the budget is spent on the top layers
 * while the lower ones are bypassed, optionally after a few warm-up layers at
 * the bottom (Section 2.4).  Because budgets never grow, keys and values that
 * earlier positions wrote in the layers that still run are read as they are
 * and never recomputed (Section 2.2).
 *
 * Conventions
 *   - "host" / "device" in a comment says where a pointer must live.
 *   - The caller owns every buffer: weights, the arena, token and logit
 *     buffers, and the CUDA stream.  The library allocates no device memory;
 *     it owns only the host-side handle.  Weight buffers are referenced, not
 *     copied: they must stay valid until sd_destroy.
 *   - Work is enqueued on the stream given to sd_create; calls return without
 *     synchronising unless stated.  Device outputs are valid once the stream
 *     reaches that point.
 *   - Every function returns 0 (SD_OK) or a negative sd_error.  A call that
 *     fails before enqueueing work changes no state.  Nothing aborts, throws
 *     or traps on the device.
 *   - Call order: sd_create -> sd_schedule -> sd_prefill -> sd_decode_step at
 *     positions P, P+1, ..., P+gen_len-1.  A new sd_prefill starts a new batch
 *     of sequences; sd_schedule may be called again between batches.
 *   - Not thread-safe per handle.
 */
#ifndef SKIPDECODE_H
#define SKIPDECODE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sd_handle sd_handle;

typedef enum {
  SD_OK = 0,
  SD_ERR_ARG = -1,       /* NULL pointer, non-positive size, unsupported shape               */
  SD_ERR_STATE = -2,     /* schedule or prefill missing                                        */
  SD_ERR_POSITION = -3,  /* position out of order, past the schedule, or >= max_pos          */
  SD_ERR_CAPACITY = -4,  /* arena too small, batch/prompt/generation beyond the configuration */
  SD_ERR_CUDA = -5,      /* a CUDA call or launch failed                                      */
  SD_ERR_DEVICE = -6     /* the device status word is non-zero (see sd_status)                */
} sd_error;

enum { SD_DTYPE_FP32 = 0, SD_DTYPE_BF16 = 1 };

/* Model and limits.  Plain data, copied by sd_create.
 * dtype selects the storage type of weights and the KV cache; the residual
 * stream, LayerNorm statistics, softmax, accumulators and logits are fp32 in
 * both modes.  In bf16 mode the inputs of the projections (LayerNorm outputs,
 * attention outputs, FFN activations) are rounded to fp16 and multiplied with
 * the weights' values held as fp16 (exact for magnitudes in [2^-14, 65504];
 * a weight beyond 65504 saturates and sets bit 8 of the device status word).  head_dim = d_model / n_heads must be 32, 64
 * or 128; d_model and d_ffn must be multiples of 8; max_prompt + max_gen <= max_pos. */
typedef struct {
  int32_t n_layers, d_model, n_heads, d_ffn, vocab, max_pos;
  int32_t max_batch, max_prompt, max_gen;
  int32_t dtype;      /* SD_DTYPE_FP32 or SD_DTYPE_BF16 */
  float ln_eps;       /* 1e-5 for OPT */
} sd_config;

/* DEVICE pointers to the weights, each matrix row-major [out, in] as a linear
 * layer stores it, element type per sd_config.dtype, 16-byte aligned.  The
 * per-layer members are HOST arrays of n_layers device pointers.  lm_head may
 * be NULL: the head is then tied to tok_emb (OPT's default). */
typedef struct {
  const void *tok_emb, *pos_emb;              /* [vocab, d], [max_pos, d]                 */
  const void *const *ln1_g, *const *ln1_b;    /* [d] each                                 */
  const void *const *w_qkv, *const *b_qkv;    /* [3d, d] rows ordered q, k, v ; [3d]      */
  const void *const *w_o, *const *b_o;        /* [d, d] ; [d]                             */
  const void *const *ln2_g, *const *ln2_b;    /* [d] each                                 */
  const void *const *w_fc1, *const *b_fc1;    /* [d_ffn, d] ; [d_ffn]                     */
  const void *const *w_fc2, *const *b_fc2;    /* [d, d_ffn] ; [d]                         */
  const void *lnf_g, *lnf_b, *lm_head;        /* [d], [d], [vocab, d] or NULL             */
} sd_weights;

/* Cache sizing plan.  Each layer's KV cache holds max_prompt positions plus
 * one position for every generated index at which the schedule
 * (max_layers, min_layers, warmup, gen_len) runs that layer: a layer that has
 * dropped out of a monotone schedule is never appended to again (Section 2.2).
 * full_capacity = 1 sizes every layer for max_prompt + max_gen positions so
 * that any schedule, including the all-layers baseline, fits. */
typedef struct {
  int32_t max_layers, min_layers, warmup, gen_len, full_capacity;
} sd_plan;

/* Bytes of device memory the arena must provide for (config, plan).
 * out: host.  Errors: SD_ERR_ARG. */
int sd_arena_bytes(const sd_config *cfg, const sd_plan *plan, size_t *out);

/* Creates a handle.  arena: device, 256-byte aligned, arena_bytes >= sd_arena_bytes;
 * it holds the per-layer KV caches [max_batch, n_heads, capacity_l, head_dim] for K
 * and for V, in bf16 mode a tile-packed copy of every weight matrix (made here, once, on
 * the stream), the activation buffers, the split-KV partial results and a status word.
 * stream: a cudaStream_t (NULL = the legacy default stream).  The arena's status and
 * counters are cleared on the stream.
 * Errors: SD_ERR_ARG (shape rules above, NULL weights), SD_ERR_CAPACITY (arena too
 * small), SD_ERR_CUDA. */
int sd_create(const sd_config *cfg, const sd_weights *weights, const sd_plan *plan,
              void *arena, size_t arena_bytes, void *stream, sd_handle **out);

/* Computes and installs the per-position layer budget (Section 2.3): generated
 * index g = position - prompt_len in [0, gen_len) gets
 *     n_active[g] = round_half_up((1 - t) * max_layers + t * min_layers),  t = g / (gen_len - 1)
 * (n_active[0] = max_layers when gen_len = 1), computed in integers, so the first
 * generated position gets max_layers and the last min_layers.  The layers that run
 * at g are [0, warmup) and [top_begin[g], n_layers), top_begin[g] = n_layers -
 * (n_active[g] - warmup) (Section 2.4); prompt positions use every layer.
 * n_active, top_begin: host, gen_len int32 each, either may be NULL.
 * Requires 0 <= warmup < min_layers <= max_layers <= n_layers, 1 <= gen_len <= max_gen.
 * Errors: SD_ERR_ARG; SD_ERR_CAPACITY if a layer would need more cache positions
 * than the plan given to sd_create reserved.  Generation restarts at the end of the
 * prompt: a prompt already processed by sd_prefill stays valid (its cache entries do
 * not depend on the schedule) unless P + gen_len now exceeds max_pos. */
int sd_schedule(sd_handle *h, int max_layers, int min_layers, int warmup, int gen_len,
                int32_t *n_active, int32_t *top_begin);

/* The same arithmetic as sd_schedule without a handle or a device (host only):
 * fills n_active[gen_len] and top_begin[gen_len] for a model of n_layers layers.
 * Errors: SD_ERR_ARG. */
int sd_schedule_compute(int n_layers, int max_layers, int min_layers, int warmup, int gen_len,
                        int32_t *n_active, int32_t *top_begin);

/* Power-law decay, the other budget function Section 2.3 names (host only):
 *     n_active[g] = round_half_up(min_layers + (max_layers - min_layers) * (1 - t)^alpha),  t = g / (gen_len - 1)
 * with an integer exponent 1 <= alpha <= 8, computed in integers; alpha = 1 is the linear schedule and
 * alpha > 1 never exceeds it, so a plan sized for the linear schedule holds every alpha.
 * Errors: SD_ERR_ARG, also when (gen_len - 1)^alpha * 2 (max_layers - min_layers) would not fit the
 * 128-bit integers the rounding is done in (gen_len beyond about 2^14 at alpha = 8). */
int sd_schedule_power_compute(int n_layers, int max_layers, int min_layers, int warmup, int gen_len, int alpha,
                              int32_t *n_active, int32_t *top_begin);

/* Installs a caller-supplied budget table (Section 2.3 allows budget functions other than the linear decay):
 * n_active: host, gen_len int32, non-increasing (Section 2.2), warmup < n_active[g] <= n_layers.
 * The layers that run at g are [0, warmup) and [n_layers - (n_active[g] - warmup), n_layers).
 * top_begin: host, gen_len int32, may be NULL.  Same effects and capacity rule as sd_schedule.
 * Errors: SD_ERR_ARG (also for a table that grows), SD_ERR_CAPACITY. */
int sd_schedule_custom(sd_handle *h, const int32_t *n_active, int warmup, int gen_len, int32_t *top_begin);

/* Cache positions the plan reserves per layer (host only): capacity[n_layers]. */
int sd_layer_capacity(const sd_config *cfg, const sd_plan *plan, int32_t *capacity);

/* Processes the prompt with all layers (Section 2.3): fills cache positions
 * 0..P-1 of every layer and writes the logits of position P-1.
 * The device status word is cleared (on the stream) before the work.
 * d_tokens: device int32 [B, P] row-major, ids in [0, vocab).  d_logits: device
 * fp32 [B, vocab].  1 <= B <= max_batch, 1 <= P <= max_prompt, P + gen_len <= max_pos.
 * Errors: SD_ERR_ARG, SD_ERR_STATE (no schedule), SD_ERR_CAPACITY, SD_ERR_CUDA. */
int sd_prefill(sd_handle *h, const int32_t *d_tokens, int B, int P, float *d_logits);

/* One decode step (Sections 2.1-2.4): the B tokens at `position` run through the
 * layers the schedule makes active there, append their keys/values in those
 * layers only, attend to cache positions 0..position, and produce next-token
 * logits.  d_token_ids: device int32 [B]; d_logits: device fp32 [B, vocab].
 * position must be P + (number of decode steps since sd_prefill).
 * Errors: SD_ERR_ARG, SD_ERR_STATE (no prefill), SD_ERR_POSITION, SD_ERR_CUDA. */
int sd_decode_step(sd_handle *h, const int32_t *d_token_ids, int position, float *d_logits);

/* sd_decode_step with the split-KV attention's partial results kept in an array that is
 * part of the library image instead of the caller's arena.  The paper has no counterpart
 * to this call; it exists for callers that must not, or cannot, allocate device memory
 * while they run: a plug-in loaded into a process whose device memory is owned and
 * fully committed by its host application, a serving or real-time loop that forbids
 * allocation after start-up, a process whose allocator is not reentrant from the thread
 * that drives decoding.  Such a caller
 * still passes the inputs and outputs (and the handle built at start-up); this call itself
 * calls no cudaMalloc, cudaFree or other allocating routine.
 *   - The array holds SD_STATIC_SCRATCH_BYTES per GPU, resident on every GPU that loads
 *     the library until the process exits.  A step needs
 *       B * n_heads * ceil((position + 1) / chunk) * (head_dim + 2) * 4 bytes
 *     (chunk = keys per attention split, see SD_OPT_ATTN_CHUNK); a step that needs more
 *     fails with SD_ERR_CAPACITY and enqueues nothing.
 *   - The first call on each device looks up the array's device address (one host-side
 *     runtime query, with that device current).  Make that first call outside any stream
 *     capture; later calls do no set-up.
 *   - The CUDA device current on the calling thread must be the one that holds the handle's
 *     arena; otherwise SD_ERR_ARG.
 *   - All handles and all calls on one GPU share the array and it keeps the previous
 *     call's contents.  Nothing in it needs clearing: each slot is written before it is
 *     read within the same step.  Two such steps that overlap in time on one GPU (two
 *     handles on two streams) overwrite each other's partial results: serialise them.
 *   - Always plain kernel launches (SD_OPT_GRAPHS is ignored); SD_OPT_TIMING is not recorded.
 * Arguments, ordering rules, results and errors are otherwise those of sd_decode_step,
 * and the two calls may be mixed freely within one sequence. */
#define SD_STATIC_SCRATCH_BYTES (16u << 20)
int sd_decode_step_static(sd_handle *h, const int32_t *d_token_ids, int position, float *d_logits);

/* Ragged batches (the batching limitation of Section 5: rows share a batch only at
 * matching positions, so prompts of different lengths are aligned at the right).
 *
 * sd_set_padding, before sd_prefill: h_pad (HOST, int32 [B]) gives each row's number of
 * left-padding slots, 0 <= h_pad[b] < P.  Row b's own sequence is d_tokens[b, h_pad[b]..P-1]:
 * its first real token takes learned position 0, it never attends to a slot before
 * h_pad[b], and what sits in the padding slots (any valid token id) has no effect on it.
 * The layer budget of a step still goes by the slot, the same for every row (Section
 * 2.1).  NULL removes the padding.  Either way the next call must be sd_prefill.
 *
 * sd_set_rows, after sd_prefill: h_rows (HOST, int32 [n], strictly increasing, each in
 * [0, B)) lists the rows that still generate, e.g. after the others emitted their end
 * token.  From then on sd_decode_step takes d_token_ids [n] and writes d_logits [n, vocab]
 * for exactly those rows, in that order, at a cost of n rows; the other rows' cache
 * entries are left as they are.  NULL restores all B rows; sd_prefill does too.
 * Both calls copy their array before returning and synchronise the stream.
 * Errors: SD_ERR_ARG (range, order, B mismatch at sd_prefill), SD_ERR_STATE (sd_set_rows
 * before sd_prefill). */
int sd_set_padding(sd_handle *h, const int32_t *h_pad, int B);
int sd_set_rows(sd_handle *h, const int32_t *h_rows, int n);

/* Restarts generation at the end of the prompt: the next sd_decode_step must be at
 * position P again.  The prompt's cache entries are kept; entries of generated
 * positions are overwritten as the new steps reach them.  Errors: SD_ERR_STATE. */
int sd_rewind(sd_handle *h);

/* The same step with HOST buffers: copies h_token_ids [B] to the device, runs the
 * step, copies the logits [B, vocab] back and synchronises the stream.  Pinned
 * host memory makes the copies asynchronous to the host but is not required. */
int sd_decode_step_host(sd_handle *h, const int32_t *h_token_ids, int position, float *h_logits);

/* Greedy choice: d_next[b] = lowest index attaining the maximum of d_logits[b, :].
 * d_logits: device fp32 [B, vocab]; d_next: device int32 [B]. */
int sd_greedy(sd_handle *h, const float *d_logits, int B, int32_t *d_next);

/* Sampled choice with the paper's generation settings (Section 3.2, Datasets: beam 1,
 * top-p 0.7, temperature 0.3), any values accepted: p = softmax(d_logits[b, :] / temperature);
 * the nucleus of row b is the smallest set of most probable tokens whose probabilities sum to
 * at least top_p (equal probabilities: lower token id first); with the nucleus in order of
 * decreasing probability and M its total probability, d_next[b] is the first token whose
 * running sum exceeds d_uniforms[b] * M.  The random numbers are the caller's:
 * d_uniforms: device fp32 [B], each in [0, 1) (values outside are clamped into the range).
 * Probabilities are summed as 2^-40 fixed-point integers, so the result does not depend on
 * thread order.  d_logits: device fp32 [B, vocab]; d_next: device int32 [B].
 * Errors: SD_ERR_ARG unless temperature > 0 and 0 < top_p <= 1 (both finite). */
int sd_sample_top_p(sd_handle *h, const float *d_logits, int B, float temperature, float top_p,
                    const float *d_uniforms, int32_t *d_next);

/* Synchronises the stream and reads the device status word (0 = no error; kernels
 * set bits on an out-of-range token id or a bounded wait that expired).
 * Returns SD_ERR_DEVICE when it is non-zero. */
int sd_status(sd_handle *h, int32_t *device_status);

/* Decode steps run since sd_create and the number of layer executions they made
 * (their ratio is the mean active layers per generated token). */
int sd_stats(sd_handle *h, int64_t *steps, int64_t *layer_steps);

/* Kernels this handle has launched since sd_create (graph replays count their nodes). */
int sd_launch_count(sd_handle *h, int64_t *launches);

/* Tuning knobs; every value of every option computes the same function. */
enum {
  SD_OPT_GRAPHS = 1,       /* 1 (default): replay one CUDA graph per step shape; 0: plain launches */
  SD_OPT_ATTN_CHUNK = 2,   /* keys per split of the decode attention (multiple of 32); 0 = automatic */
  SD_OPT_GEMM = 3,         /* bf16 mode: 0 = automatic (tensor-core kernels, CUDA cores for shapes they do
                              not take); 1 = CUDA cores only; 2 = same as 0                              */
  SD_OPT_TIMING = 4,       /* 1: record per-kernel-class device time (plain launches, slower)      */
  SD_OPT_PDL = 5,          /* programmatic dependent launch: mask of kernel classes (1 << SD_K_*) whose
                              kernels may begin before their predecessor ends; 0 = none             */
  SD_OPT_PREFILL_ATTN = 8, /* 1 (default): sd_prefill's causal attention runs as 64x64 tensor-core tiles
                              (bf16 storage, head size 64 or 128); 0: one decode-style block per query row */
  SD_OPT_GEMM_PERSISTENT = 10, /* 1 (default): products with more than 64 tokens and more output tiles than SMs
                              run on the persistent kernel (one block per SM, double-buffered accumulator,
                              epilogue overlapped with the next tile's main loop; token tiles of 128, or of 96
                              where that takes fewer rounds of tiles per block); 2: the same with 128-token
                              tiles only; 0: one block per tile */
  SD_OPT_GEMM_SPLITK = 11, /* 0..8, default 8 = the most splits of K for a QKV, fc1 or LM-head product whose output
                              tiles cover fewer than half of the SMs (every split keeps at least 8 k-blocks of 64);
                              the partial tiles are parked in the arena and the block that arrives last adds them in
                              split order and runs the epilogue (results do not depend on arrival order);
                              0: K is split for the two residual products only */
  SD_OPT_DETERMINISTIC = 12, /* 0 (default): the out-projection and fc2, whose K is split over several blocks, add their
                              partial sums to the residual stream with atomic adds, i.e. in arrival order, so two runs
                              can differ in the last bits; 1: these products park their partial tiles like the others and
                              the block that arrives last adds them in split order: every run gives the same bits,
                              at a tenth to a fifth of the decode rate (a second pass over every tile of those products) */
  SD_OPT_TEST_WAIT_EXPIRY = 13, /* test hook, one shot: the next tensor-core product never reports its accumulator
                              complete, its epilogue gives up the bounded wait after about a millisecond, writes
                              nothing, and sets the wait-expired bit of the status word (sd_status then returns
                              SD_ERR_DEVICE).  Nothing is left in flight and the handle stays usable: the following
                              sd_prefill clears the status word.  The step that contained the product returns garbage. */
  SD_OPT_ATTN_STAGED = 14    /* bf16 storage: 1 (default) = decode-attention launches with at least 12 (row, head) pairs per
                              SM, on a handle configured for at least 1024 positions (max_prompt + max_gen), stream K and V
                              through a ring of shared-memory stages filled by 8 KB bulk copies; 2 = the same without the
                              length condition; 0 = every launch uses the kernel that loads them straight into registers
                              (as fp32 storage and smaller launches always do) */
};
int sd_set_option(sd_handle *h, int option, int value);
#define SD_PDL_ALL 0x1ff
/* Default: the five GEMM classes and the LayerNorms.  A GEMM that starts early sets up its barriers and
 * tensor memory and streams its first weight tiles while its predecessor drains (measured +1.5 % at the
 * OPT-6.7B shape); a LayerNorm that starts early saves its launch latency after the residual product, which is
 * nothing at the OPT-6.7B shape and +3 % / +5 % at the OPT-1.3B / OPT-125M shapes, where the products are short;
 * starting the attention kernel early gains nothing anywhere and costs 7 % at the OPT-1.3B shape. */
#define SD_PDL_DEFAULT ((1 << 1) | (1 << 2) | (1 << 5) | (1 << 6) | (1 << 7) | (1 << 8))

/* Device time and launch count accumulated per kernel class while SD_OPT_TIMING is
 * on; synchronises the stream.  ms, launches: host. */
enum { SD_K_EMBED = 0, SD_K_LAYERNORM = 1, SD_K_GEMM_QKV = 2, SD_K_KV_APPEND = 3,
       SD_K_ATTENTION = 4, SD_K_LM_HEAD = 5, SD_K_GEMM_OUT = 6, SD_K_GEMM_FC1 = 7,
       SD_K_GEMM_FC2 = 8, SD_K_COUNT = 9 };
int sd_kernel_time(sd_handle *h, int kernel_class, double *ms, int64_t *launches);
int sd_kernel_time_reset(sd_handle *h);

const char *sd_strerror(int code);
void sd_destroy(sd_handle *h);

#ifdef __cplusplus
}
#endif
#endif /* SKIPDECODE_H */
