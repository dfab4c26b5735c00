/*
 * tlr -- token-level routing step on one NVIDIA B200 (sm_100a).
 *
 * For n decoding positions the library takes the small model's last-layer hidden
 * states h[n,d] and its LM-head matrix W[V,d] and produces, without ever writing the
 * n x V logits to memory,
 *
 *     token[i]      = argmax_v  z[i,v],   z[i,v] = sum_k h[i,k] W[v,k]   (lowest v on ties)
 *     conf[i]       = max_v softmax(z[i,:])_v          (the "confidence score")
 *     entropy[i]    = -sum_v p_v ln p_v                (nats)
 *     route_mask[i] = conf[i] < tau ? 1 : 0            (1 = send this token to the large model)
 *     routed_idx    = ascending list of the i with route_mask[i] = 1
 *     routed_count  = length of that list
 *
 * Where this comes from in the paper ("Token Level Routing Inference System for Edge
 * Devices", arXiv 2504.07878): Sec. 3.1 "Front End" defines the decision -- a score is
 * computed from the small model's last-layer hidden state and the token is routed to
 * the large model when the score falls below the threshold; Sec. 2.1 names the
 * threshold tau; Sec. 3.3 "Backend" exposes the last-layer hidden state, which is the
 * LM head's input; the record of Fig. 5 carries the same quantities (hidden_states,
 * routing_threshold, current_token, per-token route flag, token_index).  The paper
 * gives no dimensions or weights for its learned score, so the score here is the small
 * model's own max softmax probability; entropy is reported beside it.  Batching over n
 * positions and the index list are this library's data-parallel restatement of the
 * paper's one-token-at-a-time loop.
 *
 * All pointers named *_dev are device pointers on the context's GPU; *_host are host
 * pointers.  The library never takes ownership of a caller's buffer.  Every function
 * returns a status code; none throws, aborts or prints.
 */
#ifndef TLR_H_
#define TLR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tlr_ctx tlr_ctx; /* opaque */

typedef enum {
  TLR_OK = 0,
  TLR_ERR_ARG = 1,           /* null pointer, negative size, n > max_n, ... */
  TLR_ERR_ALIGN = 2,         /* W or h not 16-byte aligned */
  TLR_ERR_UNSUPPORTED = 3,   /* device is not sm_100, or a shape the kernels cannot address */
  TLR_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed */
  TLR_ERR_NOMEM = 5,         /* workspace allocation failed */
  TLR_ERR_TOO_MANY_ROWS = 6, /* n > max_n given at creation */
  TLR_ERR_DEVICE_STATUS = 7  /* a kernel reported a fault flag (see tlr_last_device_status) */
} tlr_status;

/* Which projection kernel a call of n rows uses. */
typedef enum {
  TLR_PATH_AUTO = 0,   /* choose by shape (default) */
  TLR_PATH_SIMT = 1,   /* CUDA-core kernel: any d, any V; the only path when d % 8 != 0 */
  TLR_PATH_TC = 2      /* tcgen05 tensor-core kernel fed by TMA; needs d % 8 == 0 */
} tlr_path;

/* Launch plan of the projection kernel for a given n (for reports and tests). */
typedef struct {
  int32_t path;          /* tlr_path actually used */
  int32_t grid;          /* CTAs launched */
  int32_t block;         /* threads per CTA */
  int32_t row_units;     /* ceil(n / rows per CTA tile) */
  int32_t vocab_chunks;  /* partial results per row that the merge step folds */
  int32_t smem_bytes;    /* dynamic shared memory per CTA */
  int32_t launches;      /* kernels launched per tlr_route call */
  int32_t reserved;
} tlr_plan;

/* Bits of the device status word (tlr_last_device_status). */
#define TLR_DEV_WAIT_TIMEOUT 1u   /* a bounded barrier wait inside a kernel gave up */
#define TLR_DEV_NONFINITE 2u      /* a row produced a confidence that is not a number */

/*
 * tlr_create -- bind an LM head to a context (Sec. 3.3: the head whose input is the
 * exposed last-layer hidden state).
 *   d, V        hidden size and vocabulary size, both > 0.
 *   W_bf16_dev  device pointer to W, bf16, row-major [V, d] (row v = output embedding of
 *               token v), 16-byte aligned.  BORROWED for the life of the context: the
 *               caller keeps it allocated and unchanged; it is not copied.
 *   max_n       largest n any later call will pass (>= 1).  Sizes the workspace.
 *   out         receives the context.
 * The only call that allocates device memory: the per-row partial-result workspace,
 * a status word, and two sets of staging buffers (device and pinned host) for tlr_route_host.  Uses the current CUDA device;
 * every later call on the context must be made with that device current.
 * Errors: TLR_ERR_ARG, TLR_ERR_ALIGN, TLR_ERR_UNSUPPORTED (not an sm_100 device),
 * TLR_ERR_NOMEM, TLR_ERR_CUDA.  On error *out is NULL and nothing is leaked.
 */
tlr_status tlr_create(int32_t d, int32_t V, const void* W_bf16_dev, int32_t max_n, tlr_ctx** out);

/*
 * tlr_route -- the routing step for n positions (Sec. 3.1 decision rule; Sec. 2.1 tau).
 *   h_bf16_dev        bf16 row-major [n, d], 16-byte aligned, caller-owned.
 *   n                 0 <= n <= max_n.  n == 0 writes routed_count = 0 and nothing else.
 *   tau               threshold; not range-checked (tau <= 0 routes nothing, tau > 1 routes all).
 *                     A row whose confidence is not a number is routed and raises
 *                     TLR_DEV_NONFINITE.
 *   token_dev         int32 [n]   out
 *   conf_dev          float [n]   out
 *   entropy_dev       float [n]   out
 *   route_mask_dev    uint8 [n]   out, 0 or 1
 *   routed_idx_dev    int32 [n]   out, capacity n; entries [0, routed_count) are valid and
 *                                 ascending, the rest are left untouched
 *   routed_count_dev  int32 [1]   out, stays on the device
 *   cuda_stream       a cudaStream_t (NULL = legacy default stream)
 * Enqueues its kernels on cuda_stream and returns without synchronising; outputs are
 * valid once the stream reaches that point.  Allocates nothing.  Calls on one context
 * share its workspace, so they must be ordered (same stream, or externally serialised).
 * Because it neither allocates, nor reads anything back, nor synchronises, the call may be
 * captured in a CUDA graph (stream capture) and replayed: the graph then reads h and writes
 * the outputs at the captured addresses, with the captured n and tau.
 * Errors (all detected on the host before any launch): TLR_ERR_ARG, TLR_ERR_ALIGN,
 * TLR_ERR_TOO_MANY_ROWS, TLR_ERR_CUDA.
 */
tlr_status tlr_route(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, float tau,
                     int32_t* token_dev, float* conf_dev, float* entropy_dev,
                     uint8_t* route_mask_dev, int32_t* routed_idx_dev,
                     int32_t* routed_count_dev, void* cuda_stream);

/*
 * tlr_route_ex -- tlr_route with the routing variants the paper's Sec. 2 and Sec. 3 name.
 *   opt->tau_per_row_dev   optional float [n] on the device: row i is compared with
 *                          tau_per_row_dev[i] instead of the scalar tau (the threshold is a
 *                          per-user setting in the paper's front end, Sec. 3.1, so a batch of
 *                          sessions carries one threshold per row).  NULL = scalar tau.
 *   opt->route_above       0: route iff score < tau (Sec. 3.1).  1: route iff score > tau, the
 *                          polarity of the deferral rule of Sec. 2.2 (defer when the deferral
 *                          probability exceeds eta).  A row whose score is not a number is
 *                          routed under either polarity.
 *   opt->score_source,     which score decides (see tlr_set_router_mlp below); mlp_score_dev optionally
 *   opt->mlp_score_dev     receives the learned score of every row.
 *   opt->seq_len,          when seq_len > 0 the n rows are n / seq_len sequences of seq_len
 *   opt->first_routed_dev  consecutive positions (n must be a multiple of seq_len) and
 *                          first_routed_dev (int32 [n / seq_len], device) receives, per
 *                          sequence, the position within the sequence of its first routed row,
 *                          or seq_len if none is routed: after the large model has supplied a
 *                          token the small model re-processes the whole context (Sec. 4.1, the
 *                          multi-round prefill of Sec. 3), and this is where it has to stop next.
 * opt == NULL behaves exactly like tlr_route.  Same outputs, stream semantics and errors as
 * tlr_route; TLR_ERR_ARG also for seq_len > 0 with n % seq_len != 0 or a NULL first_routed_dev.
 */
typedef struct {
  const float* tau_per_row_dev;
  int32_t route_above;
  int32_t seq_len;
  int32_t* first_routed_dev;
  int32_t score_source;      /* TLR_SCORE_CONF (0) or TLR_SCORE_MLP (1): which score is compared with tau */
  float* mlp_score_dev;      /* optional float [n] out: the learned score of every row (needs tlr_set_router_mlp) */
} tlr_route_options;

#define TLR_SCORE_CONF 0   /* the small model's max softmax probability (default) */
#define TLR_SCORE_MLP 1    /* the learned score of tlr_set_router_mlp */

/*
 * tlr_set_router_mlp -- attach a learned router to the context.  The score the paper deploys is a
 * small learned classifier (an MLP) fed with the last-layer hidden state (Sec. 3.1, Sec. 2.1); its
 * width, activation and weights are not given, so the shape here is this library's assumption:
 *     score(h) = sigmoid( w2 . relu(W1 h + b1) + b2 )        in (0, 1), high = keep the small model
 *   d_hidden        hidden width, > 0
 *   W1_bf16_dev     bf16 [d_hidden, d] row-major on the device;  b1_dev, w2_dev  float [d_hidden];  b2 scalar
 * The pointers are BORROWED for the life of the context (or until replaced by another call).
 * Allocates ceil(d_hidden / 32) floats per max_n row for partial sums.  With a router attached, tlr_route_ex computes
 * the learned score of every row when opt->score_source == TLR_SCORE_MLP or opt->mlp_score_dev != NULL; token, conf
 * and entropy are produced as always.  Where the tensor-core projection kernel runs (bf16 head, d % 8 == 0, W1
 * 16-byte aligned) the rows of W1 are walked by that same launch as one more work unit per 128 or 256 token rows --
 * same staged hidden states, same MMAs, an epilogue that applies b1, ReLU and w2 and sums -- so the step keeps its
 * two launches; otherwise one extra small kernel computes the score on CUDA cores.
 * Errors: TLR_ERR_ARG, TLR_ERR_NOMEM.  tlr_route_ex returns TLR_ERR_ARG when the learned score is
 * requested but no router is attached.
 */
tlr_status tlr_set_router_mlp(tlr_ctx* ctx, int32_t d_hidden, const void* W1_bf16_dev, const float* b1_dev,
                              const float* w2_dev, float b2);

tlr_status tlr_route_ex(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, float tau,
                        const tlr_route_options* opt, int32_t* token_dev, float* conf_dev,
                        float* entropy_dev, uint8_t* route_mask_dev, int32_t* routed_idx_dev,
                        int32_t* routed_count_dev, void* cuda_stream);

/*
 * tlr_shard_summary / tlr_shard_finish -- the routing step with the vocabulary sharded over several
 * GPUs (one process per GPU).  The paper decodes on one device; this is the data-parallel
 * restatement for decode batches, where streaming W from HBM dominates the step (the LM-head
 * contraction on the hidden state of Sec. 3.3, the decision of Sec. 3.1): GPU g holds the
 * contiguous rows [v_offset, v_offset + V) of the full W, and its context is created on that block.
 *
 * tlr_shard_summary runs the projection over the shard and writes, for each of the n rows, one
 * 16-byte summary {float m; int32 idx; float s; float t} into summary_dev[n] (device, 16-byte
 * aligned, caller-owned): m = the largest logit in the shard, idx = the lowest GLOBAL vocabulary
 * index attaining it (v_offset already added), s = sum exp(z - m), t = sum exp(z - m)(z - m) over
 * the shard.  No decision is taken.  The caller then exchanges the summaries -- an all-gather of
 * n x 16 bytes per GPU, NCCL in the Python helper -- into a block laid out [shards][n].
 *
 * tlr_shard_finish merges the `shards` summaries of every row (the same associative rule that merges
 * the chunks of one GPU; ties go to the lower index), and produces the six outputs of tlr_route.
 * Any context of the same max_n can run it; 1 <= shards <= 192.  Same ownership, stream and error
 * rules as tlr_route; nothing is allocated.  The result differs from the one-GPU result only by
 * fp32 summation order (conf and entropy agree to a few ulp; token, route_mask, routed_idx and
 * routed_count are identical unless a row sits within rounding of a tie or of tau).
 */
tlr_status tlr_shard_summary(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, int32_t v_offset, void* summary_dev,
                             void* cuda_stream);
tlr_status tlr_shard_finish(tlr_ctx* ctx, const void* summaries_dev, int32_t shards, int32_t n, float tau,
                            int32_t* token_dev, float* conf_dev, float* entropy_dev, uint8_t* route_mask_dev,
                            int32_t* routed_idx_dev, int32_t* routed_count_dev, void* cuda_stream);

/*
 * tlr_shard_attach / tlr_shard_push / tlr_shard_finish_fused -- the vocabulary-sharded step with the exchange
 * fused into the kernels (the per-token decision of Sec. 3.1 sits on the decode critical path -- Table 1,
 * "TBT for SLM" -- so at decode sizes the exchange latency is what sharding must not add back): instead of an
 * all-gather between two calls, every GPU STORES its per-row summaries straight into a block of every peer's
 * memory and then sets a flag there; the peer's merge kernel waits for the flags of all ranks.  Peer stores
 * only: nothing is loaded from a peer, nothing is multicast.
 *
 * Each GPU owns one exchange block of tlr_shard_block_bytes(max_n, shards) bytes (max_n as given to tlr_create
 * on every rank), 256-byte aligned, that all peers can write (peer-mapped or symmetric memory), ZEROED by its
 * owner before the first call.  Layout: 2 x shards uint32 flags, padded to 256 bytes, then 2 x shards slots of
 * max_n summaries of 16 bytes; the two sets alternate from call to call, so a rank that is one call ahead
 * does not overwrite what a slower peer still reads.
 *
 * tlr_shard_attach   rank in [0, shards), shards <= 192; peer_block_dev is a HOST array of `shards` device
 *                    pointers, entry g = GPU g's block as addressable from this GPU (entry `rank` = this GPU's
 *                    own block).  Allocates four small pointer tables; resets the call counter.  The blocks are
 *                    BORROWED for the life of the context.
 * tlr_shard_push     projection over this rank's rows of W (context created on them; v_offset = index of its
 *                    first row in the full vocabulary), then one kernel that folds the chunk partials into the
 *                    per-row summaries, stores them into this rank's slot on every peer and, after a
 *                    system-wide fence, sets this rank's flag on every peer to the call number.
 * tlr_shard_finish_fused  waits until the flags of all ranks in this GPU's block hold the current call number
 *                    (bounded: after 2 s -- or the limit given to tlr_debug_inject -- the kernel raises
 *                    TLR_DEV_WAIT_TIMEOUT and finishes on what is there), then merges the summaries in place
 *                    and produces the six outputs of tlr_route.
 * Every rank makes the same sequence of calls with the same n: push, finish, push, finish, ...  Stream,
 * ownership and error rules as tlr_route; only tlr_shard_attach allocates.
 * Errors: TLR_ERR_ARG (also: not attached, or finish before the first push), TLR_ERR_ALIGN,
 * TLR_ERR_TOO_MANY_ROWS, TLR_ERR_UNSUPPORTED, TLR_ERR_NOMEM, TLR_ERR_CUDA.
 */
size_t tlr_shard_block_bytes(int32_t max_n, int32_t shards);
tlr_status tlr_shard_attach(tlr_ctx* ctx, int32_t rank, int32_t shards, void* const* peer_block_dev);
tlr_status tlr_shard_push(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, int32_t v_offset, void* cuda_stream);
tlr_status tlr_shard_finish_fused(tlr_ctx* ctx, int32_t n, float tau, int32_t* token_dev, float* conf_dev,
                                  float* entropy_dev, uint8_t* route_mask_dev, int32_t* routed_idx_dev,
                                  int32_t* routed_count_dev, void* cuda_stream);

/*
 * tlr_rows_merge -- row-sharded batches (every GPU routes its own rows of a large batch with its own copy of
 * W; positions are independent, Sec. 3.1): turns the ranks' routed-index lists into ONE ascending list of
 * global row numbers.  gathered_idx_dev is int32 [ranks][cap] (slot g = rank g's routed_idx, as an all-gather
 * with slots of `cap` entries delivers it), counts_dev int32 [ranks] (the ranks' routed_count) and
 * row_offsets_dev int32 [ranks] (global number of rank g's first row; ascending with g).  Writes
 * global_idx_dev[0 .. total) = the lists of rank 0, 1, ... back to back with each rank's offset added, and
 * *global_count_dev = total = the sum of the counts.  global_idx_dev needs room for that sum (at most
 * ranks * cap).  All device memory, caller-owned; needs no context; asynchronous on cuda_stream.
 * Errors: TLR_ERR_ARG, TLR_ERR_CUDA.
 */
tlr_status tlr_rows_merge(const int32_t* gathered_idx_dev, const int32_t* counts_dev, const int32_t* row_offsets_dev,
                          int32_t ranks, int32_t cap, int32_t* global_idx_dev, int32_t* global_count_dev,
                          void* cuda_stream);

/*
 * tlr_route_host -- the same step with HOST buffers: brings h to the device, runs
 * tlr_route with the six results written straight into a pinned, device-visible buffer of
 * the context, synchronises the stream and hands them out to the caller's buffers.  Host
 * buffers may be pageable or pinned.  A pinned (or registered), 16-byte aligned h of up to
 * 4 MB is fetched by a copy kernel rather than the copy engine, so that the projection
 * kernel is launched, and streams W, while h is still on its way; anything else goes
 * through cudaMemcpyAsync.  Not reentrant on one context.  Output
 * pointers may be NULL to skip that copy, except routed_count_host.  routed_idx_host
 * needs capacity n; only the first *routed_count_host entries are written.
 * Same errors as tlr_route, plus TLR_ERR_DEVICE_STATUS when a kernel raised
 * TLR_DEV_WAIT_TIMEOUT (outputs are then not to be trusted).  The flag stays raised, and
 * this call keeps returning that code, until tlr_last_device_status has read it.
 */
tlr_status tlr_route_host(tlr_ctx* ctx, const void* h_bf16_host, int32_t n, float tau,
                          int32_t* token_host, float* conf_host, float* entropy_host,
                          uint8_t* route_mask_host, int32_t* routed_idx_host,
                          int32_t* routed_count_host, void* cuda_stream);

/*
 * tlr_route_host_submit / tlr_route_host_collect -- tlr_route_host in two halves, so that a caller can keep TWO
 * calls in flight: while the GPU works on one batch the host hands in the next, and the transfer of its hidden
 * states over PCIe, the kernels' launch and the wake-up of the host overlap the previous batch's kernels
 * (a serving loop that decodes for many sessions has the next batch ready before the last one is back).
 *   submit   enqueues the copy of h to the device, the routing step and the write-back of its results into a
 *            pinned block of the context, and returns without waiting.  h_bf16_host must hold the batch when
 *            submit is called (the GPU may start reading it while earlier work in the stream is still running;
 *            that work must therefore not be what produces it) and must stay valid and unchanged until the
 *            matching collect has returned.  At most two submitted calls may be waiting to
 *            be collected (a third returns TLR_ERR_ARG); all on one stream, or on streams the caller orders.
 *   collect  waits for the OLDEST submitted call and hands out its results exactly as tlr_route_host does
 *            (same optional pointers, same TLR_ERR_DEVICE_STATUS rule); TLR_ERR_ARG if none is waiting.
 * tlr_route_host is submit followed by collect and returns TLR_ERR_ARG while submitted calls are waiting.
 * Nothing is allocated (tlr_create sets up two staging slots).
 */
tlr_status tlr_route_host_submit(tlr_ctx* ctx, const void* h_bf16_host, int32_t n, float tau, void* cuda_stream);
tlr_status tlr_route_host_collect(tlr_ctx* ctx, int32_t* token_host, float* conf_host, float* entropy_host,
                                  uint8_t* route_mask_host, int32_t* routed_idx_host, int32_t* routed_count_host);

/*
 * tlr_create_fp8 -- bind an 8-bit copy of the LM head for DECODE batches (the per-token step of
 * Sec. 3.1 / 3.3 at the sizes where it is the time to read W): W_e4m3_dev holds e4m3 codes (OCP
 * 8-bit float: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities, 0x7f / 0xff
 * are NaN), row-major [V, d], 16-byte aligned, and wscale_dev one float per row, so that
 * W[v][k] = wscale[v] * value(code[v][k]).  Both are device memory, BORROWED for the life of the
 * context.  d must be a multiple of 16.  Calls on this context accept n <= 128 rows
 * (TLR_ERR_UNSUPPORTED above: larger batches are bound by the tensor cores, not by HBM, and gain
 * nothing from a smaller W); h stays bf16 and is NOT rounded to 8 bits -- each call splits it
 * into two e4m3 parts whose sum is the bf16 value (exact down to 2^-10 of a row's largest
 * element), so the result is that of the bf16 path run on the de-quantised W, to fp32 rounding.
 * All other calls (tlr_route, tlr_route_ex, tlr_route_host, ...) work on the context unchanged;
 * tlr_set_path(TLR_PATH_SIMT) is not available.  Allocates like tlr_create, plus 2 x 128 x d bytes.
 */
tlr_status tlr_create_fp8(int32_t d, int32_t V, const void* W_e4m3_dev, const float* wscale_dev, int32_t max_n,
                          tlr_ctx** out);

/* tlr_destroy -- free the context's workspace.  W is left alone.  NULL is TLR_OK. */
tlr_status tlr_destroy(tlr_ctx* ctx);

/* Static, never-NULL description of a status code. */
const char* tlr_status_string(tlr_status s);

/*
 * tlr_last_device_status -- read and clear the device status word (an OR of TLR_DEV_*
 * bits raised by kernels since the last read).  Synchronises the device.
 */
tlr_status tlr_last_device_status(tlr_ctx* ctx, uint32_t* out_host);

/* tlr_set_path -- force the projection kernel (tests, diagnostics).  TLR_ERR_UNSUPPORTED
 * if the shape cannot run on the requested path. */
tlr_status tlr_set_path(tlr_ctx* ctx, tlr_path path);

/*
 * tlr_debug_inject -- test hook for the kernels' failure handling.  Every barrier wait inside
 * the projection kernel is bounded; when one runs out the kernel raises TLR_DEV_WAIT_TIMEOUT,
 * lets its copies in flight land, frees its tensor memory and returns, and the context stays
 * usable.  kind = 1 makes the next calls' W producer issue no copies, so the consumer's wait
 * runs out (nothing faults, traps or spins forever); wait_limit_ms shortens the limit of every
 * wait (0 = default, 2 s).  kind = 0 restores normal operation.  Tensor-core path only.
 */
tlr_status tlr_debug_inject(tlr_ctx* ctx, int32_t kind, uint32_t wait_limit_ms);

/*
 * tlr_debug_plan_tiles -- host-only view of the tensor-core kernel's static schedule for n rows,
 * a vocabulary of V and sm_count SMs (no GPU needed; used by the CPU tests of the planner).
 * mlp_hidden > 0 plans the launch with a learned router of that hidden width inside it: the rows of
 * its first layer are walked as one more unit per row unit and are reported as vocabulary rows
 * V .. V + mlp_hidden (rounded up to the granule).
 * Writes up to `capacity` records of five int32 {worker, unit, first token row, first vocabulary
 * row, vocabulary rows} -- one per tile, in the order the workers walk them -- and the total
 * number of tiles to *count.  plan_out (optional) receives grid, chunks, row units and, in
 * `reserved`, the granule size in rows.
 */
tlr_status tlr_debug_plan_tiles(int32_t n, int32_t V, int32_t sm_count, int32_t mlp_hidden, int32_t* out,
                                int32_t capacity, int32_t* count, tlr_plan* plan_out);

/*
 * tlr_debug_shard_table -- host-only: the addresses tlr_shard_attach derives for one rank and one parity of the
 * call counter from the ranks' exchange-block addresses (no GPU needed; used by the CPU tests of the layout).
 * slot_out[g] / flag_out[g] = where rank `rank` stores its summaries / its flag on peer g.
 */
tlr_status tlr_debug_shard_table(int32_t max_n, int32_t rank, int32_t shards, void* const* peer_block_dev,
                                 int32_t parity, void** slot_out, void** flag_out);

/* tlr_plan_query -- the launch plan a call with n rows would use.  No device work. */
tlr_status tlr_plan_query(tlr_ctx* ctx, int32_t n, tlr_plan* out);

/*
 * tlr_set_kernel_timing -- when enabled, every tlr_route call brackets its projection
 * kernel (the dominant one) with CUDA events on the call's stream.
 * tlr_read_kernel_timing synchronises those events and returns the number of bracketed
 * launches since the last read and their summed device time in milliseconds, then
 * resets the tally.  At most 4096 launches are kept between reads.
 */
tlr_status tlr_set_kernel_timing(tlr_ctx* ctx, int32_t enabled);
tlr_status tlr_read_kernel_timing(tlr_ctx* ctx, int32_t* launches_out, float* total_ms_out);

/*
 * tlr_route_static -- the routing step for callers that cannot allocate device memory.
 * (No counterpart in the paper: this is a deployment convenience of the library.)
 *
 * Who needs it: a serving process that has already given all free HBM to its own pools,
 * so that a cudaMalloc would fail or disturb them; a decode loop that cannot tolerate the
 * device-wide synchronisation an allocation may cause; a plug-in whose host forbids
 * allocation in its callbacks.  tlr_create allocates a workspace, so such callers cannot
 * use it; this call needs no context and calls no cudaMalloc, cudaFree or other
 * allocating routine.  Its scratch (per-row partial results and a ticket counter) is a
 * fixed array inside the library image, about 3 MiB, which every GPU that loads the
 * library holds until the process exits.
 *
 * Arguments are those of tlr_create + tlr_route: d, V and W (bf16 [V,d], 16-byte aligned,
 * only read), then h, n, tau and the six outputs with the same layouts and meaning.
 *   n           0 <= n <= TLR_STATIC_MAX_ROWS; more rows return TLR_ERR_TOO_MANY_ROWS
 *               (the fixed scratch cannot hold them; use a context for larger batches).
 *   status_dev  optional uint32 [1] on the device: receives the TLR_DEV_* flags of this
 *               call (cleared at its start).  NULL keeps the flags in the scratch, unread.
 * Asynchronous on cuda_stream like tlr_route.
 *
 * The first call on each device performs a one-time set-up for that device (it looks up
 * the scratch array's device address and opts the kernels in to their shared-memory
 * size); make that first call outside any stream capture.  All calls share the one
 * scratch array, which keeps the previous call's contents (the call clears what must
 * start at zero): calls must not overlap on the GPU -- issue them on one stream, or
 * order them yourself; two calls in flight at once race.
 * Errors: TLR_ERR_ARG, TLR_ERR_ALIGN, TLR_ERR_TOO_MANY_ROWS, TLR_ERR_UNSUPPORTED (device
 * is not sm_100), TLR_ERR_CUDA.
 */
#define TLR_STATIC_MAX_ROWS 1024
tlr_status tlr_route_static(int32_t d, int32_t V, const void* W_bf16_dev, const void* h_bf16_dev,
                            int32_t n, float tau, int32_t* token_dev, float* conf_dev,
                            float* entropy_dev, uint8_t* route_mask_dev, int32_t* routed_idx_dev,
                            int32_t* routed_count_dev, uint32_t* status_dev, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TLR_H_ */
