/*
 * tova.h - C ABI of the bounded multi-state (KV cache) decode step with TOVA
 * eviction, for NVIDIA B200 (sm_100a).
 *
 * A transformer layer is run as a bounded multi-state RNN (Section 3.3 of
 * "Transformers are Multi-State RNNs"): the state of a layer is the pair
 * (K, V) with at most `capacity` rows per sequence.  One decoding step appends
 * the new token's (k, v) to the state (Eq. 6), attends with the new query over
 * all rows (Eq. 4, Eq. 7) and, once the appended state holds capacity+1 rows,
 * drops the row whose attention weight, averaged over the query heads of the
 * layer, is lowest (Section 4, Eq. 9, Algorithm 1).
 *
 * General conventions
 *  - One tova_cache holds the state of ONE layer for `batch` independent
 *    sequences that advance in lock step (one token each per call).
 *  - Unless a parameter says "host", every tensor pointer is a DEVICE pointer,
 *    16-byte aligned, contiguous in the stated layout, owned by the caller.
 *    The library allocates no device memory: the caller provides one block of
 *    tova_cache_bytes() bytes at init, which must outlive the handle.
 *  - q, k, v have the cache's dtype (fp32 or bf16); outputs are fp32.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *    the default stream) and return without synchronising.  All calls on one
 *    cache must be issued on one stream or otherwise ordered by the caller.
 *  - Return value: TOVA_OK or a negative tova_status.  Argument errors are
 *    detected on the host before anything is launched.  There is no CPU
 *    fallback: without a usable CUDA device the calls fail with TOVA_ERR_CUDA.
 *  - Keys are cached as given (callers pass post-RoPE q and k); positions are
 *    metadata that travel with the rows, so eviction never re-rotates a key.
 */
#ifndef TOVA_H_
#define TOVA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tova_cache tova_cache; /* opaque host handle */

enum { TOVA_DTYPE_FP32 = 0, TOVA_DTYPE_BF16 = 1 };

/* Pass as `pos` / `first_pos`: the token's position is the previous token's
 * position in this cache plus one (0 for the first token), taken from a
 * counter on the device; a recorded sequence of steps (a CUDA graph) can then
 * be replayed and still give every token a fresh position. */
#define TOVA_POS_AUTO (-1)

typedef enum {
  TOVA_OK = 0,
  TOVA_ERR_NULL = -1,        /* a required pointer is NULL                        */
  TOVA_ERR_BAD_SHAPE = -2,   /* batch/heads/capacity/n_tokens out of range        */
  TOVA_ERR_UNSUPPORTED = -3, /* head_dim not in {64,128}, unknown dtype           */
  TOVA_ERR_ALIGN = -4,       /* a device pointer is not 16-byte aligned           */
  TOVA_ERR_WORKSPACE = -5,   /* dev_bytes < tova_cache_bytes()                    */
  TOVA_ERR_FULL = -6,        /* evict == 0 and the state already holds capacity   */
  TOVA_ERR_CUDA = -7,        /* a CUDA runtime call or launch failed              */
  TOVA_ERR_DEVICE = -8,      /* a kernel reported a failed internal check         */
  TOVA_ERR_STATIC_LIMIT = -9 /* tova_decode_step_static: shape exceeds the built-in scratch */
} tova_status;

typedef struct {
  int32_t batch;      /* B >= 1 sequences                                          */
  int32_t n_q_heads;  /* H >= 1 query heads                                        */
  int32_t n_kv_heads; /* Hkv >= 1, H % Hkv == 0 (H == Hkv: MHA, else GQA)          */
  int32_t head_dim;   /* D in {64, 128}                                            */
  int32_t capacity;   /* k >= 1 rows per sequence (the multi-state size)           */
  int32_t dtype;      /* TOVA_DTYPE_FP32 or TOVA_DTYPE_BF16 for q, k, v, K, V      */
  float sm_scale;     /* logit scale; 0 selects 1/sqrt(head_dim)                   */
  int32_t evict;      /* 1: TOVA policy; 0: unbounded arm (a full state is an error) */
} tova_config;

/* Device bytes a cache of this shape needs (K, V, positions, lengths, the
 * logit / partial-result scratch, counters, status, host-call staging).
 * Returns 0 when the configuration is invalid. */
size_t tova_cache_bytes(const tova_config* cfg);

/* Create a cache in caller-provided device memory `dev_mem` (256-byte aligned,
 * dev_bytes >= tova_cache_bytes(cfg)) and enqueue its initialisation (empty
 * state: length 0, positions -1).  The multi-state H_0 is empty (Section 3.1).
 * `*out` receives a host handle to be released with tova_cache_destroy. */
int tova_cache_init(tova_cache** out, const tova_config* cfg, void* dev_mem, size_t dev_bytes,
                    void* cuda_stream);

/* One decoding step of the layer for every sequence (Eq. 6, Eq. 4, Eq. 7,
 * then Algorithm 1 / Eq. 9):
 *   q [B,H,D], k and v [B,Hkv,D]   the new token's projections (cache dtype)
 *   pos                            its original position (metadata), or TOVA_POS_AUTO
 *   out [B,H,D] fp32               attention output over all n+1 rows, the
 *                                  row dropped at this step included
 *   evicted_pos [B] int32 or NULL  position of the dropped token; -1 when the
 *                                  state was not full; `pos` when the new
 *                                  token itself was dropped
 * The new token takes the dropped row's slot in place (slot order is not
 * position order).  Ties of the arg-min go to the lowest slot, the new token
 * counting as slot `capacity`. */
int tova_decode_step(tova_cache* c, const void* q, const void* k, const void* v, int32_t pos,
                     float* out, int32_t* evicted_pos, void* cuda_stream);

/* The same per-token policy run over n_tokens consecutive prompt tokens at
 * positions first_pos, first_pos+1, ... (first_pos = TOVA_POS_AUTO continues
 * from the previous token): the state, the dropped positions and every later
 * step are identical to n_tokens calls of tova_decode_step.
 *   q [T,B,H,D], k and v [T,B,Hkv,D]; out [T,B,H,D] fp32 or NULL;
 *   evicted_pos [T,B] or NULL.
 * Tokens that find a free row are never followed by a deletion (the state
 * holds g(t) = min(t, k) tokens, Section 3.3; Algorithm 1 returns early while
 * the cache is within its size), so for them Eq. 6-7 are ordinary causal
 * attention.  On bf16 states a run of at least 4 such tokens is therefore
 * processed in bulk - one copy of the rows, one tensor-core causal-attention
 * kernel (skipped when out is NULL; tcgen05 with accumulators in tensor memory
 * where head_dim is 128), one small commit kernel - instead of
 * token by token; its outputs equal the per-token ones up to floating-point
 * summation order (within the library's output tolerance), everything else
 * bit for bit.  The tokens that remain once the state is full are processed
 * one at a time, or - where tova_cache_set_prefill_workspace has given the
 * cache a workspace - in chunks of up to 64 tokens (see there).
 * tova_cache_set_bulk_prefill(c, 0) forces the per-token route for all of
 * them (then outputs are bit-identical to decode steps). */
int tova_prefill(tova_cache* c, const void* q, const void* k, const void* v, int32_t n_tokens,
                 int32_t first_pos, float* out, int32_t* evicted_pos, void* cuda_stream);

/* Prompt tokens that meet a FULL state, many per launch.  Each of them drops a
 * row (Algorithm 1) and thereby changes what the next one attends to; the
 * paper's language-modelling runs handle whole chunks of tokens at once by
 * masking the attention according to the layer's attention weights (appendix
 * "Experimental Details").  With a workspace, tova_prefill does the same,
 * exactly: per chunk of up to 64 tokens one dense pass computes the logits of
 * all its queries against the state as the chunk found it and against the
 * chunk's own tokens, one thread block per sequence replays the chunk's
 * deletions in order from those logits alone (the same candidates, head-averaged
 * weights and arg-min as token-by-token steps), a second dense pass forms the
 * outputs with every query's weights masked to the rows alive at its step, and
 * the surviving tokens are written to the slots they took.  Five launches per
 * 64 tokens instead of 128.  Results equal token-by-token processing up to
 * floating-point summation order (the library's output tolerance; a victim may
 * differ only between candidates whose averages differ by rounding).
 *   tova_prefill_workspace_bytes   device bytes needed (about
 *        B*H*64*(capacity+64)*4 for the logits); 0 for an invalid or fp32
 *        configuration.
 *   tova_cache_set_prefill_workspace   dev_mem: 256-byte aligned device memory of
 *        at least that size, owned by the caller, to outlive the handle (or
 *        until replaced; NULL switches the chunked route off).  It may be
 *        shared by caches of one shape whose calls are ordered on one stream.
 *        TOVA_ERR_UNSUPPORTED for fp32 states and for capacities beyond what the
 *        deletion kernel's shared memory holds (about 25,000 rows).
 * Used for the TOVA and Window policies (with or without protected first positions) on bf16
 * states, for runs of at least 8 tokens; everything else takes the per-token
 * route as before. */
size_t tova_prefill_workspace_bytes(const tova_config* cfg);
int tova_cache_set_prefill_workspace(tova_cache* c, void* dev_mem, size_t dev_bytes);

/* Tuning of the chunked prompt route: thread blocks per sequence in the kernel
 * that replays a chunk's deletions.  0 (default): as many as keep all
 * sequences resident at once, up to 8, as one thread-block cluster with the
 * logits staged in shared memory; 1, 2, 4, 8: that many; -1: one block per
 * sequence reading the logits from global memory (also taken where not even
 * one token's logits fit the shared memory).  Results do not depend on it
 * beyond floating-point summation order.  Other values: TOVA_ERR_BAD_SHAPE. */
int tova_cache_set_chunk_cluster(tova_cache* c, int32_t ctas);

/* ... and how the blocks of such a cluster meet.  0 (default): once per token
 * where the logits of two tokens fit the shared memory (a token's normaliser is
 * then the row sum minus the terms of the rows dropped so far, and candidates
 * are scored in one pass), else twice per token; 2: always twice (normaliser
 * summed over the live rows, then the scores).  Same results up to
 * floating-point summation order.  Other values: TOVA_ERR_BAD_SHAPE. */
int tova_cache_set_chunk_barriers(tova_cache* c, int32_t per_token);

/* tova_decode_step with HOST buffers; returns after `cuda_stream` has been
 * synchronised, when out (and evicted_pos if not NULL) hold the results.
 * Page-locked buffers (pinned or registered, 16-byte aligned; all of them):
 * the kernels read q, k, v over the bus (directly, or through one small fetch
 * kernel when many warps share them) and write the outputs in place - no
 * copy calls.
 * Otherwise (pageable memory) q, k, v are copied to the device, the step runs
 * and the results are copied back, all on `cuda_stream`. */
int tova_decode_step_host(tova_cache* c, const void* q_host, const void* k_host,
                          const void* v_host, int32_t pos, float* out_host,
                          int32_t* evicted_pos_host, void* cuda_stream);

/* Copy the state out (device to DEVICE buffers of the caller; any may be NULL):
 *   len [B] int32, positions [B,capacity] int32 in slot order (-1 = unused),
 *   k_out, v_out [B,Hkv,capacity,D] in the cache dtype,
 *   status [1] int32: 0, or a nonzero code left by a failed device-side check. */
int tova_cache_read(const tova_cache* c, int32_t* len, int32_t* positions, void* k_out,
                    void* v_out, int32_t* status, void* cuda_stream);

/* Deferred eviction (off by default).  The attention output of a step is what
 * the rest of a model waits for; which row is dropped (Algorithm 1) only has
 * to be settled before the SAME cache sees its next token, a whole model pass
 * later.  With on != 0, tova_decode_step enqueues attention and output on the
 * caller's stream, while the head average, the arg-min and the in-place insert
 * run on a stream the cache owns and overlap whatever the caller enqueues
 * next (normally the next layer's step).  Consequences for the caller:
 *   - `out` is ready in stream order as before; `evicted_pos`, and the state as
 *     tova_cache_read sees it, are ready only after tova_cache_join;
 *   - the next tova_decode_step / tova_prefill on this cache waits for the
 *     pending eviction by itself; the k and v buffers may be reused at once
 *     (the library keeps copies), `evicted_pos` must stay valid until the join;
 *   - when capturing a CUDA graph, call tova_cache_join on the capturing
 *     stream for every cache before the capture ends, and have no eviction
 *     pending when it begins.
 * Results are identical to the default mode.  tova_prefill and
 * tova_decode_step_host always run undeferred.  Switching off with an eviction
 * pending is refused (TOVA_ERR_BAD_SHAPE): join first. */
int tova_cache_set_deferred_eviction(tova_cache* c, int32_t on);

/* Make `cuda_stream` wait for this cache's pending deferred eviction, if any. */
int tova_cache_join(tova_cache* c, void* cuda_stream);

/* Tuning: rows of the state one warp of the streaming kernel covers (a multiple
 * of 32 up to 8192; 0 restores the automatic choice made at init).  Results do
 * not depend on it beyond floating-point summation order. */
int tova_cache_set_chunk_rows(tova_cache* c, int32_t rows);

/* Other compression policies of the paper, on the same streaming kernels (only
 * the choice of the row to drop changes; the attention output of a step never
 * depends on it):
 *   TOVA_POLICY_TOVA (default)   the row with the lowest head-averaged attention
 *          weight goes (Section 4, Algorithm 1);
 *   TOVA_POLICY_WINDOW           first in, first out: the row holding the earliest
 *          position goes (Section 4.1, "Window");
 *     for these two, arg = i >= 0: rows holding positions 0..i-1 are never dropped:
 *          Window+i (Section 4.1) and TOVA+i (appendix ablation); i < capacity;
 *   TOVA_POLICY_TOVA_HEAD        every head drops the row with ITS lowest weight, so
 *          heads come to hold different tokens (Section 4; appendix ablation,
 *          "TOVA-head"); arg must be 0;
 *   TOVA_POLICY_H2O_LAYER, TOVA_POLICY_H2O_HEAD   a window of the most recent tokens
 *          always stays; among the older rows the one whose attention weight, summed
 *          over all the steps it has spent in the state, is lowest goes (Section 4.1,
 *          "H2O"), with weights averaged over the layer's heads or per head;
 *          arg = size of the recent window, 1..capacity, or 0 for capacity minus
 *          half the capacity (the paper's setting: half the state for non-window rows).
 * Under grouped-query attention the "head" that owns rows is a KV head, scored by
 * the mean weight of the query heads that read it.  For the head-wise policies
 * evicted_pos of the step calls is [B,Hkv] ([T,B,Hkv] for tova_prefill) and
 * tova_cache_read returns positions as [B,Hkv,capacity]: one slot table per KV head.
 * Allowed only while the state is empty (before the first token), else
 * TOVA_ERR_BAD_SHAPE; an unknown policy gives TOVA_ERR_UNSUPPORTED.  Positions
 * passed to the step calls must be >= 0, distinct and increasing for Window, "+i"
 * and H2O to mean what the paper describes; ties go to the lowest slot as
 * everywhere.  H2O processes prompts token by token (its scores accumulate from
 * the first token on); head-wise TOVA takes the bulk route for prompt tokens that
 * find free rows and goes token by token from there.  With deferred eviction
 * their victim choice and insert run on the cache's stream like the layer
 * policies'.  Not available through tova_decode_step_static. */
#define TOVA_POLICY_TOVA 0
#define TOVA_POLICY_WINDOW 1
#define TOVA_POLICY_TOVA_HEAD 2
#define TOVA_POLICY_H2O_LAYER 3
#define TOVA_POLICY_H2O_HEAD 4
int tova_cache_set_policy(tova_cache* c, int32_t policy, int32_t arg);

/* H2O policies: copy out the accumulated attention weight of every slot
 * (Section 4.1), scores [B,U,capacity] fp32 on the DEVICE, U = 1 (layer-wise) or
 * Hkv (head-wise); entries of unused slots are 0.  TOVA_ERR_UNSUPPORTED under
 * any other policy. */
int tova_cache_read_scores(const tova_cache* c, float* scores, void* cuda_stream);

/* Slot tables this cache keeps per sequence: Hkv under a head-wise policy, else 1. */
int32_t tova_cache_units(const tova_cache* c);

/* Position compression for streams longer than the model's training context
 * (Section "Extrapolation with TOVA").  The positional encoding of the cached
 * tokens is adapted so that no distance unseen in training occurs: between
 * neighbouring retained tokens (in position order, the new token last) a gap g
 * becomes ln(ln(g)), and stays g while g <= 10; the new positions accumulate
 * along that chain, the earliest retained token at 0 (attention depends on
 * differences only).  In this mode the LIBRARY applies the rotary embedding:
 * callers pass q and k WITHOUT it, keys are cached as given, and at every step
 * the query and every cached key are rotated at their current compressed
 * position (rotate-half pairs d, d + D/2, angle p' * rope_base^(-2d/D), the
 * convention of the model families the paper runs; rope_base 10000 there).
 * Everything after the logits is the ordinary step, under the TOVA or Window
 * policy with or without protected first positions.
 *   tova_position_workspace_bytes  device bytes needed: a (cos, sin) table of
 *        B*(capacity+1)*D/2 pairs, the rotated query, the positions.
 *   tova_cache_set_position_compression  dev_mem: 256-byte aligned device
 *        memory of that size, owned by the caller, to outlive the handle (NULL:
 *        off); only while the state is empty; capacity up to 8191 rows
 *        (TOVA_ERR_UNSUPPORTED beyond, and together with head-wise policies or
 *        sharding).  The step then takes three launches and a slower streaming
 *        kernel (a table read and a rotation per cached row); prompts go token
 *        by token; deferred eviction is ignored.
 *   tova_cache_read_compressed_positions  cpos [B,capacity+1] doubles on the
 *        DEVICE: the positions the LAST step used, by slot, the new token's at
 *        index min(tokens before it, capacity). */
size_t tova_position_workspace_bytes(const tova_config* cfg);
int tova_cache_set_position_compression(tova_cache* c, void* dev_mem, size_t dev_bytes, float rope_base);
int tova_cache_read_compressed_positions(const tova_cache* c, double* cpos, void* cuda_stream);

/* One layer sharded by KV head over several GPUs (one process per GPU).
 * Algorithm 1 averages the last query's weights over the heads of the layer - a
 * sum over heads - so ranks that each hold some of the KV heads (with the
 * query heads that read them) only have to exchange, once a row is due to go,
 * their partial head sums: one fp32 vector of capacity+1 entries per sequence.
 * Everything else of the step (Eq. 4, Eq. 6, Eq. 7, the insert of Eq. 9) is
 * local to a rank's heads.  A sharded cache is created like any other, with
 * cfg.n_q_heads / cfg.n_kv_heads = the heads THIS rank holds, and then:
 *
 *   tova_cache_set_shard(c, rank, world, n_q_heads_total, peer_tables, peer_flags)
 *       while the state is empty; world <= 8; TOVA policy (with or without
 *       protected first positions).  Two ways to exchange:
 *       peer stores - peer_tables[r] / peer_flags[r] (HOST arrays of `world`
 *         DEVICE pointers) address rank r's score table of
 *         tova_shard_table_bytes(cfg, world) bytes and its `world` int32 flags
 *         (zeroed by the caller once), mapped into this process (CUDA IPC or
 *         symmetric memory; for a single-process emulation plain device
 *         memory).  The scores kernel stores this rank's partial sums into
 *         every rank's table with ordinary stores and raises its flag there;
 *         the commit kernel waits - bounded: a rank that never reports leaves
 *         status code 3 and the state untouched - and adds the parts in rank
 *         order, so every rank computes the same bits and the same victim;
 *       caller reduces - peer_flags = NULL: only peer_tables[rank] is used,
 *         [B, ld] floats with ld = capacity+1 rounded up to 4; between the two
 *         calls below the caller sums that vector over the ranks in place
 *         (e.g. an NCCL all-reduce on the same stream).
 *   tova_decode_step_scores(c, q, k, v, pos, out, stream)
 *       this rank's heads: q [B,H_local,D], k and v [B,Hkv_local,D]; attention
 *       output for them; the rank's partial head sums published.
 *   tova_decode_step_commit(c, k, v, evicted_pos, stream)
 *       the victim from the summed vector (arg-min, lowest slot on ties, the new
 *       token being slot `capacity`) and the insert into this rank's KV heads.
 *       evicted_pos [B] or NULL: the same on every rank.
 * The two calls alternate; tova_decode_step, tova_prefill and
 * tova_decode_step_host are refused (TOVA_ERR_BAD_SHAPE) on a sharded cache.
 * No TMA multicast and no library kernel reads or writes peer memory. */
size_t tova_shard_table_bytes(const tova_config* cfg, int32_t world);
int tova_cache_set_shard(tova_cache* c, int32_t rank, int32_t world, int32_t n_q_heads_total,
                         void* const* peer_tables, void* const* peer_flags);
int tova_decode_step_scores(tova_cache* c, const void* q, const void* k, const void* v, int32_t pos, float* out,
                            void* cuda_stream);
int tova_decode_step_commit(tova_cache* c, const void* k, const void* v, int32_t* evicted_pos, void* cuda_stream);

/* Tuning: where the per-chunk partial results of a head are merged into the
 * attention output (Eq. 7 evaluated chunk by chunk).  on (default): when the
 * state splits into at most 8 chunks, the streaming warps of a head group run
 * as one thread block and merge through shared memory, so the outputs are
 * final when the streaming kernel ends.  off: the partials go through global
 * memory to the second kernel.  Larger chunk counts always take the second
 * route.  Results do not depend on it beyond
 * floating-point summation order.  Returns TOVA_ERR_NULL for a null handle. */
int tova_cache_set_fused_merge(tova_cache* c, int32_t on);

/* Bulk processing of the prompt tokens that fill free rows (see tova_prefill;
 * used on bf16 states).  mode 1 (default): the causal attention of the run
 * goes through the tcgen05 / tensor-memory kernel where head_dim is 128, else
 * through the warp-level MMA kernel; mode 2: always the warp-level MMA kernel;
 * mode 0: every prompt token takes the decode kernels.  Returns TOVA_ERR_NULL
 * for a null handle, TOVA_ERR_BAD_SHAPE for any other mode. */
int tova_cache_set_bulk_prefill(tova_cache* c, int32_t mode);

/* Rows each sequence holds now, min(tokens fed, capacity) = g(t) of Section
 * 3.3, tracked on the host (sequences advance in lock step). */
int32_t tova_cache_len(const tova_cache* c);

/* Kernel launches issued for this cache so far (for benchmarks). */
int64_t tova_cache_launches(const tova_cache* c);

/* Release the host handle (device memory stays with the caller). */
int tova_cache_destroy(tova_cache* c);

const char* tova_strerror(int status);

/* One decode step WITHOUT any workspace from the caller and without a cache
 * handle (the paper has no counterpart: this is a packaging variant of
 * tova_decode_step, same kernels, same results).
 *
 * Who needs it: code that runs where device memory cannot be requested - a
 * plugin or callback inside another framework's execution engine that owns
 * the allocator, code between the begin and end of someone else's stream
 * capture, a process whose memory budget was fixed at start-up.  Such callers
 * usually do hold the K/V tensors themselves but have nowhere to put the
 * scratch the two kernels exchange (logits, per-chunk soft-max partials,
 * block minima, status words).  For this call that scratch is an array
 * compiled into the library: TOVA_STATIC_SCRATCH_BYTES (8 MiB) of device
 * memory that every GPU context loading the library holds until it exits.
 *
 *   cfg                          shape, dtype, scale, policy (as for tova_cache_init)
 *   K, V [B,Hkv,capacity,D]      the caller's state, updated in place (zero it before
 *                                the first token: rows not yet written are read with
 *                                weight zero and must hold finite numbers)
 *   positions [B,capacity] int32 slot table, updated in place (caller sets
 *                                unused slots to -1 before the first token)
 *   n_live                       rows each sequence holds before this token,
 *                                min(tokens fed so far, capacity): the caller
 *                                tracks it
 *   q, k, v, pos, out, evicted_pos   as for tova_decode_step (pos >= 0)
 *   status [1] int32 or NULL     device word that receives 0, or the code of a
 *                                device-side check this call failed (a copy that
 *                                did not land, an arg-min out of range); cleared
 *                                by the call.  With NULL such failures go
 *                                unreported: there is no handle to read them from
 *
 * Scratch need: about 4*B*H*(capacity+5) bytes of logits plus
 * B*H*(D*4+8)*ceil(capacity/chunk) bytes of partials (chunk = 32..256 rows,
 * chosen from the shape); the LLaMA-2-7B layer at batch 8, capacity 512 takes
 * under 1 MiB.  A shape that needs more than the array holds is refused with
 * TOVA_ERR_STATIC_LIMIT before anything is launched.
 *
 * The call allocates nothing, on the device or through any library.  Its first
 * use on a device looks up the array's device address (cudaGetSymbolAddress)
 * and the SM count, and the first use of each kind of shape (dtype, head_dim,
 * query-group size, state short or long) sets launch attributes of the kernels
 * it picks and may look up a driver entry point: make the first call on a
 * device, and the first call of every shape, outside any stream capture.
 * That one-time set-up is guarded, so first calls may come from several host
 * threads.  All calls on a device share the one array, which keeps whatever the
 * previous call left: the call clears its status words itself (a memset on
 * `cuda_stream`), but two calls whose kernels overlap on the GPU - different
 * streams, or different host threads without ordering - race on it.  Issue them
 * on one stream or order them with events. */
#define TOVA_STATIC_SCRATCH_BYTES (8u << 20)
int tova_decode_step_static(const tova_config* cfg, void* K, void* V, int32_t* positions,
                            int32_t n_live, const void* q, const void* k, const void* v, int32_t pos,
                            float* out, int32_t* evicted_pos, int32_t* status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TOVA_H_ */
