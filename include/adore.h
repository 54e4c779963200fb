/*
 * adore.h - C ABI of the ADORE decode path for NVIDIA B200 (sm_100a).
 *
 * ADORE (adaptive token release) keeps a fixed-capacity KV cache during decoding: a small
 * controller scores every token, the lowest-scoring cached token is released when a new one
 * arrives, and the most valuable released tokens are recomputed ("rebuilt") so that the next
 * attention can still see them. One decode step for one layer is
 *
 *   1. attention of the current query over the occupied cache slots plus the current token's
 *      own key/value, restricted to the K largest logits, with the per-slot weights emitted;
 *   2. (once per step, at layer 0) controller scoring of the new token, release of the least
 *      valuable retained token, in-place admission of the new token, choice of the rebuild list;
 *   3. rebuild: K/V projection of the listed tokens' layer-input rows, rotary embedding at the
 *      token's original position, scatter into the freed slots.
 *
 * Conventions
 *   - Every function returns an adore_status_t. Nothing throws, aborts or traps the device.
 *   - All device work is queued on the CUDA stream given at create time and is asynchronous;
 *     only adore_cache_sync_status, the host-buffer step calls (for their output), the state snapshot
 *     calls and adore_cache_destroy wait for the device.
 *   - "device" pointers are CUDA device addresses of the cache's GPU; "host" pointers are
 *     ordinary (ideally pinned) host memory. The library borrows per-call buffers until the
 *     stream has passed the call, and borrows projection weights until the cache is destroyed.
 *   - Element type T is float (ADORE_F32) or bfloat16 (ADORE_BF16), chosen at create time, for
 *     q, k, v, x, out, the cache and the projection weights. Row-major everywhere.
 *   - Argument errors are found on the host before anything is launched. Inconsistencies only
 *     the device can see (an explicit rebuild entry that is out of range, a bounded wait that
 *     ran out) set a bit in a device error word, turn the offending item into a no-op and are
 *     reported by adore_cache_sync_status.
 *   - A cache is not thread-safe; use one thread per cache.
 *
 * Sequences of one cache move in lockstep: all B sequences hold the same number of tokens n.
 */
#ifndef ADORE_H_
#define ADORE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adore_cache adore_cache_t; /* opaque; owned by the library */

typedef enum {
  ADORE_OK = 0,
  ADORE_ERR_INVALID_ARG = 1,      /* NULL where not allowed, size or enum out of range          */
  ADORE_ERR_OOM = 2,              /* device or host allocation failed                           */
  ADORE_ERR_TOKEN_TABLE_FULL = 3, /* n would exceed max_tokens                                  */
  ADORE_ERR_STATE = 4,            /* call order (e.g. layer l>0 before layer 0 of the step)     */
  ADORE_ERR_CUDA = 5,             /* a CUDA runtime/driver call failed                          */
  ADORE_ERR_DEVICE_FLAG = 6,      /* device error word set: bad explicit entry / bounds check   */
  ADORE_ERR_TIMEOUT = 7,          /* a bounded device-side wait gave up                         */
  ADORE_ERR_UNSUPPORTED = 8       /* shape outside what the kernels are built for               */
} adore_status_t;

typedef enum { ADORE_F32 = 0, ADORE_BF16 = 1 } adore_dtype_t;

/* How the rebuild list is chosen each step (Section 2.3, first sentence).
 * POLICY:   the min(R_max, #released) released tokens with the highest controller score.
 * EXPLICIT: the caller names candidate token positions per step; entries that are resident
 *           are dropped, duplicates removed, and if more than R_max remain the R_max with the
 *           highest score are kept. */
typedef enum { ADORE_REBUILD_POLICY = 0, ADORE_REBUILD_EXPLICIT = 1 } adore_rebuild_mode_t;

/* Slot roles in the slot map. */
enum { ADORE_SLOT_EMPTY = 0, ADORE_SLOT_RETAINED = 1, ADORE_SLOT_REBUILT = 2 };

/* Controller ablation "w/o GRU" (Section 3.5.3, Table 5): the cell keeps no memory. Every token is scored
 * from its own embedding alone, z_i = GRU(x_i, 0), then the same MLP. The paper does not say how the embedding
 * reaches the MLP without the GRU; applying the cell to a zero state needs no extra parameters. */
#define ADORE_FLAG_NO_RECURRENCE 1u
/* Score source of the H2O and H2O(Rebuilt) baselines (Section 3.1, items 6 and 7) on the same kernels: no controller;
 * a token's value is the attention weight it has received so far, summed over heads, layers and steps (float32). The
 * weights of a step count from the next step's selection on; prompt tokens start at zero, so a prompt is cut to its
 * most recent tokens. adore_decode_step then accumulates after every layer's attention (weights == NULL is fine: an
 * internal buffer is used); adore_step_begin returns ADORE_ERR_UNSUPPORTED. */
#define ADORE_FLAG_SCORE_FROM_ATTENTION 2u
/* Position feature of the controller read as the distance to the token being decoded (Section 1 and the caption of
 * Figure 2 speak of importance with respect to the current token, for all earlier tokens, cached or released; Eq. 2
 * itself only says "position embedding"): u = (n - i) / pos_scale, so every earlier token is scored anew at every
 * step, from the GRU state it had when it arrived, and the step's release and rebuild list rank by those fresh scores.
 * A prompt is scored once, as seen from its last token. adore_cache_scores() then shows tokens 0..n-1 as seen from
 * token n-1. Needs max_tokens * ctrl_hidden * 8 bytes per sequence more; not with ADORE_FLAG_SCORE_FROM_ATTENTION. */
#define ADORE_FLAG_RELATIVE_POSITION 4u

typedef struct {
  uint32_t struct_size;  /* sizeof(adore_config_t), for versioning                               */
  int32_t batch;         /* B  sequences                                                        */
  int32_t n_layers;      /* L                                                                   */
  int32_t n_heads;       /* H                                                                   */
  int32_t head_dim;      /* dh: 64 or 128                                                       */
  int32_t hidden;        /* d: controller input width and projection inner dimension            */
  int32_t capacity;      /* C  slots per sequence, 1 <= C <= 4096                               */
  int32_t rebuild_max;   /* R_max, 0 <= R_max < C; retained budget m = C - R_max (Section 2.3)   */
  int32_t topk;          /* K >= 1 of the attention mask (Section 2.2); K >= C+1 disables it     */
  int32_t max_tokens;    /* token-table rows per sequence, <= 8192                              */
  int32_t ctrl_hidden;   /* d' (Appendix B: 128), <= 256                                        */
  adore_dtype_t dtype;
  adore_rebuild_mode_t rebuild_mode;
  float rope_theta;      /* rotary base; 0 disables the rotation                                 */
  float pos_scale;       /* position feature of the controller is n / pos_scale                  */
  uint32_t flags;        /* ADORE_FLAG_* bits; unknown bits are rejected                         */
} adore_config_t;

/* Controller parameters (Section 2.2 Eq. 2 and Appendix B), float32, HOST pointers, copied at
 * create. Stacked GRU gate order: reset, update, candidate. */
typedef struct {
  const float *gru_w_ih; /* [3d', d]  */
  const float *gru_w_hh; /* [3d', d'] */
  const float *gru_b_ih; /* [3d']     */
  const float *gru_b_hh; /* [3d']     */
  const float *pos_w;    /* [d']   position layer FC(1 -> d') */
  const float *pos_b;    /* [d']   */
  const float *mlp_w1;   /* [d', d'] interaction layer (Tanh)  */
  const float *mlp_b1;   /* [d']   */
  const float *mlp_w2;   /* [d']   output layer FC(d' -> 1), sigmoid applied to its output */
  const float *mlp_b2;   /* [1]    */
} adore_controller_weights_t;

/* Creates an empty cache on the current CUDA device (Section 2.1: a cache of m selected rows per
 * layer; here C = m + R_max slots). cuda_stream is a cudaStream_t (NULL = default stream). The
 * library allocates the K/V slots [L][B][H][C][dh], the token table (hidden rows, scores, slot
 * index per token), controller state and scratch. Errors: INVALID_ARG, UNSUPPORTED, OOM, CUDA. */
adore_status_t adore_cache_create(const adore_config_t *cfg, const adore_controller_weights_t *ctrl,
                                  void *cuda_stream, adore_cache_t **out);

/* Waits for the stream, frees everything the cache owns. NULL is accepted. */
adore_status_t adore_cache_destroy(adore_cache_t *cache);

/* Registers the K/V projection of a layer (Section 2.3: rebuilt states are recomputed from token
 * embeddings). w_kv: device, T[2*H*dh, d] row-major, key rows first then value rows; borrowed
 * until destroy; must be 16-byte aligned. */
adore_status_t adore_cache_set_projection(adore_cache_t *cache, int32_t layer, const void *w_kv);

/* Bulk load of T prompt tokens into an EMPTY cache (Section 2.1: user input tokens t_1..t_s).
 * x: device T[B, T, d]. Runs the controller over the T tokens, retains the newest token plus the
 * min(m-1, T-1) highest-scoring earlier ones in ascending position from slot 0 (the set that
 * releasing one token at a time would reach), chooses the rebuild list as in a decode step
 * (POLICY mode only), and fills every layer whose projection is set from these rows.
 * Errors: STATE (cache not empty), TOKEN_TABLE_FULL, INVALID_ARG. */
adore_status_t adore_cache_append_tokens(adore_cache_t *cache, const void *x, int32_t T);

/* Recomputes the K/V rows of every resident token of `layer` from x_table[b, tok, :]
 * (device T[B, max_tokens, d]); NULL uses the cache's own stored rows. For stacks whose layers
 * have their own input rows (Section 2.3 recomputes states layer by layer). */
adore_status_t adore_cache_fill_layer(adore_cache_t *cache, int32_t layer, const void *x_table);

/* One decode step for one layer (Sections 2.1-2.3). Call layer 0 first in every step; it also
 * runs the controller for the new token, releases / admits / chooses the rebuild list, and
 * advances n. All pointers are DEVICE pointers; q, k_new, v_new, x_new and out must start on a
 * 16-byte boundary (INVALID_ARG otherwise; the same holds for the row pointers of
 * adore_step_begin / adore_attend_rows and for x_table of adore_rebuild / adore_cache_fill_layer).
 *   q, k_new, v_new : T[B, H, dh]; k_new already carries the rotary embedding of position n.
 *   x_new           : T[B, d], read at layer 0 only (stored in the token table), else ignored.
 *   explicit_list   : int32[B, r_in] candidate token positions, explicit_count int32[B] how many
 *                     are valid per sequence; both NULL in POLICY mode. Read at layer 0 only.
 *                     x_new and the lists are read by kernels on the library's own streams; the
 *                     caller's stream is made to wait for those reads before the call returns,
 *                     so work queued on it afterwards may overwrite them.
 *   out             : T[B, H, dh].
 *   weights         : float[B, H, C+1] or NULL. Entry s < C is slot s, entry C the current
 *                     token; masked or empty entries are 0.
 * The attention reads the cache as the previous step left it (retained + last step's rebuilt
 * rows), i.e. the m+R+1 rows of Section 2.3; the new token's row is then written in place.
 * Errors: INVALID_ARG, STATE, TOKEN_TABLE_FULL, CUDA. */
adore_status_t adore_decode_step(adore_cache_t *cache, int32_t layer, const void *q, const void *k_new,
                                 const void *v_new, const void *x_new, const int32_t *explicit_list,
                                 const int32_t *explicit_count, int32_t r_in, void *out, float *weights);

/* Same step (Sections 2.1-2.3) with HOST buffers: copies q, k_new, v_new, x_new and the explicit
 * list to the device, runs adore_decode_step, copies `out` back and waits for the stream. Pinned
 * host memory makes the copies asynchronous up to the final wait. `weights` stays a DEVICE pointer
 * (float[B, H, C+1]) or NULL: the per-slot weights are eight times the size of `out` and are meant
 * for consumers on the device, so they are emitted there and not copied. */
adore_status_t adore_decode_step_host(adore_cache_t *cache, int32_t layer, const void *q, const void *k_new,
                                      const void *v_new, const void *x_new, const int32_t *explicit_list,
                                      const int32_t *explicit_count, int32_t r_in, void *out, float *weights);

/* adore_decode_step_host followed by adore_rebuild(cache, layer, x_table) (Sections 2.1-2.3), with one difference in
 * what the host waits for: the rebuild is queued before the wait, and the call returns as soon as `out` has reached
 * the host, so the GPU runs from the attention straight into the rebuild while the caller consumes `out` and hands in
 * the next inputs. x_table as for adore_rebuild (DEVICE or NULL); everything else as for adore_decode_step_host.
 * Errors as for the two calls (STATE if the layer has no projection). */
adore_status_t adore_decode_rebuild_host(adore_cache_t *cache, int32_t layer, const void *q, const void *k_new,
                                         const void *v_new, const void *x_new, const int32_t *explicit_list,
                                         const int32_t *explicit_count, int32_t r_in, const void *x_table, void *out,
                                         float *weights);

/* The same step and rebuild (Sections 2.1-2.3) with HOST buffers, QUEUED: the call returns without waiting for
 * anything, so the calls of all layers of a step (and of the next steps) can be issued back to back and the host
 * waits once, with adore_cache_wait_outputs (or adore_cache_sync_status), before it reads the `out` buffers. Every layer has a staging set of its own
 * on the device; its upload waits (on the device) for the previous step's use of that set. All host buffers must be
 * pinned for the copies to be asynchronous and must stay valid and unchanged until that wait; `out` of different calls
 * in flight must be different buffers. Arguments and errors as for adore_decode_rebuild_host. The first call
 * allocates the staging sets. */
adore_status_t adore_decode_rebuild_host_queued(adore_cache_t *cache, int32_t layer, const void *q, const void *k_new,
                                                const void *v_new, const void *x_new, const int32_t *explicit_list,
                                                const int32_t *explicit_count, int32_t r_in, const void *x_table,
                                                void *out, float *weights);

/* Host-side wait for the `out` buffers of every adore_decode_rebuild_host_queued call issued so far (Section 2.1's
 * attention output of each layer), and for nothing else: the rebuilds queued by those calls may still be running,
 * and the next step's calls can be issued beside them. By then the host input buffers of those calls have been read
 * too. Does not report the device error word (adore_cache_sync_status does). Errors: INVALID_ARG, CUDA. */
adore_status_t adore_cache_wait_outputs(adore_cache_t *cache);

/* Rebuild for one layer (Section 2.3): Y = X_L [W_k ; W_v]^T for the rows of this step's rebuild
 * list, rotary embedding on the key half at each token's original position, rounding to T and
 * scatter into the list's slots. x_table: device T[B, max_tokens, d] rows indexed by token
 * position, or NULL for the cache's stored rows. Call after adore_decode_step of the same layer.
 * In a cache of several layers (attend-first order) the work is queued on a stream of the library's own, behind
 * everything the cache's stream holds at the time of the call, and runs beside the attention of the following
 * layers: nothing reads this layer's rows before the next step's adore_decode_step of this layer, which waits for
 * it, as does every other call that touches what the rebuild reads or writes. x_table is therefore borrowed until
 * the next adore_decode_step of layer 0, adore_cache_join or adore_cache_sync_status.
 * Errors: STATE (no projection / no step), INVALID_ARG, CUDA. */
adore_status_t adore_rebuild(adore_cache_t *cache, int32_t layer, const void *x_table);

/* Makes the stream given at create wait for everything the library has queued on its own streams (the controller of
 * the last token, rebuilds that run beside later layers), without waiting on the host: work queued on that stream
 * afterwards, an event recorded on it for timing included, comes after all of the step (Sections 2.2-2.3).
 * Errors: INVALID_ARG, CUDA. */
adore_status_t adore_cache_join(adore_cache_t *cache);

/* Read-only DEVICE views of the state of Sections 2.2-2.3 for checking; valid until the next
 * call that changes the cache. */
adore_status_t adore_cache_slot_map(adore_cache_t *cache, const int32_t **slot_tok /*[B,C]*/,
                                    const uint8_t **slot_role /*[B,C]*/);
adore_status_t adore_cache_rebuild_list(adore_cache_t *cache, const int32_t **tok /*[B,R_max]*/,
                                        const int32_t **slot /*[B,R_max]*/, const int32_t **count /*[B]*/);
adore_status_t adore_cache_step_info(adore_cache_t *cache, const int32_t **admit_slot /*[B]*/,
                                     const int32_t **evicted_tok /*[B]*/);
adore_status_t adore_cache_scores(adore_cache_t *cache, const float **score /*[B,max_tokens]*/,
                                  const float **sigma /*[B,max_tokens]*/);
adore_status_t adore_cache_kv(adore_cache_t *cache, int32_t layer, const void **k, const void **v);

/* Number of tokens n per sequence (host value). */
int32_t adore_cache_num_tokens(const adore_cache_t *cache);

/* Kernel launches issued by this cache so far (host counter). */
int64_t adore_cache_launch_count(const adore_cache_t *cache);

/* Per-stage device timing for benchmarks (no counterpart in the paper beyond its Appendix D
 * runtime split between the controller and the rest). When enabled, every kernel launch of the
 * cache is bracketed by CUDA events on its stream. adore_cache_stage_times waits for the stream,
 * adds up the elapsed milliseconds and launch counts per stage since the last call and resets
 * them. Stage index: 0 attention (with the fused admit of layers > 0), 1 controller + selection,
 * 2 rebuild projection (gather + GEMM), 3 the separate admit launch of layer 0.
 * enable: 0 off, 1 per-stage timing, 2 group timing (see adore_cache_group_times).
 * ms and launches: HOST arrays of 4. While per-stage timing is enabled the controller runs on the main
 * stream instead of beside the attention, so that the stage times add up. Event recording costs a few microseconds per launch, so
 * whole-step throughput should be measured with timing disabled. */
adore_status_t adore_cache_set_stage_timing(adore_cache_t *cache, int32_t enable);
adore_status_t adore_cache_stage_times(adore_cache_t *cache, double *ms, int64_t *launches);

/* Device time of the attention + selection group as the step really runs it (no counterpart in the paper; Section 1
 * and Section 3.2 name the attention's KV traffic as the cost that matters). With adore_cache_set_stage_timing(cache, 2)
 * the schedule stays as it is: selection and controller on their side streams beside the attention, rebuilds beside
 * the following layers. Per attend-first step three events are recorded: where the group starts (before the attention
 * of layer 0), where its main-stream part ends (after the last layer's attention; in a one-layer cache after the new
 * token's row has been written) and where the controller chain ends. adore_cache_group_times waits for the streams and
 * returns, summed over the steps since the last call, in *ms the time from the first event to the later of the other
 * two, in *ms_main the time from the first event to the second alone (what the rest of the step waits for: the
 * controller of token n starts when the attention of layer 0 is done and its score is first read by the next step's
 * selection), and the number of steps; all are reset. ms, ms_main, steps: HOST pointers. In a cache of several layers
 * the rebuilds of layers 0..L-2 run inside that window, on their own stream. */
adore_status_t adore_cache_group_times(adore_cache_t *cache, double *ms, double *ms_main, int64_t *steps);

/* Total number of rows rebuilt by decode steps so far (Section 2.3: sum over steps and sequences
 * of the rebuild-list lengths); waits for the stream. rows: HOST pointer. */
adore_status_t adore_cache_rebuild_rows(adore_cache_t *cache, int64_t *rows);

/* Controller scoring for callers that cannot allocate device memory. (The paper has no
 * counterpart: this is a packaging of its controller, Section 2.2 Eq. 2, for a constrained
 * caller.) Some users of this library run where cudaMalloc is off limits: a scheduler thread
 * that scores tokens while another thread is capturing or replaying CUDA graphs, a service whose
 * device memory was carved up once at start-up and is owned by a different allocator, or code
 * that must not take the driver's allocation lock on its latency path. The cache-based path
 * gets its scratch (the k-split partial sums of the gate product W_ih x) from cudaMalloc in
 * adore_cache_create; this entry point keeps the same scratch in a fixed 2 MiB array inside
 * the library image instead, and needs no cache object at all.
 *
 * It scores ONE new token per sequence: z <- GRU(x, z), score = MLP(p + z), sigma = sigmoid.
 *   w         : HOST struct of DEVICE pointers to the float32 parameters, same shapes and gate
 *               order as adore_controller_weights_t describes (row-major, not transposed).
 *   x         : device T[batch, hidden] rows of the new tokens (T by `dtype`).
 *   z         : device double[batch, ctrl_hidden], the GRU state; read and overwritten (start a
 *               sequence with zeros).
 *   position  : position n of the new token; the position feature is n / pos_scale.
 *   score, sigma : device float[batch] outputs (pre-sigmoid score and sigma).
 * The arithmetic is the cache-based path's (float64, rounded to float32 at the end); only the
 * number of k-slices may differ, so results agree to the last float32 digit or one unit of it.
 *
 * Limits and rules:
 *   - batch * 3 * ctrl_hidden doubles must fit the 2 MiB array (batch <= 682 for d' = 128);
 *     larger requests return ADORE_ERR_UNSUPPORTED and launch nothing.
 *   - hidden must be a multiple of 64 (as for adore_cache_create), x and w->gru_w_ih must be
 *     16-byte aligned and z 8-byte aligned; otherwise ADORE_ERR_UNSUPPORTED, nothing is launched.
 *   - The array is part of the library image: every GPU on which the library runs holds
 *     these 2 MiB until the process exits.
 *   - The first call on each device looks up the array's device address (no allocation). Make
 *     that first call outside any stream capture.
 *   - All calls on a device share the array. It is fully rewritten by each call, so nothing
 *     needs clearing, but two calls whose kernels overlap on the GPU (different streams) race;
 *     keep calls on one stream or order them with events.
 *   - No cudaMalloc, cudaFree or other allocating routine is called; work is queued on
 *     cuda_stream (a cudaStream_t, NULL = default stream) and not waited for. */
adore_status_t adore_controller_score_static(const adore_controller_weights_t *w, adore_dtype_t dtype,
                                             int32_t batch, int32_t hidden, int32_t ctrl_hidden, const void *x,
                                             double *z, int32_t position, float pos_scale, float *score,
                                             float *sigma, void *cuda_stream);

/* The step in the order Section 2.3 prints it: select first, then rebuild, then one attention in which the rebuilt
 * tokens' query rows and the current token's share the key and value rows.
 *
 * adore_step_begin: controller + selection for the new token n (Section 2.2 Eq. 2 and release rule, Section 2.3
 *   first sentence); x_new [B, d] DEVICE and the explicit list as for adore_decode_step at layer 0. Afterwards the
 *   slot map holds the retained tokens, the slots of this step's rebuild list and the slot token n will get.
 * Then per layer: adore_rebuild(cache, layer, x_table) writes the listed tokens' K/V rows, and
 * adore_attend_rows runs Section 2.3's attention: q_rows [B, H, R_max+1, dh] DEVICE, row i < R_max for the i-th
 *   token of adore_cache_rebuild_list() (rows past a sequence's count are ignored and produce zeros), the last row
 *   for token n; k_new, v_new [B, H, dh] DEVICE are token n's own rows. Row i attends over the occupied slots
 *   whose token position is at most its own (the cached and the rebuilt rows), the last row over token n's own
 *   row too; each row keeps its topk largest logits. out [B, H, R_max+1, dh] DEVICE; weights
 *   [B, H, R_max+1, C+1] float DEVICE or NULL. The call then stores k_new, v_new in token n's slot.
 *   Needs head_dim 64 or 128 (ADORE_ERR_UNSUPPORTED otherwise).
 * A step opened by adore_step_begin must be finished with these calls; adore_decode_step at layer 0 opens a
 * step of the other kind. Mixing the two within a step returns ADORE_ERR_STATE. */
adore_status_t adore_step_begin(adore_cache_t *cache, const void *x_new, const int32_t *explicit_list,
                                const int32_t *explicit_count, int32_t r_in);
adore_status_t adore_attend_rows(adore_cache_t *cache, int32_t layer, const void *q_rows, const void *k_new,
                                 const void *v_new, void *out, float *weights);

/* Labels for training the controller and the uniform-token-set statistics (Section 2.2 last paragraph, Appendix B
 * "training data collection", Appendix C / Figure 7) from the per-slot weights one decode step emitted for all layers.
 * Needs no cache; runs on the given CUDA stream (NULL = default stream) and allocates nothing.
 *   weights  [n_layers, batch, n_heads, n_slots] float DEVICE (n_slots = C + 1 for weights of adore_decode_step;
 *            zero = masked or empty), n_slots <= 4096 (else ADORE_ERR_UNSUPPORTED)
 *   sets     [n_layers, batch, n_heads, topk/2] int32 DEVICE out: per layer and head the topk/2 slots with the
 *            largest positive weight, descending, equal weights lower slot first, -1 padded
 *   count    [batch, n_slots] int32 DEVICE out: how many of those sets contain the slot
 *   label    [batch, n_slots] uint8 DEVICE out: 1 for the topk slots with the largest positive count (equal counts:
 *            lower slot first), else 0
 *   coverage [n_layers, batch] float DEVICE out: share of the layer's set members that carry the label
 *   mass     [n_layers, batch] float DEVICE out: weight of the labelled slots at that layer, averaged over heads */
adore_status_t adore_label_tokens(const float *weights, int32_t n_layers, int32_t batch, int32_t n_heads, int32_t n_slots,
                                  int32_t topk, void *cuda_stream, int32_t *sets, int32_t *count, uint8_t *label,
                                  float *coverage, float *mass);

/* Snapshot of the small per-sequence state that scoring and selection carry from step to step
 * (Section 2.2: which tokens hold which slots, every token's controller score and the GRU state z;
 * Section 2.3: the step's rebuild list): both slot-map buffers, the token-to-slot table, score and sigma
 * of all tokens, z, the step's admit/evict/rebuild lists and row table, and n. NOT included: the K/V
 * cache rows and the stored layer-input rows (they are large; a caller that wants to rewind a cache keeps
 * or recomputes them itself).
 *   export: host_buf == NULL stores the size needed in *bytes. Otherwise *bytes is the capacity of
 *           host_buf (HOST memory, written by the call) and receives the size written; too small a
 *           buffer returns ADORE_ERR_INVALID_ARG with the size needed in *bytes.
 *   import: host_buf is a snapshot taken from a cache created with the same batch, capacity,
 *           rebuild_max, max_tokens and ctrl_hidden; anything else returns ADORE_ERR_INVALID_ARG and
 *           changes nothing.
 * Both wait for the cache's streams before copying (synchronous calls).
 *
 * Layout of a snapshot (version 1, little endian, every section padded to a multiple of 8 bytes):
 *   header, 64 bytes: uint32 magic 0x54534441, uint32 version = 1, then int32 batch, capacity, rebuild_max, max_tokens,
 *     ctrl_hidden, n, cur (which of the two slot-map buffers is the current one), attn (the one the cache rows follow),
 *     step_open (0 none, 1 attend-first, 2 rebuild-first), uint32 flag word (ADORE_FLAG_RELATIVE_POSITION bit), 16 bytes zero;
 *   sections, with B = batch, C = capacity, T = max_tokens, R = max(rebuild_max, 1):
 *     int32 slot_tok[2][B][C] (as two sections), uint8 slot_role[2][B][C] (two sections), int32 tok_slot[B][T],
 *     float score[B][T], float sigma[B][T], double z[B][ctrl_hidden], int32 admit_slot[B], int32 evicted_tok[B],
 *     int32 rebuild_tok[B][R], int32 rebuild_slot[B][R], int32 rebuild_count[B], int32 row_b[B*R], int32 row_tok[B*R],
 *     int32 row_slot[B*R], int32 row_total[1]; with ADORE_FLAG_RELATIVE_POSITION also double a[B][T][ctrl_hidden].
 * import checks every index of the integer sections against the cache's shape before anything is copied to the
 * device (token positions < n, slots < C, roles, counts within m and R_max, row table entries within the batch);
 * a snapshot that fails returns ADORE_ERR_INVALID_ARG and changes nothing. */
adore_status_t adore_cache_export_state(adore_cache_t *cache, void *host_buf, size_t *bytes);
adore_status_t adore_cache_import_state(adore_cache_t *cache, const void *host_buf, size_t bytes);

/* Waits for the stream and turns the device error word into a status (OK, DEVICE_FLAG, TIMEOUT,
 * or CUDA if the stream itself failed). The word is cleared. */
adore_status_t adore_cache_sync_status(adore_cache_t *cache);

const char *adore_status_string(adore_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* ADORE_H_ */
