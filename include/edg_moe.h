/*
 * edg_moe.h -- C ABI of the streaming-MoE per-layer decode step for NVIDIA B200 (sm_100a).
 *
 * The library implements one thing: the routed-expert block of a streaming mixture-of-experts
 * decoder as the paper states it (Sec. 3 "System Design" and Appendix A "Routing Math"):
 *
 *   a1  prerouter logits       l = W_pre . s                       (Sec. 3.2 "Head", linear path)
 *   a2  softmax top-k          g = softmax(l), inds = top-k(g, K),
 *                              w = g[inds] / sum g[inds]            (Appendix A, softmax-topk)
 *   a3  slot map + staging     slots = take(slot_table, inds); only missing experts are copied
 *                              into a fixed pool of sticky slots     (Sec. 3.1, "staged" path)
 *   a4  gate/up                h = silu(gate(x)) * up(x)            (Sec. 3.1 "Math contract")
 *   a5  down                   o = down(h)
 *       every projection is  W_int4(x) + (alpha/r) B A x,  W dequantised on the fly and the
 *       LoRA delta added as a parallel branch, never merged          (Sec. 3.3, Fig. 1 caption)
 *   a6  reduce                 y = sum_k w_k o_k                    (Appendix A weights)
 *
 * Conventions
 *   - Plain C: pointers and sizes only.  "dev" = device (HBM) pointer, "host" = host pointer,
 *     "pinned" = page-locked host memory.  Streams are cudaStream_t passed as void*.
 *   - Every call returns an int32 status: EDG_OK or a negative EDG_E_* code.  Nothing throws.
 *   - The caller owns every buffer and every stream.  The library owns only the opaque store
 *     handle (allocator state, CUDA events, a small pinned ring for slot-table updates).
 *   - Device work is asynchronous on the stream given.  The hot calls (prerouter_topk,
 *     moe_expert_ffn_int4_lora, moe_layer_decode) neither allocate nor synchronise with the host.
 *   - Device pointers must be 16-byte aligned; slot records must be 256-byte aligned (the record
 *     size is always a multiple of 256).
 *   - bf16 and fp16 values are passed as their 16-bit patterns.
 *
 * Quantised weight format (Sec. 3.1: int4, group-wise affine, one scale and one second parameter
 * per group of `group` consecutive input elements):  w[n][k] = scale[n][k/group] * (q[n][k] -
 * zero[n][k/group]),  q in 0..15, scale and zero stored as fp16.  Zero points are values in
 * [0, 16] that are multiples of 1/128 (integers 0..15 in the usual asymmetric scheme): for those
 * every kernel forms q - zero without rounding, whichever precision it subtracts in;
 * edg_pack_expert rejects any other zero point with EDG_E_RANGE.  Canonical interchange layout:
 * row-major [out][in]; byte j of a row holds q[2j] in its low nibble and q[2j+1] in its high nibble.
 * One expert = gate [I][H], up [I][H], down [H][I].  edg_pack_expert turns canonical tensors into
 * the record the kernels read; its size is edg_record_bytes (1,769,472 B at H=2048, I=512,
 * group 64 -- the paper's 1.77 MB per expert).
 */
#ifndef EDG_MOE_H
#define EDG_MOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define EDG_OK          0
#define EDG_E_INVAL    -1   /* null pointer, misaligned pointer, bad enum, bad handle            */
#define EDG_E_SHAPE    -2   /* a dimension the kernels do not support (see edg_check_desc)     */
#define EDG_E_SLOTS    -3   /* more experts to stage than slots in the pool                     */
#define EDG_E_RANGE    -4   /* expert / layer / slot index out of range, or duplicate expert    */
#define EDG_E_CUDA     -5   /* a CUDA runtime call failed; see edg_last_cuda_error              */
#define EDG_E_TIMEOUT  -6   /* a bounded wait (host or device side) ran out                     */
#define EDG_E_WORKSPACE -7  /* workspace too small or misaligned                                */

/* dtypes */
#define EDG_F32   0
#define EDG_F16   1
#define EDG_BF16  2

/* Shape of one MoE layer: the paper's model spec (expert count, K, quantisation, ...), Sec. 3. */
typedef struct edg_layer_desc {
    int32_t H;           /* hidden size                                                          */
    int32_t I;           /* expert intermediate size                                             */
    int32_t E;           /* experts per layer                                                    */
    int32_t K;           /* experts routed per token (top-k)                                     */
    int32_t group;       /* quantisation group size along the input dimension                    */
    int32_t rank;        /* LoRA rank r (0 = no adapter)                                         */
    int32_t n_adapters;  /* 1: one adapter shared by all experts of the layer; E: one per expert */
    int32_t n_slots;     /* slots per layer in the HBM pool                                      */
    int32_t pre_dtype;   /* storage type of the prerouter head: EDG_F32 or EDG_F16               */
    int32_t out_dtype;   /* type of y: EDG_F32, EDG_F16 or EDG_BF16                              */
    float   lora_scale;  /* alpha / r                                                            */
} edg_layer_desc;

/* Unmerged LoRA factors of one layer, bf16, all dev.  Leading dimension n_adapters.
 * A maps the projection's input to rank r, B maps rank r to its output (Sec. 3.3). */
typedef struct edg_lora {
    const void* A_gate;  /* [n_adapters][rank][H] */
    const void* B_gate;  /* [n_adapters][I][rank] */
    const void* A_up;    /* [n_adapters][rank][H] */
    const void* B_up;    /* [n_adapters][I][rank] */
    const void* A_down;  /* [n_adapters][rank][I] */
    const void* B_down;  /* [n_adapters][H][rank] */
} edg_lora;

typedef struct edg_store edg_store;   /* opaque slot-pool expert store */

typedef struct edg_store_stats {
    int64_t stage_calls;    /* calls of stage_experts_to_slots                     */
    int64_t hits;           /* staged experts already resident (nothing copied)    */
    int64_t misses;         /* staged experts copied host -> HBM                   */
    int64_t bytes_copied;   /* misses * record bytes                               */
    int64_t table_updates;  /* device slot-table rows rewritten                    */
} edg_store_stats;

/* ---------------------------------------------------------------- utilities (host, synchronous) */

/* Version of this ABI (major * 1000 + minor). */
int32_t edg_version(void);

/* Last cudaError_t seen by this library on the calling thread (0 = none), and its text. */
int32_t edg_last_cuda_error(void);
const char* edg_last_cuda_error_string(void);

/* Checks a descriptor against what the kernels support: H and I multiples of 128 and at most
 * 4096 with H/32 and I/32 a power of two; group a multiple of 32 dividing H and I; 1 <= K <= 32;
 * K <= E <= 1024; 0 <= rank <= 64; n_adapters 1 or E; n_slots >= 1.  Returns EDG_OK or EDG_E_SHAPE. */
int32_t edg_check_desc(const edg_layer_desc* desc);

/* Bytes of one expert record: 3*H*I/2 code bytes + 3*(H*I/group) (scale, zero) fp16 pairs. */
int32_t edg_record_bytes(const edg_layer_desc* desc, size_t* bytes);

/* One-time host repack of canonical tensors (layout above; scales/zeros as fp16 bit patterns,
 * [out][in/group]) into the record the kernels read.  `record` is host memory of
 * edg_record_bytes bytes.  Never on the hot path.  edg_unpack_expert is its exact inverse.
 * Returns EDG_E_RANGE (and writes nothing) when a zero point is outside [0, 16] or is not a
 * multiple of 1/128. */
int32_t edg_pack_expert(const edg_layer_desc* desc,
                        const uint8_t* codes_gate, const uint16_t* scales_gate, const uint16_t* zeros_gate,
                        const uint8_t* codes_up,   const uint16_t* scales_up,   const uint16_t* zeros_up,
                        const uint8_t* codes_down, const uint16_t* scales_down, const uint16_t* zeros_down,
                        void* record);
int32_t edg_unpack_expert(const edg_layer_desc* desc, const void* record,
                          uint8_t* codes_gate, uint16_t* scales_gate, uint16_t* zeros_gate,
                          uint8_t* codes_up,   uint16_t* scales_up,   uint16_t* zeros_up,
                          uint8_t* codes_down, uint16_t* scales_down, uint16_t* zeros_down);

/* Bytes of device scratch the FFN calls need for T tokens (T = 1 for batch-1 decode). */
int32_t edg_ffn_workspace_bytes(const edg_layer_desc* desc, int32_t T, size_t* bytes);

/* Reads the device-side status word that the kernels keep at the start of a workspace: 0, an
 * EDG_E_RANGE raised by a slot or expert index outside its range (the kernel skips that access
 * instead of faulting), or an EDG_E_TIMEOUT raised by a bounded device-side wait that gave up (the
 * kernel then falls back to waiting for the previous kernel, or goes on with a flagged result).
 * Synchronises `stream`. */
int32_t edg_workspace_status(const void* workspace, void* stream, int32_t* status);

/* Tracing: with a dev buffer of (CTAs in the grid) x 32 uint64 (the batch-1 layer kernel launches
 * at most 16 (K + 1) + E / 16 + 3 CTAs), every CTA stamps the GPU's nanosecond timer
 * at its phase boundaries, in slot 0 start, 1 first copies issued, 2 adapter projections sent,
 * 3 first weights landed, 4 gate/up of the first quarter done, 5 peers' projections in, 6 h sent,
 * 7 h of the quarter in, 8 partial output written, 9 end, 10 slot taken, 12 head row summed,
 * 13 head row published, 14 routing known, 19 routing read from the hand-off ring,
 * 24 first quarter finished; 15-18 are stamped by the warp that computes the
 * caller's top-k.  NULL switches it off (the default).  Process-wide; set it while no launch is
 * in flight. */
int32_t edg_set_trace_buffer(void* dev_buffer);

/* ---------------------------------------------------------------- a1 + a2: prerouter */

/* Prerouter head + routing (Sec. 3.2; Appendix A softmax-topk), for n_heads independent
 * (head, hidden state) pairs in one launch -- the "single flush per step" that predicts every
 * staged layer at once.
 *   W_pre   dev [n_heads][E][H], pre_dtype           s       dev bf16 [n_heads][H]
 *   inds    dev int32 [n_heads][K], ascending expert index, distinct
 *   gates   dev float [n_heads][K], aligned with inds, sum to 1
 *   logits_opt  dev float [n_heads][E] or NULL: the fp32 logits the selection was made on
 *   inds_host_mirror_opt  int32 [n_heads][K] in mapped pinned host memory (cudaHostAlloc; with
 *               unified addressing the host pointer is what the kernel is given), or NULL: the
 *               kernel stores the indices there too, so that the stager on the host can read the
 *               prediction without a device-to-host copy and without synchronising the stream.
 *               Protocol: the caller fills the mirror with -1 before the call; every entry is final
 *               by itself once it is >= 0; a head's prediction is complete when its K entries are.
 * Equal logits go to the lower expert index. */
int32_t prerouter_topk(const edg_layer_desc* desc, const void* W_pre, const void* s, int32_t n_heads,
                       int32_t* inds, float* gates, float* logits_opt, int32_t* inds_host_mirror_opt,
                       void* stream);

/* The same for T hidden states that all use ONE head (batched decode of one layer):
 * W_pre dev [E][H]; s dev bf16 [T][H]; outputs [T][K] / [T][E]. */
int32_t prerouter_topk_tokens(const edg_layer_desc* desc, const void* W_pre, const void* s, int32_t T,
                              int32_t* inds, float* gates, float* logits_opt, void* stream);

/* a2 alone on given logits (a router's own gate at prefill): logits dev float [T][E] ->
 * inds dev int32 [T][K], gates dev float [T][K].  Same ordering and tie rule. */
int32_t softmax_topk_rows(const edg_layer_desc* desc, const float* logits, int32_t T,
                          int32_t* inds, float* gates, void* stream);

/* The full prerouter head of a layer (Sec. 3.2 "Head"): fc1 -> erf-gelu -> fc2 plus a linear residual
 * path.  The input feature is the hidden state followed by two K-hot vectors over the E experts --
 * the experts this layer routed to at this token and at the previous token -- so its dimension is
 * H + 2E (2560 at the 35B tier) and the hidden width D is 512 there.  With f = [s ; hot(cur) ; hot(prev)]:
 *     z = W1 f + b1,    l = W2 gelu(z) + b2 + W_res s,    gelu(z) = z/2 (1 + erf(z / sqrt 2)),
 * followed by the same softmax top-k with renormalised gates as prerouter_topk.  The residual path acts
 * on the hidden state alone (it is what the paper warm-starts from the next layer's router weight).
 * All tensors are device memory owned by the caller; biases and the residual path may be NULL. */
typedef struct edg_mlp_head {
    const void* W1;     /* fp16 [n_heads][D][H + 2E]                                   */
    const void* b1;     /* fp16 [n_heads][D] or NULL                                   */
    const void* W2;     /* fp16 [n_heads][E][D]                                        */
    const void* b2;     /* fp16 [n_heads][E] or NULL                                   */
    const void* W_res;  /* [n_heads][E][H] of desc->pre_dtype, or NULL                 */
    int32_t width;      /* D: a multiple of 8, 8 <= D <= 4096                          */
} edg_mlp_head;

/* s dev bf16 [n_heads][H]; cur_inds / prev_inds dev int32 [n_heads][K] (entries outside 0..E-1 are
 * ignored); inds dev int32 [n_heads][K] ascending; gates dev float [n_heads][K]; logits_opt dev float
 * [n_heads][E] or NULL.  One cluster of 8 CTAs per head; fp32 accumulation; (E + H + D) * 4 bytes of
 * shared memory must fit 48 KB, else EDG_E_SHAPE.  Pointers 16-byte aligned, else EDG_E_INVAL. */
int32_t prerouter_mlp_topk(const edg_layer_desc* desc, const edg_mlp_head* head, const void* s,
                           const int32_t* cur_inds, const int32_t* prev_inds, int32_t n_heads,
                           int32_t* inds, float* gates, float* logits_opt, void* stream);

/* The other routing family of the paper (Appendix A, "Sigmoid-group"; its 8B tier runs n = 8 groups,
 * keep G = 4, K = 8, scale 2.5, E = 128) on given logits: sigma = sigmoid(l); a group's score is the
 * sum of its two largest selection scores, where the selection score is sigma, plus bias_opt[e] when a
 * bias is given (the "biased score" of the paper's remark); the keep_groups best groups survive,
 * ties to the lower group; the K best survivors by selection score are taken, ties to the lower
 * index; gates = scale * sigma[inds] / (sum of sigma[inds] + 1e-20) -- the raw sigmoid, not the biased
 * score.  logits dev float [T][E]; bias_opt dev float [E] or NULL; inds dev int32 [T][K] in
 * ascending index; gates dev float [T][K] aligned with inds.  E <= 1024, n_groups <= 32 dividing E
 * with at least two experts a group, K <= 32 and <= keep_groups * E / n_groups; else EDG_E_SHAPE.
 * One warp per row; no workspace; arithmetic in fp32 (the decision is taken in the kernel's
 * precision). */
int32_t sigmoid_group_topk_rows(const float* logits, int32_t T, int32_t E, int32_t K, int32_t n_groups,
                                int32_t keep_groups, float scale, const float* bias_opt,
                                int32_t* inds, float* gates, void* stream);

/* ---------------------------------------------------------------- a3: slot-pool expert store */

/* Creates the store of n_layers layers (Sec. 3.1 "staged" path; Fig. 1: bounded streaming pool
 * with fixed staged slots).
 *   host_layers  host array of n_layers pointers, each to pinned [E][record bytes] (the tier that
 *                stands in for the paper's SSD); layers may alias
 *   dev_slots    dev [n_layers][n_slots][record bytes]
 *   dev_tables   dev int32 [n_layers][E]: slot of each expert, -1 if not resident; the store
 *                initialises it and keeps it current
 *   loras        host array of n_layers edg_lora (copied), or NULL for no adapter
 *   copy_stream  side stream the staging copies run on
 * Allocates events and a small pinned ring; not a hot call. */
int32_t edg_store_create(const edg_layer_desc* desc, int32_t n_layers, const void* const* host_layers,
                         void* dev_slots, int32_t* dev_tables, const edg_lora* loras,
                         void* copy_stream, edg_store** out);
int32_t edg_store_destroy(edg_store* store);

/* What the store asks of the machine when it stages: copies, events, stream ordering, a little
 * pinned memory.  The default engine is the CUDA runtime.  A caller may pass its own -- the
 * host-side tests do, with an engine that runs on plain host memory, completes operations late and
 * out of order across streams (honouring only the orderings the store has asked for) and so shows
 * whether the store asks for every ordering it needs.  All functions return 0 on success; `ctx` is
 * passed back as given.  With a foreign engine only the host-side calls are usable
 * (stage_experts_to_slots, edg_store_wait_staged, edg_store_mark_computed, snapshots, stats):
 * moe_layer_decode and edg_stack_decode_token launch kernels and return EDG_E_INVAL. */
typedef struct edg_copy_engine {
    void* ctx;
    int32_t (*copy_h2d)(void* ctx, void* dst, const void* src, size_t bytes, void* stream);   /* asynchronous on stream */
    int32_t (*fill)(void* ctx, void* dst, int32_t byte, size_t bytes, void* stream);          /* asynchronous memset    */
    int32_t (*event_create)(void* ctx, void** event_out);
    int32_t (*event_destroy)(void* ctx, void* event);
    int32_t (*event_record)(void* ctx, void* event, void* stream);
    int32_t (*stream_wait_event)(void* ctx, void* stream, void* event);
    int32_t (*event_synchronize)(void* ctx, void* event);       /* host waits */
    int32_t (*stream_synchronize)(void* ctx, void* stream);     /* host waits */
    int32_t (*host_alloc)(void* ctx, void** ptr_out, size_t bytes);   /* page-locked where that means something */
    int32_t (*host_free)(void* ctx, void* ptr);
} edg_copy_engine;

/* edg_store_create with a caller-supplied engine (NULL = the CUDA runtime, i.e. edg_store_create). */
int32_t edg_store_create_ex(const edg_layer_desc* desc, int32_t n_layers, const void* const* host_layers,
                            void* dev_slots, int32_t* dev_tables, const edg_lora* loras,
                            void* copy_stream, const edg_copy_engine* engine_opt, edg_store** out);

/* The "hot" executor path (Sec. 3.1: a fixed set of LRU-resident hot experts per layer; hits run
 * from their slots, misses fall to the on-demand path).  Switch it on before the first staging call.
 * Each layer's pool of n_slots slots is then split: the first n_slots - K slots hold the hot set,
 * the last K are transient slots, one per routed expert of the step in flight.
 *   - stage_experts_to_slots(layer, P) becomes the hot set's bookkeeping for one step: resident
 *     experts are hits (returned slot >= 0); the others are misses (returned slot -1) that the step
 *     serves on demand.  A miss whose expert has by now been routed `admit_after` times (1 = plain
 *     LRU, more = a popularity cache) also enters the hot set for LATER steps, in place of the
 *     least recently used slot this step neither hits nor has given away; its copy (copy engine,
 *     side stream) is queued by the layer's next edg_store_mark_computed, i.e. behind this step's
 *     compute, so the step never waits for it.
 *   - moe_layer_decode serves the misses itself, on the compute stream: a fetch kernel maps the
 *     routed experts through the device slot table and, for each one that is not resident, the SMs
 *     read its record straight from the pinned-host tier (plain 16-byte loads of mapped host
 *     memory) into a transient slot -- device-initiated, no host round trip, the indices never
 *     leave the GPU; the layer kernel then runs over hot and transient slots alike.  host_layers
 *     must be device-accessible (cudaHostAlloc memory is, under unified addressing).
 * Chaining does not apply to hot-path steps.  n_slots must exceed K; admit_after >= 1. */
int32_t edg_store_set_hot(edg_store* store, int32_t enable, int32_t admit_after);

/* The full prerouter head inside the layer-step (Sec. 3.2 "Head" and "Feature drift": a head's input
 * includes the routing its layer actually executed -- at decode, the head's own earlier prediction).
 * With a head set for a layer, moe_layer_decode of that layer predicts inds_next / gates_next with
 *     l = W2 gelu(W1 [x ; hot(cur) ; hot(prev)] + b1) + b2 + W_res x
 * where cur is the routing this call executes (inds_cur) and prev the routing the layer executed at
 * its previous call, which the store keeps on the device and updates after every call (empty before
 * the first call and after edg_store_reset_feedback: a new sequence).  W_pre_next is then ignored;
 * the prediction is made whenever inds_next is non-NULL.  The struct is copied; its tensors stay
 * the caller's (one head: leading dimension 1).  NULL removes the head (back to the linear path).
 * Steps of such a layer are never chained.  Allocates a small device buffer on first use: not hot. */
int32_t edg_store_set_mlp_head(edg_store* store, int32_t layer, const edg_mlp_head* head);
int32_t edg_store_reset_feedback(edg_store* store, int32_t layer);

/* The whole-layer executor path (Sec. 3.1: "all experts of a layer loaded in one shot for prefill
 * ... CPU load overlaps the previous layer's GPU execution").  Needs a pool as large as the layer
 * (n_slots == E, else EDG_E_SLOTS).  Queues on the copy stream, behind the last compute recorded for
 * this pool layer (edg_store_mark_computed), ONE copy of all E records -- from host_layer_opt
 * (pinned [E][record bytes]) if given, else from the layer's own host tier -- then the identity
 * slot table and the layer's copy-done event; edg_store_wait_staged makes the compute stream wait
 * for it.  With host_layer_opt a store of two pool layers serves a model of any depth as a double
 * buffer: load layer l+1 into pool (l+1) % 2 while layer l computes in pool l % 2. */
int32_t edg_store_load_whole_layer(edg_store* store, int32_t layer, const void* host_layer_opt);

/* The layer's shared expert (Sec. 3.1 "Problem" lists it beside the routed experts; Sec. 4 "Phase 2"
 * attaches the recovery adapter to its projections): one more SwiGLU expert of the same shape and
 * record format that every token runs, whatever the routing.  With a shared expert set,
 * moe_layer_decode computes
 *     y = sum_k w_k expert_k(x) + shared(x),
 * the shared expert in the same kernel launch as the routed ones (K + 1 experts, the last with
 * weight 1 and an adapter of its own), each projection again int4 base + lora_scale * B (A .).
 *   dev_record  dev, one record as written by edg_pack_expert, 256-byte aligned, resident for the
 *               lifetime of the store (never staged or evicted); NULL removes the shared expert
 *   lora_opt    its adapter: A/B tensors with leading dimension 1 and the descriptor's rank, or NULL.
 *               Routed experts may run without an adapter (store created with loras == NULL) while
 *               the shared expert has one -- the placement the paper trains.
 * Only for shapes the batch-1 layer kernel covers (else EDG_E_SHAPE); not used by the T > 1 calls. */
int32_t edg_store_set_shared_expert(edg_store* store, int32_t layer, const void* dev_record, const edg_lora* lora_opt);

typedef struct edg_hot_stats {
    int64_t hits;         /* routed experts found in the hot set                      */
    int64_t misses;       /* routed experts served on demand                          */
    int64_t admitted;     /* misses that entered the hot set for later steps          */
    int64_t bytes_direct; /* record bytes the SMs fetched from the host tier          */
} edg_hot_stats;
int32_t edg_store_get_hot_stats(const edg_store* store, edg_hot_stats* out);
int32_t edg_store_get_stats(const edg_store* store, edg_store_stats* out);

/* Host side of a3.  `inds_host` holds n distinct experts (n <= n_slots; n = K for one token, up to
 * the union of a batch).  Experts already resident keep their slot and copy nothing (sticky slots);
 * each missing expert, in the order given, replaces the least recently used slot that this call
 * does not need.  For every miss one cudaMemcpyAsync host->HBM is enqueued on the copy stream,
 * after the layer's last compute (ordered by an event), followed by the slot-table row update and
 * the layer's copy-done event.  Hits enqueue nothing.  Returns the slots (aligned with inds_host)
 * and the number of misses.  The prediction is consumed as the routing, so the staged set equals
 * the routed set by construction (Sec. 3.2 "Prediction-as-routing"). */
int32_t stage_experts_to_slots(edg_store* store, int32_t layer, const int32_t* inds_host, int32_t n,
                               int32_t* slots_host_out, int32_t* n_miss_out);

/* Host copy of a layer's tables, for inspection: expert_of_slot [n_slots], slot_of_expert [E]
 * (either may be NULL). */
int32_t edg_store_snapshot(const edg_store* store, int32_t layer, int32_t* expert_of_slot, int32_t* slot_of_expert);

/* Ordering hooks for callers that run the FFN themselves instead of through moe_layer_decode
 * (batched decode, prefill): edg_store_wait_staged makes `stream` wait for the layer's pending
 * staging copies (no-op when none are pending); edg_store_mark_computed tells the store that
 * everything enqueued on `stream` so far must finish before the layer's slots may be overwritten
 * (no-op for a pool that never evicts, n_slots == E). */
int32_t edg_store_wait_staged(edg_store* store, int32_t layer, void* stream);
int32_t edg_store_mark_computed(edg_store* store, int32_t layer, void* stream);

/* ---------------------------------------------------------------- a4-a6: expert FFN */

/* y = sum_k gates[k] * down_k( silu(gate_k(x)) * up_k(x) ), each projection = int4 base
 * dequantised on the fly + lora_scale * B (A .) (Sec. 3.1 "Math contract", Sec. 3.3), over
 * exactly the K given slots, summed in the order given.
 *   slot_pool   dev: n_slots records of one layer
 *   slot_table  dev int32 [E] or NULL.  NULL: `slots` holds slot indices in [0, n_slots).
 *               Non-NULL: `slots` holds expert ids, mapped on the device through the table
 *               (the paper's take; the indices never leave the GPU)
 *   slots       dev int32 [T][K]
 *   experts     dev int32 [T][K] expert ids, read only to pick per-expert adapters when
 *               n_adapters == E and slot_table is NULL; may be NULL otherwise
 *   gates       dev float [T][K]                        x       dev bf16 [T][H]
 *   lora        host struct of dev pointers, or NULL for no adapter
 *   y           dev [T][H] of out_dtype
 *   workspace   dev, edg_ffn_workspace_bytes(desc, T) bytes, 256-byte aligned; holds the
 *               intermediate h and the rank-r projections.  Its first 4096 bytes are a control
 *               block (sticky status word, see edg_workspace_status, and arrival counters) that
 *               the caller zeroes once before first use; the rest needs no initialisation.
 *               Calls that share a workspace must be ordered on the device.
 * An index outside its range makes the kernels skip that expert and raise the status word; no
 * out-of-range address is ever formed.
 * T = 1 is batch-1 decode (fused dequant GEMV kernels).  T > 1 is batched decode / prefill. */
int32_t moe_expert_ffn_int4_lora(const edg_layer_desc* desc, const void* slot_pool, const int32_t* slot_table,
                                 int32_t T, const int32_t* slots, const int32_t* experts, const float* gates,
                                 const void* x, const edg_lora* lora, void* y,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* The same batch-1 FFN (T = 1) for callers that cannot allocate device memory -- code running
 * inside another engine's memory plan, a loop that must stay away from the allocator once it has
 * started, a process whose GPU memory belongs to a pool it does not control.  (The paper has no
 * counterpart: this is an addition for such hosts.)  Inputs and outputs are passed as for
 * moe_expert_ffn_int4_lora; the kernel's scratch lives in a fixed 2 MiB array inside the library's
 * device image (every GPU that loads the library holds it until the process exits).  The call
 * makes no cudaMalloc / cudaFree and uses no allocating library routine.
 *   - Shapes whose scratch would not fit the array, or that the batch-1 kernel does not cover,
 *     are rejected with EDG_E_WORKSPACE / EDG_E_SHAPE.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before any stream capture.
 *   - All calls on a device share the array.  Each call clears the control block it needs at zero
 *     on `stream`; calls that overlap on the GPU (different streams without ordering) race.
 *   - Out-of-range slot or expert indices are skipped as in the other entry points, but there is
 *     no status word to read back. */
int32_t moe_expert_ffn_int4_lora_static(const edg_layer_desc* desc, const void* slot_pool,
                                        const int32_t* slot_table, const int32_t* slots,
                                        const int32_t* experts, const float* gates, const void* x,
                                        const edg_lora* lora, void* y, void* stream);

/* ---------------------------------------------------------------- the whole layer-step */

/* One layer-step of batch-1 decode (Sec. 3.2 "Motivation": the double shift).  On `stream`:
 * waits for the layer's staging copies, maps inds_cur through the layer's device slot table (take;
 * the indices never leave the GPU), runs a4-a6 for the current token with the routing predicted one
 * token earlier, and evaluates the head W_pre_next on the same hidden state to predict the next
 * layer-step's routing (a1-a2); then marks the layer's slots free for restaging.
 *   x dev bf16 [H]; inds_cur dev int32 [K]; gates_cur dev float [K];
 *   W_pre_next dev [E][H] (NULL skips the prediction); inds_next dev int32 [K];
 *   gates_next dev float [K]; logits_next_opt dev float [E] or NULL;
 *   inds_next_host_mirror_opt int32 [K] in mapped pinned host memory or NULL: a second copy of
 *   inds_next for the host-side stager, same protocol as in prerouter_topk;
 *   y dev [H] of out_dtype; workspace as for moe_expert_ffn_int4_lora with T = 1.
 *
 * Chained calls (opt-in, see edg_store_set_chaining).  When chaining is on and a call's inds_cur / gates_cur are the very buffers the previous call on this
 * store wrote as inds_next / gates_next, with the same workspace and stream, the two layer-steps
 * are chained: the later kernel is launched as a programmatic dependent of the earlier one, starts
 * as soon as that one is running, and takes its routing from a ring inside the workspace: the
 * earlier kernel leaves the logits of its head there and, behind them, the (expert, gate) pairs it
 * selects from them -- the same values it writes to inds_next / gates_next.  Up to 128 chained
 * steps share the GPU.  The results are those of unchained calls; what changes is the
 * contract on the inputs: a chained call reads x, W_pre_next and the slot pool as soon as it
 * starts, so they must already be valid when the call is made -- not produced by work queued
 * on the stream between the two calls.  Callers that cannot promise this leave chaining off
 * (the default).  A chain captured in a CUDA graph that is replayed back to back
 * must hold a multiple of 128 layer-steps, so that every replay finds the ring where the
 * previous one left it.  A replay is ordered behind the one before it like any other work on the
 * stream, so the chain of overlapping steps drains and refills once per replay (about half the
 * lifetime of a CTA): capture long chains (thousands of steps), not short ones. */
int32_t moe_layer_decode(edg_store* store, int32_t layer, const void* x,
                         const int32_t* inds_cur, const float* gates_cur,
                         const void* W_pre_next, int32_t* inds_next, float* gates_next,
                         float* logits_next_opt, int32_t* inds_next_host_mirror_opt, void* y,
                         void* workspace, size_t workspace_bytes, void* stream);

/* The same layer-step for a chain of data-dependent steps: besides y the kernel writes
 *     x_next = bf16(rmsnorm(x + y)),   rmsnorm(v) = v / sqrt(mean(v^2) + eps),  unit gain
 * (what edg_next_hidden_state computes, folded into the layer kernel's reduce: no second launch).
 * x_next dev bf16 [H], 16-byte aligned, not x itself.  With chaining switched on
 * (edg_store_set_chaining), a following call whose x is this call's x_next and whose inds_cur /
 * gates_cur are this call's inds_next / gates_next (same workspace and stream) is launched as a
 * programmatic dependent in the all-SM form: it starts while this step is still computing, takes
 * its routing from the hand-off ring, streams the first weights of its experts, and only then waits
 * (bounded, on a device flag) for this step to write x_next -- the overlap the paper's lead buys:
 * the routing is known a step ahead, the hidden state is not.  Results equal those of unchained calls. */
int32_t moe_layer_decode_dependent(edg_store* store, int32_t layer, const void* x,
                                   const int32_t* inds_cur, const float* gates_cur,
                                   const void* W_pre_next, int32_t* inds_next, float* gates_next,
                                   float* logits_next_opt, int32_t* inds_next_host_mirror_opt, void* y,
                                   void* x_next, float eps,
                                   void* workspace, size_t workspace_bytes, void* stream);

/* One token through all n_layers layers of the store (the paper's decode timeline, Sec. 3.2
 * "Motivation": full-token lead, one hand-off per token).  On the host: waits (bounded, 5 s) until the
 * previous token's kernels have mirrored the routing of every layer into mirror_cur; resets
 * mirror_next to -1; with prefetch != 0 stages the missing experts of ALL layers first, so that the
 * copies of later layers overlap the compute of earlier ones (prefetch == 0: each layer is staged
 * right before it runs -- the on-demand arm); then enqueues the n_layers layer-steps.  The head
 * owned by layer l, evaluated on layer l's input, predicts layer (l + 1) mod n_layers at the next
 * token (the double shift).  No stream synchronisation.
 *   x dev bf16 [L][H] layer inputs; inds_cur dev int32 [L][K], gates_cur dev float [L][K]: this
 *   token's routing; W_pre dev [L][E][H]; inds_next / gates_next dev [L][K], logits_next_opt dev
 *   [L][E] or NULL: the next token's routing (row (l+1) mod L written by layer l);
 *   mirror_cur / mirror_next int32 [L][K] in mapped pinned host memory: host copies of inds_cur
 *   (complete when all entries are >= 0) and of inds_next; y dev [L][H] of out_dtype;
 *   n_miss_out host, may be NULL: experts copied for this token.
 * Returns EDG_E_TIMEOUT when the routing does not arrive, EDG_E_RANGE on an expert id >= E. */
int32_t edg_stack_decode_token(edg_store* store, const void* x, const int32_t* inds_cur, const float* gates_cur,
                               const void* W_pre, int32_t* inds_next, float* gates_next, float* logits_next_opt,
                               const int32_t* mirror_cur, int32_t* mirror_next, void* y,
                               void* workspace, size_t workspace_bytes, void* stream,
                               int32_t prefetch, int32_t* n_miss_out);

/* Measurement of exposed staging time: with edg_store_time_waits(store, 1) every wait that
 * edg_store_wait_staged / moe_layer_decode actually enqueues on a compute stream is bracketed by a
 * pair of timing events (outside stream capture); edg_store_exposed_wait_ms synchronises on them,
 * returns the summed time the compute streams were held up by staging copies since the last call
 * and the number of waits, and resets both.  Enabling allocates events: not a hot call. */
int32_t edg_store_time_waits(edg_store* store, int32_t enable);
int32_t edg_store_exposed_wait_ms(edg_store* store, double* ms_out, int64_t* n_waits_out);

/* The hidden state a decoder would hand to the next layer-step: x_next = bf16(rmsnorm(x + y)),
 * unit gain, rmsnorm(v) = v / sqrt(mean(v^2) + eps) -- residual connection plus the next block's
 * input norm.  The paper's method has no such step (attention and the shared expert sit between
 * two MoE blocks there); this is the benchmark's stand-in that makes consecutive layer-steps
 * data-dependent.  x dev bf16 [H]; y dev [H] of desc->out_dtype; x_next dev bf16 [H]; H <= 4096. */
int32_t edg_next_hidden_state(const edg_layer_desc* desc, const void* x, const void* y, void* x_next,
                              float eps, void* stream);

/* Chaining of consecutive moe_layer_decode calls: 0 (default) off -- every layer-step is an
 * ordinary stream-ordered launch and the usual stream semantics hold for every input; 1 a call is
 * chained when the buffers line up and the step before it is still in flight (its completion
 * event has not fired) or the stream is being captured -- a step that finds the GPU idle is
 * launched on its own, across all SMs, which is several times faster for that single step;
 * 2 chained whenever the buffers line up.  Switching it on accepts the contract on the inputs of
 * chained calls stated above. */
int32_t edg_store_set_chaining(edg_store* store, int32_t enable);

#ifdef __cplusplus
}
#endif
#endif /* EDG_MOE_H */
