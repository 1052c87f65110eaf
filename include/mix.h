/*
 * mix.h -- C ABI of the per-layer MI hook for NVIDIA B200 (sm_100a).
 *
 * One call, mix_apply(), applies every registered MI function to the hidden states
 * bf16[T, d] of a continuously batched, ragged set of requests at one hook.  A device-side
 * token->slot map routes each token row to its request's function:
 *
 *   MIX_PROBE  read primitive  (paper, Section 3 "Read"; Section 4.2 "Executable units"):
 *              z_c = b_c + sum_i W[c,i] h[t,i];  score = sigmoid(z) | softmax(z) | z,
 *              written to the caller's score buffer (Section 4.2 "State and dataflow");
 *              the hidden row is not modified.
 *   MIX_STEER  write primitive (Section 3 "Write": add or subtract a vector):
 *              h[t,:] <- bf16( h[t,:] + alpha * v ), in place.
 *   MIX_SAE    sparse-autoencoder function (the paper names feature dictionaries only;
 *              the arithmetic is the standard one): z = W_enc h + b_enc, activation
 *              ReLU | JumpReLU (z > theta) | TopK (k largest pre-activations, then ReLU),
 *              per-feature edits (clamp: f_j = c; ablate: f_j = 0), decode from W_dec,
 *              optionally with the reconstruction error of the UNEDITED features added
 *              back:  h' = xhat(f') + (h - xhat(f)).
 *   MIX_PROJECT directional ablation, the usual statement of "subtract a vector" for a refusal-style
 *              direction (Section 3 "Write"; Table 1, row 1): h[t,:] <- bf16( h - beta (h . r) r ),
 *              in place; r is used as given (pass a unit vector for an orthogonal projection).
 *   slot -1    no app: the row is never written and stays bit-identical (Section 4.2 "Toggling
 *              semantics": an inactive app costs a request nothing).  It is not read either, with one
 *              exception: in a batch of more than 2048 rows, the 128-row tiles that hold multi-class
 *              probe rows are streamed whole by the probe kernel when those tiles are, together, at
 *              least half full of such rows; the rows of a tile that are not its own are discarded.
 *
 * Rows are independent.  Activation of an app for a request is data (the slot map and the
 * small device tables), never launch structure: mix_apply() only enqueues kernels with a
 * launch geometry fixed at mix_create(), performs no allocation, no host<->device
 * synchronisation and no host read of device state, so it may be captured once in a CUDA
 * graph at T_max rows and replayed while apps are toggled by the stream-ordered
 * mix_set_* / mix_register_* / mix_update_* calls (Section 4.2 "CUDA-graph-safe kernel
 * design", "Graph-level toggling and continuous batching").
 *
 * Conventions
 *   - every function returns MIX_OK (0) or a negative mix_status; nothing throws, aborts
 *     or prints.  mix_last_error() gives a message for the last failure on that context.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - "device" pointers are CUDA device pointers on the context's GPU; "host" pointers are
 *     ordinary host memory.  bf16 tensors are row-major, densely packed.
 *   - weights are BORROWED: the caller keeps them alive and unchanged until the app /
 *     weight set is unregistered (or the context destroyed) and work already enqueued has
 *     finished.  (The library may also keep its own copy of small weights -- contexts with
 *     T_max <= 2048 copy steering / projection vectors and one-class probe weights and biases at
 *     registration -- so changing borrowed weights in place needs a new registration.)
 *     Everything else (tables, edit lists, slot map) is copied.
 *   - one host thread per context at a time.
 */
#ifndef MIX_H_
#define MIX_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mix_ctx mix_ctx;

typedef enum {
  MIX_OK = 0,
  MIX_ERR_INVALID_ARG = -1,   /* NULL pointer, bad enum, misaligned pointer */
  MIX_ERR_OUT_OF_RANGE = -2,  /* an index or size exceeds what mix_create() was told */
  MIX_ERR_UNSUPPORTED = -3,   /* shape not supported by the kernels (see mix_create) */
  MIX_ERR_NO_MEMORY = -4,     /* device allocation failed in mix_create() */
  MIX_ERR_CUDA = -5           /* a CUDA call failed; see mix_last_error() */
} mix_status;

enum { MIX_PROBE = 1, MIX_STEER = 2, MIX_SAE = 3, MIX_PROJECT = 4, MIX_ROUTER = 5 };   /* app kinds */
enum { MIX_ACT_SIGMOID = 0, MIX_ACT_SOFTMAX = 1, MIX_ACT_NONE = 2 };   /* probe activations */
enum { MIX_SAE_RELU = 0, MIX_SAE_JUMPRELU = 1, MIX_SAE_TOPK = 2 };     /* SAE activations */
enum { MIX_EDIT_CLAMP = 0, MIX_EDIT_ABLATE = 1 };                      /* per-feature edits */
enum { MIX_GATE_GE = 0, MIX_GATE_LT = 1 };                             /* gate comparisons */

/* bits of the device status word (mix_get_status) */
enum {
  MIX_STATUS_BAD_SLOT = 1u << 0,      /* a live row named a slot id < -1, >= n_slots_max or unregistered; treated as -1 */
  MIX_STATUS_BAD_GROUP = 1u << 1,     /* an SAE app names a weight set that is not registered; rows pass through */
  MIX_STATUS_WAIT_TIMEOUT = 1u << 2,  /* a bounded wait inside the encode kernel expired; results of that call are invalid */
  MIX_STATUS_TOPK_GENERAL = 1u << 3   /* informational: a row's TopK needed the general (many-ties) selection path */
};

/* flags for mix_config.flags */
enum {
  MIX_FLAG_ENCODE_SIMT = 1u << 0,     /* run the SAE encode on the plain CUDA-core kernel instead of tcgen05 (cross-check) */
  MIX_FLAG_RETILE_W_ENC = 1u << 1     /* keep a library-owned copy of every registered W_enc, re-laid out so that each
                                         256-feature x 64-column encode tile is one contiguous 32 KiB block: the encode then
                                         streams whole DRAM pages instead of 128-byte pieces of 256 different rows.  Costs
                                         2 * d_sae * d bytes per weight set, allocated at registration (W_enc itself is no
                                         longer read by mix_apply and need not stay alive) */,
  MIX_FLAG_TEST_STALL_ENCODE = 1u << 2 /* test hook for the time-out path: the producer of the encode kernel (and of the
                                         tensor-core probe kernel) never delivers a
                                         tile and every bounded wait is capped at ~1 ms, so each CTA gives up, raises
                                         MIX_STATUS_WAIT_TIMEOUT, frees its tensor memory and returns; the SAE rows of that
                                         call are not meaningful.  Nothing hangs and the context stays usable */,
  MIX_FLAG_SAE_EDIT_ONLY = 1u << 3    /* algorithmic shortcut: rows of a ReLU / JumpReLU weight set whose app has the
                                         error term on skip the encode; only the pre-activations of their edited
                                         features are computed (|edits| dot products per row).  Same hidden output;
                                         n_active is not produced for those rows.  TopK rows are unaffected */,
  MIX_FLAG_SLOT_CHAINS = 1u << 4      /* allow mix_set_chain(): several apps applied, in order, to the same row in one
                                         mix_apply.  Probes and steering then run in one kernel that keeps the row in
                                         registers across the apps of its chain, and the SAE chain starts only after
                                         that kernel (the two no longer overlap).  Not together with
                                         MIX_FLAG_SAE_EDIT_ONLY */,
  MIX_FLAG_FP8_W_ENC = 1u << 5        /* every weight set of the context gives its encoder as 8-bit E4M3 codes with one
                                         fp32 scale per feature (mix_sae_weights.W_enc / W_enc_scale): the encoder takes
                                         half the HBM and the encode streams half the bytes.  The hidden state stays
                                         bf16: when an SAE row is packed it is split into two E4M3 operands hi + lo with
                                         one power-of-two scale s per row (s as under MIX_FLAG_FP8_ACT; hi = E4M3 nearest
                                         to h_i / s, lo = E4M3 nearest to the remainder), which reproduces h_i exactly for
                                         |h_i| >= s / 4 and to within s * 2^-10 (<= 4.4e-6 max|h|) below that, and the
                                         8-bit tensor-core contraction (kind::f8f6f4) accumulates hi W and lo W into one
                                         fp32 accumulator that the epilogue scales by s * W_enc_scale[j].  Measured: 1.3x
                                         faster than the bf16 encoder where the stream of W_enc is the bound, 1.1x where
                                         the tensor pipe is.  The paper has no counterpart.  Needs d_model to be a
                                         multiple of 128.  Not together with MIX_FLAG_ENCODE_SIMT,
                                         MIX_FLAG_SAE_EDIT_ONLY or center_input */,
  MIX_FLAG_FP8_ACT = 1u << 6          /* only with MIX_FLAG_FP8_W_ENC: the encoder's INPUT is quantised to 8 bits too
                                         (one E4M3 operand per row instead of the exact pair): half the tensor work and
                                         half the panel bytes of the flag above.  Each SAE row of `hidden` is quantised when it is
                                         packed: s = the smallest power of two with max|h_i| / s <= 448 (2^0 for a zero
                                         row, never below 2^-100), code_i = E4M3 nearest to h_i / s, ties to the even
                                         code; the encoder then sees s * e4m3(code_i) in place of h_i:
                                           z_j = s * W_enc_scale[j] * sum_i e4m3(code_i) e4m3(W_enc[j, i]) + b_enc[j].
                                         Everything after the pre-activations (selection, edits, decode, the error term
                                         and the write-back) works on the unquantised bf16 row as before.  This changes
                                         the pre-activations by up to the quantisation step of the row (2^-4 relative per
                                         element): an accuracy / speed trade the caller opts into; the paper has no
                                         counterpart.  Rows with non-finite entries are not supported by either 8-bit
                                         flag */
};

typedef struct {
  int d_model;          /* hidden width d; multiple of 64 (16-byte vectors, 128-byte TMA rows) */
  int T_max;            /* rows of every `hidden` passed to mix_apply (the capture size) */
  int n_slots_max;      /* app slots 0 .. n_slots_max-1 */
  int n_groups_max;     /* SAE weight sets 0 .. n_groups_max-1; 0 = no SAE kernels are ever launched */
  int C_max;            /* row stride of scores_out and largest n_classes (<= 64) */
  int k_max;            /* largest TopK k (<= 1024); also the row stride of the feature outputs */
  int r_max;            /* largest edit list per SAE app (<= 64) */
  long long d_sae_max;  /* largest SAE width; multiple of 256 */
  unsigned flags;       /* MIX_FLAG_* */
} mix_config;

/* Read primitive.  W: device bf16 [n_classes, d].  b: device fp32 [n_classes] or NULL (= 0).
   act = MIX_ACT_SIGMOID requires n_classes == 1. */
typedef struct {
  int n_classes;
  int act;
  const void* W;
  const float* b;
} mix_probe;

/* Write primitive.  v: device bf16 [d]; used as given (not normalised); alpha any sign. */
typedef struct {
  const void* v;
  float alpha;
} mix_steer;

/* Directional ablation.  r: device bf16 [d], used as given; beta = 1 removes the component along
   r (for unit r), 0 < beta < 1 shrinks it, beta = 0 leaves the row untouched bit for bit. */
typedef struct {
  const void* r;
  float beta;
} mix_project;

/* MoE router-logit steering (paper, Table 1 row 7: a conditional write whose target is the router
   logits, used to switch experts on or off).  delta: device fp32 [n_experts], added to the router
   logits of the app's rows by mix_apply_router(); +-INFINITY entries force an expert in or out of
   the top-k that the model's router takes afterwards.  mix_apply() ignores apps of this kind. */
typedef struct {
  int n_experts;
  const float* delta;
} mix_router;

/* One SAE weight set, shared by any number of app slots.  All pointers device.
   W_enc bf16 [d_sae, d]: row j = encoder direction j.  b_enc fp32 [d_sae].
   theta fp32 [d_sae] (JumpReLU only, else NULL).  W_dec bf16 [d_sae, d]: row j = decoder
   direction j.  b_dec fp32 [d] or NULL.  center_input != 0 subtracts b_dec from the input
   before the encoder (folded into an effective bias at registration; needs b_dec).
   k: TopK only, 1 <= k <= min(k_max, d_sae).
   In a context created with MIX_FLAG_FP8_W_ENC, W_enc is uint8 [d_sae, d] instead: E4M3 codes
   (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; the NaN codes 0x7F / 0xFF must not
   occur), and W_enc_scale fp32 [d_sae] is required: encoder entry (j, i) = e4m3(code[j, i]) *
   W_enc_scale[j].  The library keeps its own tile-ordered copy of the codes (d_sae * d bytes);
   W_enc need not stay alive after registration, W_enc_scale must.  Otherwise W_enc_scale is
   ignored. */
typedef struct {
  long long d_sae;
  int act;
  int k;
  const void* W_enc;
  const float* b_enc;
  const float* theta;
  const void* W_dec;
  const float* b_dec;
  int center_input;
  const float* W_enc_scale;
} mix_sae_weights;

/* One SAE app slot = (weight set, edit list, error-term flag).  idx/val/mode are HOST arrays
   of n_edit entries, copied; if an index occurs twice the later entry wins.  add_error != 0:
   h' = xhat(f') + (h - xhat(f)) (a row with no effective edit is left untouched, bit for
   bit); add_error == 0: h' = xhat(f'). */
typedef struct {
  int group;
  int n_edit;
  const int* idx;
  const float* val;
  const unsigned char* mode;
  int add_error;
} mix_sae_app;

/* Create a context on the CURRENT CUDA device and allocate every table and workspace the
   hook will ever need (the only allocating call besides registration of a centred SAE).
   (Paper, Section 4.2 "State and dataflow": an app's state -- parameters, buffers -- is set up ahead
   of time and lives on the device; "CUDA-graph-safe kernel design": the static part of the launch
   structure is fixed once, here, at the capture size T_max.)
   Workspace: a bf16 panel of (T_max + 128*n_groups_max) x d and an fp32 pre-activation
   scratch of the same rows x d_sae_max, when n_groups_max > 0.
   Errors: INVALID_ARG (NULL, non-positive sizes), UNSUPPORTED (d_model % 64, d_sae_max % 256,
   C_max > 64, k_max > 1024, r_max > 64), NO_MEMORY, CUDA. */
int mix_create(mix_ctx** out, const mix_config* cfg);

/* Free everything the context owns.  Synchronises the device.  NULL is a no-op. */
int mix_destroy(mix_ctx* ctx);

/* Message for the last error on this context (static storage, valid until the next call). */
const char* mix_last_error(const mix_ctx* ctx);

/* Register / replace SAE weight set `group` (stream-ordered table write).  Not captured.
   Replacing a set while SAE apps are attached to it is allowed as long as the new d_sae still
   covers every feature those apps edit; otherwise the call fails and changes nothing (unregister
   the apps or give them new edit lists first).
   Errors: OUT_OF_RANGE (group, d_sae > d_sae_max, k), UNSUPPORTED (d_sae % 256), INVALID_ARG
   (NULL or pointers not 16-byte aligned, JumpReLU without theta, centring without b_dec, a
   replacement too narrow for an attached app's edits). */
int mix_register_sae_weights(mix_ctx* ctx, int group, const mix_sae_weights* w, void* stream);
int mix_unregister_sae_weights(mix_ctx* ctx, int group, void* stream);

/* Attach an MI function to `slot` (paper, Section 4.2: functions are attached ahead of time
   with their parameters).  `desc` points to a mix_probe, mix_steer, mix_sae_app, mix_project or
   mix_router according to `kind`.  Stream-ordered; an entry becomes visible atomically (its valid flag is
   written last).  Errors: OUT_OF_RANGE (slot, n_classes > C_max, n_edit > r_max, edit
   index >= d_sae of the group, group), INVALID_ARG. */
int mix_register_app(mix_ctx* ctx, int slot, int kind, const void* desc, void* stream);

/* Make `slot` pass-through again.  Rows still naming it are left untouched and raise
   MIX_STATUS_BAD_SLOT. */
int mix_unregister_app(mix_ctx* ctx, int slot, void* stream);

/* Cheap toggles that never touch launch structure (Section 4.2 "Toggling semantics").
   mix_update_steer_alpha also sets beta of a MIX_PROJECT app.  mix_update_sae_edits validates the
   whole list first: a call that fails has changed nothing, on the host or on the device. */
int mix_update_steer_alpha(mix_ctx* ctx, int slot, float alpha, void* stream);
int mix_update_sae_edits(mix_ctx* ctx, int slot, int n_edit, const int* idx, const float* val,
                         const unsigned char* mode, void* stream);

/* Conditional write driven by an earlier read (paper, Section 3 "Conditional Write": the
   condition can depend on activations at another layer; Section 4.1, the example
   gate="probe(layer=18) >= 0"; Section 4.2 "State and dataflow" / "Activation and control
   semantics": a buffer written at one hook decides, on the device, whether a function at a
   later hook runs).  After this call the app in `slot` applies to token row t only if
       scores[t * row_stride + column]  >=  threshold      (MIX_GATE_GE)
       scores[t * row_stride + column]  <   threshold      (MIX_GATE_LT)
   and the row passes through untouched otherwise (a NaN score fails either comparison).
   `scores` is a device fp32 buffer indexed by token row, typically the scores_out of a
   mix_apply() at an earlier layer of the same forward pass (use MIX_ACT_NONE probes to gate on
   the raw logit); it is read when the later mix_apply() runs, so both calls can sit in one
   captured graph.  scores == NULL removes the gate.  Registering the slot again also removes
   it.  Stream-ordered, not captured.  Works for every app kind (a gated probe writes no score
   for rows whose gate is closed).  Errors: OUT_OF_RANGE (slot), INVALID_ARG (slot not
   registered, bad cmp, row_stride < 1, column outside [0, row_stride)). */
int mix_set_gate(mix_ctx* ctx, int slot, const float* scores, int row_stride, int column, int cmp, float threshold,
                 void* stream);

/* Several apps on one row (the paper's composition model: every app contributes its own hook
   functions and state, and the runtime applies the active ones at the hook; the evaluation's
   "All Apps Combined" configuration).  After mix_set_chain(slot, next_slot) a row whose token
   slot is `slot` gets the app of `slot` and then the app of `next_slot` (and so on along
   next_slot's own link; at most 4 apps per row), each app seeing the row as the previous one left
   it, rounded to bf16 -- bit for bit what separate mix_apply calls, one app each, would give.
   Every app keeps its own gate: a closed gate skips that app only.  The probes of a chain write
   their scores side by side: a probe's first column in scores_out[t, :] is the total n_classes of
   the chain's earlier probes (whether their gates were open or not), so the sum over a chain
   must not exceed C_max.  An SAE app can only be the last app of a chain; router apps cannot be
   chained.  next_slot = -1 removes the link.  Registering `slot` again removes its link;
   unregistering a slot removes the links that point to it.  The context must have been created
   with MIX_FLAG_SLOT_CHAINS.  Stream-ordered, not captured.
   Errors: INVALID_ARG (flag missing; a slot without an app; an app kind that cannot be chained
   there; a cycle; a chain longer than 4; class columns beyond C_max), OUT_OF_RANGE (slot ids). */
int mix_set_chain(mix_ctx* ctx, int slot, int next_slot, void* stream);

/* (Paper, Section 4.2 "Toggling semantics" and "Graph-level toggling and continuous batching":
   which requests of the running batch an app is active for is per-request data that changes from
   step to step while the captured launch structure stays as it is.)
   Install the token->slot map for the next mix_apply calls: token_slot int32[T_live]
   (host if src_is_device == 0, else device), -1 = no app.  Rows >= T_live are pass-through.
   One async copy + a 4-byte store into fixed device buffers; never captured in a graph.
   A host source must stay valid until the stream reaches the copy (use pinned memory for a
   truly asynchronous copy).  Errors: OUT_OF_RANGE (T_live < 0 or > T_max). */
int mix_set_slot_map(mix_ctx* ctx, const int* token_slot, int T_live, int src_is_device, void* stream);

/* Two-level form of the same map (Section 4.2 "Toggling semantics": activation is per REQUEST; a
   continuous-batching engine already holds token -> request): slot of token t =
   req_slot[token_req[t]] (token_req < 0 or >= n_req -> -1), composed on the device.  Both arrays
   host or both device. */
int mix_set_request_map(mix_ctx* ctx, const int* token_req, int T_live, const int* req_slot, int n_req,
                        int src_is_device, void* stream);

/* Optional feature read-out (Section 3 "Read" applied to SAE features; Section 4.2 "State and
   dataflow": values read at a hook go to buffers the app owns) (device buffers, NULL = off):
   topk_idx int32 [T_max, k_max] and
   topk_val fp32 [T_max, k_max] receive, for every TopK-SAE row, the selected feature ids
   in order of decreasing pre-activation (ties: lower id first) and those pre-activations
   (before ReLU and before edits); entries k..k_max-1 and other rows are not written.
   n_active int32 [T_max] receives, for every SAE row, the number of features with f_j > 0
   before edits.  Takes effect for later mix_apply calls; a captured graph keeps the
   pointers it was captured with. */
int mix_set_feature_out(mix_ctx* ctx, int* topk_idx, float* topk_val, int* n_active);

/* Apply the hook (Section 4.2 "Executable units": the functions attached at a hook run as GPU
   kernels on the hidden states that pass it; Section 3: read, write, conditional write; "CUDA-
   graph-safe kernel design": capturable, nothing about a request is baked into the launch).
   hidden: device bf16 [T_max, d], modified in place.  T: number of rows of
   `hidden` that may be live (<= T_max; rows >= min(T, T_live) are pass-through).  scores_out:
   device fp32 [T_max, C_max] or NULL; only the first n_classes entries of probe rows are
   written.  Enqueues kernels on `stream` (when the context has SAE weight sets, the probe /
   steering kernels run on a context-owned side stream forked from and joined back into `stream`
   by events, so they overlap the SAE chain; in a context for more than 2048 rows with multi-class
   probes and no SAE weight sets, the tensor-core probe kernel runs on that side stream beside the
   streaming kernel) and returns; safe to capture.  In a context without SAE weight sets and
   T_max <= 2048 the kernel is launched with programmatic stream serialization (see
   mix_set_pdl_mask): if the kernel in front of it in `stream` lets its successor start early, the
   part that looks up the live count, slot map, app entry and single-vector weights -- tables the
   library owns and only copies write -- overlaps that kernel; `hidden`, gate scores and
   multi-class probe weights are read only after the predecessor has completed and flushed, and the
   grid does not end before it.  Behind any other kernel nothing changes.  One launch shape follows
   from what is registered when the call is enqueued or captured -- the encode's epilogue warps
   (TopK weight set present or not); this is performance only: either shape handles every
   registration, so tables rewritten after a capture are still applied correctly.  Device-side
   problems (bad slot ids, ...) are reported through the status word, never by faulting.
   Errors: INVALID_ARG (NULL hidden, misaligned), OUT_OF_RANGE (T), CUDA (launch failure). */
int mix_apply(mix_ctx* ctx, void* hidden, int T, float* scores_out, void* stream);

/* mix_apply() with the SAE chain under a device-side predicate (implementation section of the
   paper, paragraph "Graph-level toggling and continuous batching": for true data-dependent
   control flow an upstream GPU computation decides whether a downstream intervention body
   executes, as with CUDA conditional nodes, with no CPU in the loop).  `stream` MUST be capturing: the call adds to
   the graph being captured the probe / steering kernels and the routing kernel as mix_apply() does,
   then one conditional IF node whose body holds the rest of the SAE chain (encode, selection,
   decode); the routing kernel sets the node's condition to (SAE rows routed > 0).  A
   replay with no SAE row live therefore launches none of the body's kernels, instead of four
   kernels that each find nothing to do.  Results are identical to mix_apply()'s.  The capture
   continues after the node; work captured later on `stream` depends on it.  A context without
   weight sets behaves exactly like mix_apply() (and then `stream` need not be capturing).
   Errors: as mix_apply(), plus INVALID_ARG (`stream` is not capturing; stage events are on). */
int mix_apply_conditional(mix_ctx* ctx, void* hidden, int T, float* scores_out, void* stream);

/* The hook on a different target tensor: router logits (device fp32 [T_max, n_experts], modified in
   place).  Rows whose slot holds a MIX_ROUTER app with the same n_experts (and an open gate, if it
   has one) get logits[t, :] += delta; every other row is neither read nor written.  Uses the same
   slot map, live count and gates as mix_apply(); one kernel, capturable.
   Errors: INVALID_ARG (NULL logits, n_experts < 1), OUT_OF_RANGE (T). */
int mix_apply_router(mix_ctx* ctx, float* logits, int n_experts, int T, void* stream);

/* Copy the device status word (bits MIX_STATUS_*) to *bits and clear it on the device.
   Synchronises `stream`.  (Section 4.2 "CUDA-graph-safe kernel design" rules out a host check in
   the middle of a replayed graph: device-side problems are therefore recorded in a word the host
   reads when it chooses to, never raised as a fault.) */
int mix_get_status(mix_ctx* ctx, unsigned* bits, void* stream);

/* Number of kernels one mix_apply() call launches on this context (fixed at mix_create):
   1 without SAE weight sets, else 7 (4 with MIX_FLAG_ENCODE_SIMT); one more when T_max > 2048
   and C_max > 1 (multi-class probes of large batches run in a kernel of their own), and two more
   with MIX_FLAG_SAE_EDIT_ONLY. */
int mix_launches_per_apply(const mix_ctx* ctx);

/* Per-kernel timing taps (profiling only; do not use while capturing a graph).  events: HOST
   array of mix_launches_per_apply() + 1 cudaEvent_t handles created by the caller with timing
   enabled, or NULL to switch the taps off.  Every later mix_apply() records events[0] before
   its first kernel and events[i] after its i-th kernel, on the call's stream; the array is
   copied.  Kernel order: [probe_decide,] probe_steer, [probe_multiclass: only if T_max > 2048 and C_max > 1;
   probe_decide before and probe_tc after it if also n_groups_max == 0,]
   front (routing + row pack), encode on single CTAs, encode on CTA pairs (the front kernel deals the
   call's weight sets between the two from the routing result -- sets with an even number of 128-row
   tiles to the pairs, when that pays -- and a kernel without a set returns at once; a stage event is
   recorded for both even where one is never launched), tail (selection, edits, decode, write-back), encode (row tiles flagged for the exact
   fallback selection), tail (the flagged rows); with MIX_FLAG_ENCODE_SIMT the SAE part is front, encode,
   tail; with MIX_FLAG_SAE_EDIT_ONLY an edit_only and an edit_only_delta
   kernel come last. */
int mix_set_stage_events(mix_ctx* ctx, void* const* events);

/* Measurement aid for the paper's "CUDA-graph-safe kernel design" paragraph (separate static graph
   structure from per-request dynamic parameters; reuse the instantiated graph and update only the
   affected kernel-node parameters before launch).  This library never updates node parameters: all
   dynamic state lives in device tables written by stream-ordered copies.  The call times both
   mechanisms on a one-kernel graph, `iters` times each, host wall clock per iteration including the
   graph launch, with one synchronisation at the end: (a) a 4-byte cudaMemcpyAsync into a device table
   the kernel reads, then cudaGraphLaunch; (b) cudaGraphExecKernelNodeSetParams with the new value
   as a kernel argument, then cudaGraphLaunch.  Both kernels add the value to an accumulator and
   the two sums are compared.  us_table / us_node: host floats, microseconds per iteration.
   Synchronises `stream`; not capturable; allocates and frees 8 bytes of device memory.
   Errors: INVALID_ARG (NULL outputs, iters < 1), CUDA (API failure or the two sums differ). */
int mix_bench_param_update(mix_ctx* ctx, int iters, float* us_table, float* us_node, void* stream);

/* Which launches of the library use programmatic dependent launch (a kernel's CTAs may become resident,
   and run the part of the kernel that reads only library-owned tables, while the kernel in front of
   it in the stream is still running; everything the predecessor may have written is read after an
   in-kernel wait).  Bits: 1 unused (the row pack is part of the first kernel of the SAE chain),
   2 the full SAE encode pass (the kernel in front of it lets it start only when its own rows are packed),
   4 the kernels after it, 8 the one-CTA-per-row probe / steering kernel of a context that has no SAE weight sets
   (T_max <= 2048).  Default 1 | 2 | 4 | 8, or the value of MIX_PDL_MASK in the environment when the
   library first launches.  Process-wide; affects launches (and captures) made afterwards; meant
   for A/B measurement.  Returns the previous mask.  mask < 0 only queries. */
int mix_set_pdl_mask(int mask);

/* Test / profiling taps into the SAE workspace after a mix_apply (device pointers owned by
   the context; valid until mix_destroy):  panel_rows int32 [n_panel_rows] gives the token
   index of each packed panel row (-1 = padding), z the fp32 pre-activations
   [n_panel_rows, ld_z].  Any out pointer may be NULL. */
int mix_debug_workspace(mix_ctx* ctx, const int** panel_rows, const float** z, long long* ld_z,
                        int* n_panel_rows);

/* Profiling aid (no counterpart in the paper).  A context created while MIX_PHASE_CLOCKS=1 is set in the
   environment keeps 32 words in which the first CTA of the SAE chain's front, encode and tail kernels stamps
   the GPU's nanosecond timer (words 0, 7, 8, 15, 26..31) or its SM's cycle counter (the others) at its phase
   boundaries (0..4 front: start, rows classified, routing scanned, positions found, rows packed; 7..15 tail:
   launched, predecessor done, row 0 read, candidates narrowed, sorted, TopK known, coefficients known, row
   written, CTA done; 16..25 steps inside the tail's selection and its delta role; 26..29 single-CTA encode:
   predecessor done, tensor memory allocated, last copy issued, CTA done; 30, 31 the end of the LAST CTA of the
   tail's main and fallback launches).  out32: HOST array of 32 words,
   zeros when the context was created without the variable.  Synchronises the device. */
int mix_debug_phase_clocks(mix_ctx* ctx, unsigned long long* out32);

/* ---------------------------------------------------------------------------------------
 * SAE function for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this call; it exists for integration reasons only.)
 *
 * Who needs it: code that runs inside a serving engine which has already handed the whole
 * HBM budget to its own pools (weights, KV cache) and forbids plugins to call cudaMalloc;
 * code on a latency-critical path, where cudaMalloc / cudaFree would stall the device with
 * their implicit synchronisation; and tools that must leave the process's allocator state
 * untouched.  Such callers cannot use mix_create(), which allocates the hook's tables and
 * workspace.  This single call needs no context: all of its scratch (tables, routing state,
 * the packed bf16 row panel, the fp32 pre-activations, TopK lists) sits in one fixed array
 * inside the library image, about 5.2 MiB, which every GPU that loads the library keeps
 * until the process exits.  The call allocates nothing and frees nothing.
 *
 * What it computes: the MIX_SAE function of mix_apply() for ONE app on EVERY one of the
 * n_rows rows of `hidden` (device bf16 [n_rows, d_model], modified in place): encode,
 * ReLU / JumpReLU / TopK, the app's edits, decode, error term as `app->add_error` says.
 * `w` and `app` are host structs as for registration (w's pointers device, app's edit
 * arrays host, app->group ignored).  topk_idx int32 / topk_val fp32 [n_rows, w->k]: optional
 * device outputs for TopK SAEs (NULL = off), as in mix_set_feature_out with k_max = w->k.
 * The encode runs on the CUDA-core kernel (the one MIX_FLAG_ENCODE_SIMT selects).
 *
 * Limits (the array has a fixed size): n_rows <= MIX_STATIC_MAX_ROWS, d_model <=
 * MIX_STATIC_MAX_D_MODEL (multiple of 64), w->d_sae <= MIX_STATIC_MAX_D_SAE (multiple of 256),
 * w->k <= MIX_STATIC_MAX_K, app->n_edit <= 64, no input centring.  Anything beyond returns
 * MIX_ERR_OUT_OF_RANGE / MIX_ERR_UNSUPPORTED with a message in errbuf (optional, host).
 *
 * Sharing: every call on a device uses the same array, and the array keeps the previous
 * call's contents; each call rewrites what it reads, so consecutive calls on one stream are
 * independent, but two calls that overlap on the GPU (different streams, or different host
 * threads) race on it -- serialise them.  The first call on each device looks up the
 * array's device address (no allocation); make that first call before any stream capture
 * begins.  The look-up stores one pointer per device without a lock: two host threads whose
 * first calls on one device coincide both store the same value, which is harmless, but the
 * calls themselves still race on the array as said above.  `w`, `app` and the edit arrays are
 * read before the call returns and reach the GPU as kernel arguments; no host memory of the
 * caller is referenced afterwards.  Enqueues on `stream` and returns; results are ready when
 * the stream reaches them.  The path has no status word the caller could read: every argument
 * that could raise a device-side status bit is rejected on the host instead. */
#define MIX_STATIC_MAX_ROWS 128
#define MIX_STATIC_MAX_D_MODEL 4096
#define MIX_STATIC_MAX_D_SAE 8192
#define MIX_STATIC_MAX_K 128
int mix_sae_apply_static(void* hidden, int n_rows, int d_model, const mix_sae_weights* w, const mix_sae_app* app,
                         int* topk_idx, float* topk_val, void* stream, char* errbuf, int errbuf_len);

#ifdef __cplusplus
}
#endif
#endif /* MIX_H_ */
