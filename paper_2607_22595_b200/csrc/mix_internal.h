// Internal declarations shared by the translation units of libmix.so.
// Device tables live at fixed addresses owned by the context; kernels read every piece of
// dynamic state (slot map, live count, app table, edit lists, route results) from them, so
// a captured graph never needs its kernel parameters changed.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mix.h"

namespace mix {

constexpr int kTileM = 128;        // token rows per encode tile (UMMA M)
constexpr int kTileN = 256;        // SAE features per encode tile (UMMA N)
constexpr int kTileK = 64;         // bf16 elements per 128-byte swizzled smem row
constexpr int kMaxGroups = 32;
constexpr int kTeamMaxRows = 2048;  // contexts up to this T_max run probes / steering with one CTA per row
constexpr int kMaxClasses = 64;
constexpr int kMaxK = 1024;
constexpr int kMaxEdits = 64;
constexpr int kTauSlots = 128;      // per packed row: slots of the running lower bound on the row's k-th largest pre-activation (k <= 128)
constexpr int kCandPerTile = 8;     // TopK candidates the encode epilogue keeps per (row, feature tile)
constexpr int kCandMax = 4096;      // candidates per row the tail kernel can stage in shared memory

struct __align__(16) AppEntry {
  int valid;          // written last by registration; 0 = slot is pass-through
  int kind;           // MIX_PROBE | MIX_STEER | MIX_SAE, | kKindGated
  int n_classes;      // probe
  int act;            // probe
  float alpha;        // steer
  int group;          // sae
  int n_edit;         // sae
  int add_error;      // sae
  const void* W;      // probe: bf16 [C, d]; steer: bf16 [d]
  const float* b;     // probe: fp32 [C] or null
};

constexpr int kKindMask = 0xff;     // AppEntry.kind: low byte = MIX_* kind
constexpr int kKindGated = 0x100;   //                bit 8    = the slot has a gate (see GateEntry)
constexpr int kKindChained = 0x200; //                bit 9    = another app follows on the same row (chain_next[slot])
constexpr int kMaxChain = 4;        // apps applied to one row in one call

// Gate of a slot: the app applies to row t iff cmp(scores[t * stride + col], thr).
struct __align__(16) GateEntry {
  const float* scores;
  int stride;
  int col;
  int cmp;            // MIX_GATE_GE | MIX_GATE_LT
  float thr;
  int pad_[2];
};

struct __align__(16) GroupEntry {
  int valid;
  int act;
  int k;
  int pad_;
  long long d_sae;
  const __nv_bfloat16* W_enc;
  const float* b_eff;   // b_enc, or b_enc - W_enc b_dec when the input is centred
  const float* theta;
  const __nv_bfloat16* W_dec;
  const float* b_dec;
  const float* w_scale; // 8-bit encoder: per-feature scale of the E4M3 codes, else null
  const void* pad2_;
};

// What the front kernel leaves about one packed panel row for the kernels behind the encode: two 16-byte loads
// instead of the chain panel row -> slot map -> app entry -> weight-set entry.
struct __align__(16) RowRec {
  int t;                            // token row, or -1: padding row of a tile
  int slot;                         // slot of the SAE app that acts on the row (the row's own, or the last of its chain)
  int n_edit;                       // length of that app's edit list
  int group_flags;                  // low byte: weight set; kRecAddError: the app keeps the error term; bits 16..17: the set's activation
  const __nv_bfloat16* W_dec;       // the set's decoder
  const float* theta;               // the set's JumpReLU thresholds, or null
};
constexpr int kRecGroupMask = 0xff;
constexpr int kRecAddError = 0x100;
constexpr int kRecActShift = 16;

// What sae_edit_only_kernel leaves for decode_delta_kernel about one token row.
struct __align__(16) RowDelta {
  int slot;                         // the row's slot, or -1: nothing to add (no effective edit, other kind of row)
  int n_edit;
  const __nv_bfloat16* W_dec;
};

// Census of a large batch's multi-class probe rows (contexts of more than 2048 rows with such probes and no SAE
// weight sets): which 128-row tiles hold any, how many rows in all, and which of the two probe kernels takes the call.
struct McCensus {
  int n_tiles, n_rows, use_tc, pad_;     // the result the probe kernels read
  int w_tiles, w_rows, w_done, pad2_;    // counters of the census in progress (zero between calls)
};

// Result of the routing step for the SAE path (one instance in device memory).
struct RouteState {
  int n_panel_rows;                 // rows of the packed panel in use (multiple of kTileM)
  int n_sae_rows;                   // SAE rows routed this call
  int n_mtiles;                     // = n_panel_rows / kTileM
  int total_tiles;                  // encode tiles over all groups
  int n_topk_rows;                  // SAE rows whose weight set is TopK
  int n_delta_rows;                 // ReLU / JumpReLU rows that keep the error term and have edits (the tail kernel's delta role)
  int use_pair;                     // some weight set of this call is encoded by CTA pairs (256-row tiles)
  int pair_mask;                    // bit g: weight set g is the pair kernel's this call, else the single-CTA kernel's
  int group_count[kMaxGroups];      // M_g
  int group_mtile0[kMaxGroups + 1]; // first m-tile of group g in the panel
  int group_tile0[kMaxGroups + 1];  // first linear encode tile of group g
};

struct Ctx {
  mix_config cfg;
  int device;
  int n_sms;
  char err[256];

  // tables
  int* d_token_slot;        // [T_max]
  int* d_n_live;            // [1]
  AppEntry* d_apps;         // [n_slots_max]
  GroupEntry* d_groups;     // [n_groups_max]
  GateEntry* d_gates;       // [n_slots_max]
  int* d_chain_next;        // [n_slots_max] next slot applied to the same row, or -1 (MIX_FLAG_SLOT_CHAINS)
  int* h_chain_next;        // host mirror
  int* h_edit_idx;          // host mirror of d_edit_idx (validation when a weight set is replaced)
  __nv_bfloat16* d_vec_arena;   // [n_slots_max, d] copies of single-vector weights (T_max <= kTeamMaxRows), else null
  int* d_edit_idx;          // [n_slots_max * r_max]
  float* d_edit_val;
  unsigned char* d_edit_mode;
  unsigned* d_status;
  int* d_tmp_req;           // [T_max] staging for the two-level map
  int* d_tmp_req_slot;      // [T_max]

  // host mirrors (validation only)
  AppEntry* h_apps;
  GroupEntry* h_groups;
  float** owned_b_eff;      // per group: library-owned folded bias or null
  __nv_bfloat16** owned_w_tiled;   // per group: library-owned tile-contiguous copy of W_enc or null

  // SAE workspace
  int panel_rows_cap;       // P
  __nv_bfloat16* d_panel;   // [P, d]  (MIX_FLAG_FP8_ACT: the same memory holds E4M3 codes, uint8 [P, d])
  float* d_act_scale;       // [P] row scales of the 8-bit panel (MIX_FLAG_FP8_ACT only)
  int* d_panel_row;         // [P] token index or -1
  int* d_mtile_group;       // [P / kTileM] group of each m-tile or -1
  int2* d_row_meta;         // [T_max] front kernel: per token row, what its chunk's CTA found out (weight set, edit count, flags; slot)
  int* d_front_counts;      // [chunks of 256 token rows][n_groups_max + 1] front kernel: SAE rows per weight set and chunk
  int* d_front_sync;        // [2] front kernel: chunks published / CTAs done in the running call (zero between calls)
  RowRec* d_row_rec;        // [P] per packed row: token row, slot, edit count, weight set, error-term flag
  RouteState* d_route;
  float* d_z;               // [P, d_sae_max]
  float* d_cand_val;        // [P, cand_tiles, kCandPerTile] per-tile TopK candidates (fused epilogue)
  int* d_cand_idx;          // same shape: feature ids
  float* d_cand_ninth;      // [P, cand_tiles] the (kCandPerTile+1)-th largest value of each tile
  RowDelta* d_eo_row_delta; // [T_max] edit-only shortcut: per token row, what decode_delta_kernel adds (MIX_FLAG_SAE_EDIT_ONLY)
  float* d_eo_coef;         // [T_max, r_max]
  unsigned* d_tau_min;      // [P] the smallest of the row's first k slots, as last computed by a publisher
  unsigned* d_tau;          // [P, kTauSlots] order-preserving keys of pre-activations seen so far in this call (0 = empty)
  int cand_tiles;           // d_sae_max / kTileN
  int* d_row_flag;          // [P] row needs the exact fallback selection
  int* d_mtile_flag;        // [P / kTileM] some row of the tile is flagged
  int* d_n_flagged;         // [1]
  CUtensorMap* d_tmap_w;    // [n_groups_max] W_enc maps (box kTileK x kTileN, 128B swizzle)
  CUtensorMap* d_tmap_w_half;   // [n_groups_max] the same with boxes of kTileN / 2 rows: what one CTA of a pair fetches
  CUtensorMap* d_tmap_probe;   // [n_slots_max] maps of multi-class probe matrices (box kTileK x 32), large-batch contexts only
  McCensus* d_mc_census;    // census of the 128-row tiles that hold multi-class probe rows, taken by mc_census_kernel every call
  int* d_mc_tiles;          // [ceil(T_max / 128)] those tiles, in no particular order
  CUtensorMap tmap_panel;   // panel map (box kTileK x kTileM, 128B swizzle)

  // probe/steer kernels run beside the SAE chain on this stream (created with the context)
  cudaStream_t side_stream;
  cudaStream_t body_stream;   // used only to record the body of a conditional node (mix_apply_conditional)
  cudaEvent_t ev_fork, ev_join;

  // profiling taps
  int map_from_kernel;      // the slot map was last written by compose_map_kernel, not by a copy: the next hook kernel
                            // must not read it ahead of its predecessor
  int stage_events_on;
  cudaEvent_t stage_events[16];

  unsigned long long* d_phase_clk;   // [32] profiling aid (MIX_PHASE_CLOCKS=1 at mix_create): globaltimer stamps of kernel phases, else null

  // optional outputs
  int* out_topk_idx;
  float* out_topk_val;
  int* out_n_active;
};

// Programmatic dependent launch.  The kernels of the SAE chain are short and strictly ordered, so
// what separates them is launch latency; launched this way, a kernel's CTAs may become resident
// while its predecessor in the stream still runs.  Contract inside such a kernel: pdl_wait() is its
// FIRST statement -- nothing the predecessor wrote is read before it, and no thread leaves without
// it (a grid that ended without waiting would let ITS successor run ahead of the predecessor) --
// followed by pdl_launch_dependents(), so that at most two kernels of the chain overlap.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Which launches use programmatic dependent launch: bit 0 unused (the pack step is part of the front kernel now), bit 1
// the full encode pass, bit 2 everything after it (tail, flagged-tile encode, flagged tail, edit-only kernels), bit 3
// the one-CTA-per-row probe / steering kernel of a context without weight sets.
// MIX_PDL_MASK in the environment overrides the default (A/B timing); read once.
enum { kPdlPack = 1, kPdlEncode = 2, kPdlTail = 4, kPdlHook = 8 };
int pdl_mask();

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(int which, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = (pdl_mask() & which) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

#ifdef __CUDACC__
// Profiling aid: thread `who` (a bool) stamps slot i of the phase-clock array: slots 0, 7, 8, 15 and 26.. (a kernel's
// first and last stamps; the encode kernel's) with the global nanosecond timer, the others with the SM's cycle counter -- cheap to
// read, and comparable between stamps of the same CTA.
__device__ __forceinline__ void phase_stamp(unsigned long long* clk, int i, bool who) {
  if (clk != nullptr && who) {
    unsigned long long t;
    if (i == 0 || i == 7 || i == 8 || i == 15 || i >= 26) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    else t = (unsigned long long)clock64();
    clk[i] = t;
  }
}

// Order-preserving 32-bit key of a float (larger value, larger key; -0 and +0 share one key; 0 is below every value).
__device__ __forceinline__ unsigned f2key(float f) {
  const unsigned b = __float_as_uint(f + 0.f);          // -0.0 -> +0.0: equal values, equal keys
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key2f(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
#endif

// kernel launchers (each returns the CUDA error of the launch)
cudaError_t launch_probe_steer(const Ctx* c, __nv_bfloat16* hidden, int T, float* scores, cudaStream_t s, bool allow_pdl);
// Multi-class probes of large batches have two kernels; both are launched and exactly one does the work, chosen
// on the device (mc_census_kernel lists the 128-row tiles that hold such rows and leaves the choice in
// d_mc_census): probe_tc (tcgen05, streams whole 128-row tiles of that list: batches whose listed tiles are at
// least half full of such rows) or probe_multiclass (mma.sync, 16-row tiles: rows scattered thinly).
cudaError_t launch_mc_census(const Ctx* c, int T, cudaStream_t s);
cudaError_t launch_probe_tc(const Ctx* c, const CUtensorMap& tmap_hidden, int T, float* scores, cudaStream_t s);
cudaError_t launch_probe_multiclass(const Ctx* c, const __nv_bfloat16* hidden, int T, float* scores, cudaStream_t s);
cudaError_t probe_tc_prepare();   // opt in to the large dynamic shared memory size
bool has_multiclass_stage(const Ctx* c);   // large batches with multi-class probes get a kernel of their own
bool has_tc_probe_stage(const Ctx* c);     // ... and, in contexts without SAE weight sets, the tensor-core kernel for dense batches
cudaError_t launch_router(const Ctx* c, float* logits, int n_experts, int T, cudaStream_t s);
// Routing + row pack in one launch.  cond/use_cond: graph-conditional handle the kernel sets to (SAE rows
// routed > 0); plain calls pass 0, 0
cudaError_t launch_front(const Ctx* c, const __nv_bfloat16* hidden, int T, cudaStream_t s, unsigned long long cond = 0,
                         int use_cond = 0);
int front_chunks(int T_max);       // chunks of token rows the front kernel classifies: sizes d_front_counts / d_front_sync
cudaError_t launch_encode_simt(const Ctx* c, cudaStream_t s);
cudaError_t launch_encode_tc(const Ctx* c, int mode, bool pair, cudaStream_t s);   // 0: all tiles; 1: flagged row tiles -> Z
bool encode_pair_possible(const Ctx* c);   // the CTA-pair encode kernel is part of this context's launch sequence
// Selection, edits, decode and write-back of every SAE row.  mode 0: behind the tensor-core encode (TopK from its
// candidates; rows it cannot settle are flagged); 1: behind the CUDA-core encode (TopK from Z); 2: the flagged
// rows, after their row tiles were re-encoded to Z (returns at once when nothing is flagged).
cudaError_t launch_tail(const Ctx* c, __nv_bfloat16* hidden, int mode, cudaStream_t s);
cudaError_t launch_edit_only(const Ctx* c, __nv_bfloat16* hidden, int T, cudaStream_t s);
cudaError_t launch_edit_only_delta(const Ctx* c, __nv_bfloat16* hidden, cudaStream_t s);   // decode_delta_kernel on the shortcut's token-indexed records
cudaError_t edit_only_prepare();   // opt in to the dynamic shared memory of the edit-only kernel
cudaError_t launch_compose_map(const Ctx* c, int T_live, int n_req, cudaStream_t s);
cudaError_t launch_fold_bias(const __nv_bfloat16* W_enc, const float* b_enc, const float* b_dec, float* b_eff,
                             long long d_sae, int d, cudaStream_t s);
cudaError_t launch_retile(const __nv_bfloat16* W_enc, __nv_bfloat16* W_tiled, long long d_sae, int d, cudaStream_t s);
cudaError_t launch_retile_fp8(const unsigned char* W_enc, unsigned char* W_tiled, long long d_sae, int d, int kb_bytes, cudaStream_t s);
cudaError_t encode_tc_prepare();   // opt in to the large dynamic shared memory size
// The encode has two kernels -- single CTAs on 128-row tiles, CTA pairs (tcgen05 cta_group::2) on 256-row tiles --
// and the front kernel decides per call, from the routing result, which of them works (the other returns at once).
// MIX_ENCODE_PAIR in the environment forces one: 0 single CTAs, 1 pairs; unset (or 2) = decided on the device.
constexpr int kEncodePairDefault = 2;
int encode_pair_mode(int set);     // returns the mode in force; set >= 0 changes it (A/B timing)

}  // namespace mix
