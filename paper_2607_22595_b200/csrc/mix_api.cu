// Host side of the C ABI declared in mix.h: context, device tables, registration, and the
// fixed launch sequence of mix_apply().
#include <cudaTypedefs.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

#include "mix_internal.h"

using namespace mix;

struct mix_ctx : public Ctx {};

namespace {

#define MIX_FAIL(ctx, code, ...)                          \
  do {                                                    \
    snprintf((ctx)->err, sizeof((ctx)->err), __VA_ARGS__); \
    return (code);                                        \
  } while (0)

#define MIX_CUDA(ctx, expr)                                                                  \
  do {                                                                                       \
    cudaError_t e_ = (expr);                                                                 \
    if (e_ != cudaSuccess) MIX_FAIL(ctx, MIX_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

__global__ void bench_add_from_table(const float* __restrict__ table, float* __restrict__ acc) {
  if (threadIdx.x == 0) acc[0] += table[0];
}
__global__ void bench_add_from_param(float v, float* __restrict__ acc) {
  if (threadIdx.x == 0) acc[0] += v;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

int load_encode_fn() {
  if (g_encode) return MIX_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return MIX_ERR_CUDA;
  g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  return MIX_OK;
}

// bf16 [rows, d] row-major; box = kTileK columns x box_rows rows; 128-byte swizzle.
// E4M3 codes [rows, width] row-major for the 8-bit contraction: box = 128 bytes x box_rows rows; 128-byte swizzle.
int make_tmap_e4m3(CUtensorMap* out, const void* base, unsigned long long rows, unsigned long long width, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)width, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)width};
  cuuint32_t box[2] = {(cuuint32_t)(2 * kTileK), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MIX_OK : MIX_ERR_CUDA;
}

int make_tmap(CUtensorMap* out, const void* base, unsigned long long rows, int d, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MIX_OK : MIX_ERR_CUDA;
}

template <typename T>
cudaError_t dev_alloc(T** p, size_t n) {
  *p = nullptr;
  if (n == 0) return cudaSuccess;
  return cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T));
}

void free_all(mix_ctx* c) {
  cudaFree(c->d_token_slot); cudaFree(c->d_n_live); cudaFree(c->d_apps); cudaFree(c->d_groups); cudaFree(c->d_gates); cudaFree(c->d_vec_arena); cudaFree(c->d_chain_next); cudaFree(c->d_row_meta); cudaFree(c->d_front_counts); cudaFree(c->d_front_sync); cudaFree(c->d_row_rec);
  cudaFree(c->d_edit_idx); cudaFree(c->d_edit_val); cudaFree(c->d_edit_mode); cudaFree(c->d_status);
  cudaFree(c->d_tmp_req); cudaFree(c->d_tmp_req_slot); cudaFree(c->d_panel); cudaFree(c->d_panel_row); cudaFree(c->d_act_scale); cudaFree(c->d_tau); cudaFree(c->d_tau_min); cudaFree(c->d_eo_row_delta); cudaFree(c->d_eo_coef);
  cudaFree(c->d_mtile_group); cudaFree(c->d_route); cudaFree(c->d_z);
  cudaFree(c->d_tmap_w); cudaFree(c->d_tmap_w_half); cudaFree(c->d_phase_clk); cudaFree(c->d_tmap_probe); cudaFree(c->d_mc_census); cudaFree(c->d_mc_tiles); cudaFree(c->d_cand_val); cudaFree(c->d_cand_idx);
  cudaFree(c->d_cand_ninth); cudaFree(c->d_row_flag); cudaFree(c->d_mtile_flag); cudaFree(c->d_n_flagged);
  if (c->owned_b_eff)
    for (int g = 0; g < c->cfg.n_groups_max; ++g) cudaFree(c->owned_b_eff[g]);
  if (c->owned_w_tiled)
    for (int g = 0; g < c->cfg.n_groups_max; ++g) cudaFree(c->owned_w_tiled[g]);
  free(c->owned_w_tiled);
  free(c->owned_b_eff); free(c->h_apps); free(c->h_groups); free(c->h_chain_next); free(c->h_edit_idx);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->side_stream) cudaStreamDestroy(c->side_stream);
  if (c->body_stream) cudaStreamDestroy(c->body_stream);
}

int check_slot(mix_ctx* c, int slot) {
  if (slot < 0 || slot >= c->cfg.n_slots_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "slot %d outside [0, %d)", slot, c->cfg.n_slots_max);
  return MIX_OK;
}

// Publish an app entry: body first with valid = 0, then the valid word.
// bias_src: device fp32 whose value goes into the entry's `alpha` word before the entry becomes valid (a one-class
// probe's bias in contexts whose hook kernel reads it from there), or null.
int publish_app(mix_ctx* c, int slot, cudaStream_t s, const float* bias_src = nullptr) {
  AppEntry tmp = c->h_apps[slot];
  const int valid = tmp.valid;
  tmp.valid = 0;
  MIX_CUDA(c, cudaMemcpyAsync(c->d_apps + slot, &tmp, sizeof(AppEntry), cudaMemcpyHostToDevice, s));
  if (bias_src) MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].alpha, bias_src, sizeof(float), cudaMemcpyDeviceToDevice, s));
  if (valid) MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].valid, &valid, sizeof(int), cudaMemcpyHostToDevice, s));
  return MIX_OK;
}

// Range and mode checks of an edit list against weight set `group`; changes nothing.
int check_edits(mix_ctx* c, int group, int n_edit, const int* idx, const float* val, const unsigned char* mode) {
  if (n_edit < 0 || n_edit > c->cfg.r_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "n_edit %d outside [0, r_max=%d]", n_edit, c->cfg.r_max);
  if (n_edit > 0 && (!idx || !val || !mode)) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "edit arrays are NULL");
  const long long S = c->h_groups[group].d_sae;
  for (int e = 0; e < n_edit; ++e) {
    if (idx[e] < 0 || idx[e] >= S) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "edit %d: feature %d outside [0, %lld)", e, idx[e], S);
    if (mode[e] != MIX_EDIT_CLAMP && mode[e] != MIX_EDIT_ABLATE) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "edit %d: bad mode %d", e, mode[e]);
  }
  return MIX_OK;
}

// Copies a checked edit list into the slot's rows of the device tables and into the host mirror of the
// indices (kept so that a weight set can be replaced only by one that still covers every edited feature).
int upload_edits(mix_ctx* c, int slot, int n_edit, const int* idx, const float* val, const unsigned char* mode, cudaStream_t s) {
  if (n_edit > 0) {
    const size_t off = (size_t)slot * c->cfg.r_max;
    memcpy(c->h_edit_idx + off, idx, n_edit * sizeof(int));
    MIX_CUDA(c, cudaMemcpyAsync(c->d_edit_idx + off, idx, n_edit * sizeof(int), cudaMemcpyHostToDevice, s));
    MIX_CUDA(c, cudaMemcpyAsync(c->d_edit_val + off, val, n_edit * sizeof(float), cudaMemcpyHostToDevice, s));
    MIX_CUDA(c, cudaMemcpyAsync(c->d_edit_mode + off, mode, n_edit, cudaMemcpyHostToDevice, s));
  }
  return MIX_OK;
}

// Walks every chain of the host tables and checks what mix_set_chain() promises: at most kMaxChain
// apps, only registered apps behind a link, an SAE app only at the end, no router app, and
// the probes' class columns inside C_max.  (A cycle shows up as a chain that is too long.)
int validate_chains(mix_ctx* c) {
  const int NS = c->cfg.n_slots_max;
  for (int s0 = 0; s0 < NS; ++s0) {
    if (!c->h_apps[s0].valid || c->h_chain_next[s0] < 0) continue;
    int len = 0, classes = 0;
    for (int cur = s0; cur >= 0; cur = c->h_chain_next[cur]) {
      if (len == kMaxChain) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "the chain through slot %d has a cycle or more than %d apps", s0, kMaxChain);
      const AppEntry& a = c->h_apps[cur];
      if (!a.valid) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "the chain from slot %d reaches slot %d, which has no app", s0, cur);
      const int kind = a.kind & kKindMask;
      if (kind == MIX_ROUTER) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "slot %d holds a router app: it cannot be part of a chain", cur);
      if (kind == MIX_SAE && c->h_chain_next[cur] >= 0) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "slot %d holds an SAE app: it can only end a chain", cur);
      if (kind == MIX_PROBE) classes += a.n_classes;
      ++len;
    }
    if (classes > c->cfg.C_max) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "the probes of the chain from slot %d write %d columns, C_max is %d", s0, classes, c->cfg.C_max);
  }
  return MIX_OK;
}

// Sets or clears the link of `slot` on the device: link first, then the flag in the app entry
// (when setting), the flag first (when clearing).
int upload_chain(mix_ctx* c, int slot, cudaStream_t s) {
  const int next = c->h_chain_next[slot];
  int kind = c->h_apps[slot].kind & ~kKindChained;
  if (next < 0) {
    c->h_apps[slot].kind = kind;
    if (c->h_apps[slot].valid) MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].kind, &c->h_apps[slot].kind, sizeof(int), cudaMemcpyHostToDevice, s));
    MIX_CUDA(c, cudaMemcpyAsync(c->d_chain_next + slot, c->h_chain_next + slot, sizeof(int), cudaMemcpyHostToDevice, s));
  } else {
    MIX_CUDA(c, cudaMemcpyAsync(c->d_chain_next + slot, c->h_chain_next + slot, sizeof(int), cudaMemcpyHostToDevice, s));
    c->h_apps[slot].kind = kind | kKindChained;
    MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].kind, &c->h_apps[slot].kind, sizeof(int), cudaMemcpyHostToDevice, s));
  }
  return MIX_OK;
}

}  // namespace

namespace mix {
static int g_pdl_mask = -1;        // -1: not yet read from the environment
int pdl_mask() {
  // default: not the full encode pass -- measured, its early-resident CTAs cost config 3 about 7 us
  if (g_pdl_mask < 0) g_pdl_mask = getenv("MIX_PDL_MASK") ? (atoi(getenv("MIX_PDL_MASK")) & 15) : (kPdlPack | kPdlEncode | kPdlTail | kPdlHook);
  return g_pdl_mask;
}
}  // namespace mix

extern "C" {

int mix_set_pdl_mask(int mask) {
  const int old = mix::pdl_mask();
  if (mask >= 0) mix::g_pdl_mask = mask & 15;
  return old;
}

int mix_create(mix_ctx** out, const mix_config* cfg) {
  if (!out || !cfg) return MIX_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->d_model <= 0 || cfg->T_max <= 0 || cfg->n_slots_max <= 0 || cfg->n_groups_max < 0 || cfg->C_max <= 0 ||
      cfg->k_max < 0 || cfg->r_max < 0 || cfg->d_sae_max < 0)
    return MIX_ERR_INVALID_ARG;
  if (cfg->d_model % 64 || cfg->d_model > 8192 || cfg->C_max > kMaxClasses || cfg->k_max > kMaxK ||
      cfg->r_max > kMaxEdits || cfg->n_groups_max > kMaxGroups || cfg->d_sae_max % kTileN ||
      cfg->d_sae_max > 0x7fffffffll || (cfg->n_groups_max > 0 && cfg->d_sae_max == 0))
    return MIX_ERR_UNSUPPORTED;
  {  // the routing kernel keeps (chunks of 256 rows) x (n_groups + 1) counters in shared memory
    const long long chunks = (cfg->T_max + 255) / 256;
    if (chunks * (cfg->n_groups_max + 1) * 4 > 40 * 1024) return MIX_ERR_UNSUPPORTED;
  }
  if ((cfg->flags & MIX_FLAG_SLOT_CHAINS) && (cfg->flags & MIX_FLAG_SAE_EDIT_ONLY)) return MIX_ERR_INVALID_ARG;
  if ((cfg->flags & MIX_FLAG_FP8_W_ENC) && (cfg->flags & (MIX_FLAG_ENCODE_SIMT | MIX_FLAG_SAE_EDIT_ONLY))) return MIX_ERR_INVALID_ARG;
  if ((cfg->flags & MIX_FLAG_FP8_ACT) && !(cfg->flags & MIX_FLAG_FP8_W_ENC)) return MIX_ERR_INVALID_ARG;
  if ((cfg->flags & MIX_FLAG_FP8_W_ENC) && cfg->d_model % (2 * kTileK)) return MIX_ERR_UNSUPPORTED;   // k-blocks of 128 codes
  mix_ctx* c = static_cast<mix_ctx*>(calloc(1, sizeof(mix_ctx)));
  if (!c) return MIX_ERR_NO_MEMORY;
  c->cfg = *cfg;
  if (c->cfg.r_max == 0) c->cfg.r_max = 1;      // keeps table strides non-zero
  if (c->cfg.k_max == 0) c->cfg.k_max = 1;
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, c->device);
  if (e != cudaSuccess) { free(c); return MIX_ERR_CUDA; }
  const int G = cfg->n_groups_max, NS = cfg->n_slots_max, T = cfg->T_max;
  c->h_apps = static_cast<AppEntry*>(calloc(NS, sizeof(AppEntry)));
  c->h_groups = static_cast<GroupEntry*>(calloc(G > 0 ? G : 1, sizeof(GroupEntry)));
  c->h_chain_next = static_cast<int*>(malloc(NS * sizeof(int)));
  c->h_edit_idx = static_cast<int*>(calloc((size_t)NS * c->cfg.r_max, sizeof(int)));
  if (c->h_chain_next) memset(c->h_chain_next, 0xff, NS * sizeof(int));
  c->owned_b_eff = static_cast<float**>(calloc(G > 0 ? G : 1, sizeof(float*)));
  c->owned_w_tiled = static_cast<__nv_bfloat16**>(calloc(G > 0 ? G : 1, sizeof(__nv_bfloat16*)));
  if (!c->h_apps || !c->h_groups || !c->h_chain_next || !c->h_edit_idx || !c->owned_b_eff || !c->owned_w_tiled) { free_all(c); free(c); return MIX_ERR_NO_MEMORY; }
  bool ok = true;
  ok = ok && dev_alloc(&c->d_token_slot, T) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_n_live, 1) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_apps, NS) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_groups, G > 0 ? G : 1) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_gates, NS) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_chain_next, NS) == cudaSuccess;
  if (T <= kTeamMaxRows) ok = ok && dev_alloc(&c->d_vec_arena, (size_t)NS * cfg->d_model) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_edit_idx, (size_t)NS * c->cfg.r_max) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_edit_val, (size_t)NS * c->cfg.r_max) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_edit_mode, (size_t)NS * c->cfg.r_max) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_status, 1) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_tmp_req, T) == cudaSuccess;
  ok = ok && dev_alloc(&c->d_tmp_req_slot, T) == cudaSuccess;
  if (ok && G > 0) {
    c->panel_rows_cap = ((T + kTileM - 1) / kTileM + G) * kTileM;
    const size_t P = c->panel_rows_cap;
    ok = ok && dev_alloc(&c->d_panel, P * cfg->d_model) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_panel_row, P) == cudaSuccess;
    if (cfg->flags & MIX_FLAG_FP8_W_ENC) ok = ok && dev_alloc(&c->d_act_scale, P) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_mtile_group, P / kTileM) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_row_meta, T) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_front_counts, (size_t)front_chunks(T) * (G + 1)) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_front_sync, 2) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_route, 1) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_z, P * (size_t)cfg->d_sae_max) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_tmap_w, G) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_tmap_w_half, G) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_row_rec, P) == cudaSuccess;
    if (getenv("MIX_PHASE_CLOCKS") && atoi(getenv("MIX_PHASE_CLOCKS")))
      ok = ok && dev_alloc(&c->d_phase_clk, 32) == cudaSuccess && cudaMemset(c->d_phase_clk, 0, 32 * sizeof(unsigned long long)) == cudaSuccess;
    if (cfg->flags & MIX_FLAG_SAE_EDIT_ONLY) {
      ok = ok && dev_alloc(&c->d_eo_row_delta, (size_t)T) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_eo_coef, (size_t)T * (size_t)(cfg->r_max > 0 ? cfg->r_max : 1)) == cudaSuccess;
    }
    if (!(cfg->flags & MIX_FLAG_ENCODE_SIMT)) {
      c->cand_tiles = (int)(cfg->d_sae_max / kTileN);
      const size_t nc = P * (size_t)c->cand_tiles;
      ok = ok && dev_alloc(&c->d_cand_val, nc * kCandPerTile) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_cand_idx, nc * kCandPerTile) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_cand_ninth, nc) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_row_flag, P) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_mtile_flag, P / kTileM) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_n_flagged, 1) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_tau, P * (size_t)kTauSlots) == cudaSuccess;
      ok = ok && dev_alloc(&c->d_tau_min, P) == cudaSuccess;
    }
  }
  if (!ok) { cudaGetLastError(); free_all(c); free(c); return MIX_ERR_NO_MEMORY; }
  e = cudaMemset(c->d_token_slot, 0xff, T * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->d_n_live, 0, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->d_apps, 0, NS * sizeof(AppEntry));
  if (e == cudaSuccess) e = cudaMemset(c->d_groups, 0, (G > 0 ? G : 1) * sizeof(GroupEntry));
  if (e == cudaSuccess) e = cudaMemset(c->d_gates, 0, NS * sizeof(GateEntry));
  if (e == cudaSuccess) e = cudaMemset(c->d_chain_next, 0xff, NS * sizeof(int));
  if (e == cudaSuccess && c->d_vec_arena) e = cudaMemset(c->d_vec_arena, 0, (size_t)NS * cfg->d_model * sizeof(__nv_bfloat16));
  if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, sizeof(unsigned));
  if (e == cudaSuccess && G > 0) {
    e = cudaMemset(c->d_panel, 0, (size_t)c->panel_rows_cap * cfg->d_model * sizeof(__nv_bfloat16));
    if (e == cudaSuccess) e = cudaMemset(c->d_route, 0, sizeof(RouteState));
    if (e == cudaSuccess) e = cudaMemset(c->d_front_sync, 0, 2 * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->d_panel_row, 0xff, c->panel_rows_cap * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->d_mtile_group, 0xff, c->panel_rows_cap / kTileM * sizeof(int));
    if (e == cudaSuccess && !(cfg->flags & MIX_FLAG_ENCODE_SIMT)) {
      if (load_encode_fn() != MIX_OK)
        e = cudaErrorUnknown;
      else if ((cfg->flags & MIX_FLAG_FP8_W_ENC)    // codes: P rows (8-bit input) or 2 P rows (hi, lo) in the same buffer
                   ? make_tmap_e4m3(&c->tmap_panel, c->d_panel, 2ull * c->panel_rows_cap, cfg->d_model, kTileM) != MIX_OK
                   : make_tmap(&c->tmap_panel, c->d_panel, c->panel_rows_cap, cfg->d_model, kTileM) != MIX_OK)
        e = cudaErrorUnknown;
      if (e == cudaSuccess && c->d_act_scale) e = cudaMemset(c->d_act_scale, 0, c->panel_rows_cap * sizeof(float));
      if (e == cudaSuccess) e = encode_tc_prepare();
    }
    if (e == cudaSuccess && (cfg->flags & MIX_FLAG_SAE_EDIT_ONLY)) {
      e = edit_only_prepare();
    }
  }
  if (e == cudaSuccess && has_tc_probe_stage(c)) {
    // large batches with multi-class probes: the tensor-core probe kernel needs a map per probe matrix
    if (dev_alloc(&c->d_tmap_probe, NS) != cudaSuccess || dev_alloc(&c->d_mc_census, 1) != cudaSuccess ||
        dev_alloc(&c->d_mc_tiles, (size_t)(T + kTileM - 1) / kTileM) != cudaSuccess) {
      cudaGetLastError(); free_all(c); free(c); return MIX_ERR_NO_MEMORY;
    }
    e = cudaMemset(c->d_mc_census, 0, sizeof(McCensus));
    if (load_encode_fn() != MIX_OK) e = cudaErrorUnknown;
    if (e == cudaSuccess) e = probe_tc_prepare();
  }
  if (e == cudaSuccess && (G > 0 || has_tc_probe_stage(c))) {
    e = cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->body_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { free_all(c); free(c); return MIX_ERR_CUDA; }
  c->err[0] = 0;
  *out = c;
  return MIX_OK;
}

int mix_destroy(mix_ctx* c) {
  if (!c) return MIX_OK;
  cudaDeviceSynchronize();
  free_all(c);
  free(c);
  return MIX_OK;
}

const char* mix_last_error(const mix_ctx* c) { return c ? c->err : "null context"; }

int mix_register_sae_weights(mix_ctx* c, int group, const mix_sae_weights* w, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (!w) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "weights are NULL");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (group < 0 || group >= c->cfg.n_groups_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "group %d outside [0, %d)", group, c->cfg.n_groups_max);
  if (w->d_sae <= 0 || w->d_sae > c->cfg.d_sae_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "d_sae %lld outside (0, %lld]", w->d_sae, c->cfg.d_sae_max);
  if (w->d_sae % kTileN) MIX_FAIL(c, MIX_ERR_UNSUPPORTED, "d_sae %lld is not a multiple of %d", w->d_sae, kTileN);
  if (w->act != MIX_SAE_RELU && w->act != MIX_SAE_JUMPRELU && w->act != MIX_SAE_TOPK) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "bad SAE activation %d", w->act);
  if (!w->W_enc || !w->b_enc || !w->W_dec) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "W_enc, b_enc and W_dec are required");
  if (!aligned16(w->W_enc) || !aligned16(w->W_dec) || !aligned16(w->b_enc) || (w->b_dec && !aligned16(w->b_dec)))
    MIX_FAIL(c, MIX_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
  if (w->act == MIX_SAE_JUMPRELU && !w->theta) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "JumpReLU needs theta");
  if (w->act == MIX_SAE_TOPK && (w->k < 1 || w->k > c->cfg.k_max || w->k > w->d_sae))
    MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "k %d outside [1, min(k_max=%d, d_sae)]", w->k, c->cfg.k_max);
  if (w->center_input && !w->b_dec) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "center_input needs b_dec");
  const bool fp8 = (c->cfg.flags & MIX_FLAG_FP8_W_ENC) != 0;
  if (fp8 && (!w->W_enc_scale || w->center_input))
    MIX_FAIL(c, MIX_ERR_INVALID_ARG, "an 8-bit encoder needs W_enc_scale and does not take center_input");
  // Replacing a weight set: the edit lists of the apps attached to it were range-checked against the old
  // d_sae and index W_enc / W_dec rows on the device, so the new set must still cover every edited feature.
  for (int sl = 0; sl < c->cfg.n_slots_max; ++sl) {
    const AppEntry& a = c->h_apps[sl];
    if (!a.valid || (a.kind & kKindMask) != MIX_SAE || a.group != group) continue;
    for (int e = 0; e < a.n_edit; ++e)
      if (c->h_edit_idx[(size_t)sl * c->cfg.r_max + e] >= w->d_sae)
        MIX_FAIL(c, MIX_ERR_INVALID_ARG, "slot %d edits feature %d of weight set %d: the new d_sae %lld does not cover it "
                 "(unregister the app or change its edits first)", sl, c->h_edit_idx[(size_t)sl * c->cfg.r_max + e], group, w->d_sae);
  }

  GroupEntry ge;
  memset(&ge, 0, sizeof(ge));
  ge.valid = 1;
  ge.act = w->act;
  ge.k = w->act == MIX_SAE_TOPK ? w->k : 0;
  ge.d_sae = w->d_sae;
  ge.W_enc = fp8 ? nullptr : static_cast<const __nv_bfloat16*>(w->W_enc);
  ge.w_scale = fp8 ? w->W_enc_scale : nullptr;
  ge.b_eff = w->b_enc;
  ge.theta = w->theta;
  ge.W_dec = static_cast<const __nv_bfloat16*>(w->W_dec);
  ge.b_dec = w->b_dec;
  if (w->center_input) {
    // z = W_enc (h - b_dec) + b_enc = W_enc h + (b_enc - W_enc b_dec): fold once, here
    if (c->owned_b_eff[group]) { cudaStreamSynchronize(s); cudaFree(c->owned_b_eff[group]); c->owned_b_eff[group] = nullptr; }
    if (cudaMalloc(reinterpret_cast<void**>(&c->owned_b_eff[group]), w->d_sae * sizeof(float)) != cudaSuccess) {
      cudaGetLastError();
      MIX_FAIL(c, MIX_ERR_NO_MEMORY, "cannot allocate the folded bias");
    }
    MIX_CUDA(c, launch_fold_bias(ge.W_enc, w->b_enc, w->b_dec, c->owned_b_eff[group], w->d_sae, c->cfg.d_model, s));
    ge.b_eff = c->owned_b_eff[group];
  }
  if (!(c->cfg.flags & MIX_FLAG_ENCODE_SIMT)) {
    CUtensorMap tm, tm_half;       // boxes of 256 features, and of 128 (one CTA's share when a CTA pair works on the tile)
    if (fp8) {
      // library-owned tile-ordered copy of the codes: [S/256][d/128][256][128] bytes, seen by TMA as a 128-byte-wide
      // matrix (128-byte swizzled boxes of 256 rows)
      if (c->owned_w_tiled[group]) { cudaStreamSynchronize(s); cudaFree(c->owned_w_tiled[group]); c->owned_w_tiled[group] = nullptr; }
      const size_t n_el = (size_t)w->d_sae * c->cfg.d_model;
      if (cudaMalloc(reinterpret_cast<void**>(&c->owned_w_tiled[group]), n_el) != cudaSuccess) {
        cudaGetLastError();
        MIX_FAIL(c, MIX_ERR_NO_MEMORY, "cannot allocate the tile-ordered copy of the 8-bit W_enc");
      }
      unsigned char* tiled = reinterpret_cast<unsigned char*>(c->owned_w_tiled[group]);
      MIX_CUDA(c, launch_retile_fp8(static_cast<const unsigned char*>(w->W_enc), tiled, w->d_sae, c->cfg.d_model, 2 * kTileK, s));
      if (make_tmap_e4m3(&tm, tiled, (unsigned long long)(n_el / (2 * kTileK)), 2 * kTileK, kTileN) != MIX_OK ||
          make_tmap_e4m3(&tm_half, tiled, (unsigned long long)(n_el / (2 * kTileK)), 2 * kTileK, kTileN / 2) != MIX_OK)
        MIX_FAIL(c, MIX_ERR_CUDA, "cuTensorMapEncodeTiled failed for the 8-bit W_enc");
    } else if (c->cfg.flags & MIX_FLAG_RETILE_W_ENC) {
      // library-owned tile-contiguous copy: [S/256][d/64][256][64], seen by TMA as a 64-column matrix
      if (c->owned_w_tiled[group]) { cudaStreamSynchronize(s); cudaFree(c->owned_w_tiled[group]); c->owned_w_tiled[group] = nullptr; }
      const size_t n_el = (size_t)w->d_sae * c->cfg.d_model;
      if (cudaMalloc(reinterpret_cast<void**>(&c->owned_w_tiled[group]), n_el * sizeof(__nv_bfloat16)) != cudaSuccess) {
        cudaGetLastError();
        MIX_FAIL(c, MIX_ERR_NO_MEMORY, "cannot allocate the re-tiled copy of W_enc");
      }
      MIX_CUDA(c, launch_retile(ge.W_enc, c->owned_w_tiled[group], w->d_sae, c->cfg.d_model, s));
      if (make_tmap(&tm, c->owned_w_tiled[group], (unsigned long long)(n_el / kTileK), kTileK, kTileN) != MIX_OK ||
          make_tmap(&tm_half, c->owned_w_tiled[group], (unsigned long long)(n_el / kTileK), kTileK, kTileN / 2) != MIX_OK)
        MIX_FAIL(c, MIX_ERR_CUDA, "cuTensorMapEncodeTiled failed for the re-tiled W_enc");
    } else if (make_tmap(&tm, w->W_enc, (unsigned long long)w->d_sae, c->cfg.d_model, kTileN) != MIX_OK ||
               make_tmap(&tm_half, w->W_enc, (unsigned long long)w->d_sae, c->cfg.d_model, kTileN / 2) != MIX_OK) {
      MIX_FAIL(c, MIX_ERR_CUDA, "cuTensorMapEncodeTiled failed for W_enc");
    }
    MIX_CUDA(c, cudaMemcpyAsync(c->d_tmap_w + group, &tm, sizeof(tm), cudaMemcpyHostToDevice, s));
    MIX_CUDA(c, cudaMemcpyAsync(c->d_tmap_w_half + group, &tm_half, sizeof(tm_half), cudaMemcpyHostToDevice, s));
  }
  c->h_groups[group] = ge;
  GroupEntry tmp = ge;
  tmp.valid = 0;
  MIX_CUDA(c, cudaMemcpyAsync(c->d_groups + group, &tmp, sizeof(tmp), cudaMemcpyHostToDevice, s));
  const int one = 1;
  MIX_CUDA(c, cudaMemcpyAsync(&c->d_groups[group].valid, &one, sizeof(int), cudaMemcpyHostToDevice, s));
  return MIX_OK;
}

int mix_unregister_sae_weights(mix_ctx* c, int group, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (group < 0 || group >= c->cfg.n_groups_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "group %d outside [0, %d)", group, c->cfg.n_groups_max);
  c->h_groups[group].valid = 0;
  const int zero = 0;
  MIX_CUDA(c, cudaMemcpyAsync(&c->d_groups[group].valid, &zero, sizeof(int), cudaMemcpyHostToDevice,
                              static_cast<cudaStream_t>(stream)));
  return MIX_OK;
}

int mix_register_app(mix_ctx* c, int slot, int kind, const void* desc, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (!desc) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "descriptor is NULL");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = check_slot(c, slot);
  if (rc != MIX_OK) return rc;
  AppEntry e;
  memset(&e, 0, sizeof(e));
  e.valid = 1;
  e.kind = kind;
  if (kind == MIX_PROBE) {
    const mix_probe* p = static_cast<const mix_probe*>(desc);
    if (p->n_classes < 1 || p->n_classes > c->cfg.C_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "n_classes %d outside [1, C_max=%d]", p->n_classes, c->cfg.C_max);
    if (p->act != MIX_ACT_SIGMOID && p->act != MIX_ACT_SOFTMAX && p->act != MIX_ACT_NONE) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "bad probe activation %d", p->act);
    if (p->act == MIX_ACT_SIGMOID && p->n_classes != 1) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "sigmoid probes have one class");
    if (!p->W || !aligned16(p->W)) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "probe W is NULL or not 16-byte aligned");
    e.n_classes = p->n_classes;
    e.act = p->act;
    e.W = p->W;
    e.b = p->b;
    if (c->d_tmap_probe && p->n_classes > 1 && p->n_classes <= 32) {
      // rows of the probe matrix beyond n_classes lie outside the tensor: TMA fills them with zeros
      CUtensorMap tm;
      if (make_tmap(&tm, p->W, (unsigned long long)p->n_classes, c->cfg.d_model, 32) != MIX_OK)
        MIX_FAIL(c, MIX_ERR_CUDA, "cuTensorMapEncodeTiled failed for the probe matrix of slot %d", slot);
      MIX_CUDA(c, cudaMemcpyAsync(c->d_tmap_probe + slot, &tm, sizeof(tm), cudaMemcpyHostToDevice, s));
    }
  } else if (kind == MIX_STEER) {
    const mix_steer* p = static_cast<const mix_steer*>(desc);
    if (!p->v || !aligned16(p->v)) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "steering vector is NULL or not 16-byte aligned");
    e.W = p->v;
    e.alpha = p->alpha;
  } else if (kind == MIX_PROJECT) {
    const mix_project* p = static_cast<const mix_project*>(desc);
    if (!p->r || !aligned16(p->r)) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "projection vector is NULL or not 16-byte aligned");
    e.W = p->r;
    e.alpha = p->beta;
  } else if (kind == MIX_ROUTER) {
    const mix_router* p = static_cast<const mix_router*>(desc);
    if (p->n_experts < 1) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "n_experts %d < 1", p->n_experts);
    if (!p->delta) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "router delta is NULL");
    e.n_classes = p->n_experts;
    e.W = p->delta;
  } else if (kind == MIX_SAE) {
    const mix_sae_app* p = static_cast<const mix_sae_app*>(desc);
    if (p->group < 0 || p->group >= c->cfg.n_groups_max || !c->h_groups[p->group].valid)
      MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "SAE weight set %d is not registered", p->group);
    rc = check_edits(c, p->group, p->n_edit, p->idx, p->val, p->mode);
    if (rc == MIX_OK) rc = upload_edits(c, slot, p->n_edit, p->idx, p->val, p->mode, s);
    if (rc != MIX_OK) return rc;
    e.group = p->group;
    e.n_edit = p->n_edit;
    e.add_error = p->add_error ? 1 : 0;
  } else {
    MIX_FAIL(c, MIX_ERR_INVALID_ARG, "bad app kind %d", kind);
  }
  // Single-vector weights are copied into the context's vector arena (row = slot), so that the
  // one-CTA-per-row kernel can request them from the slot id alone, before it has the entry.
  if (c->d_vec_arena && (kind == MIX_STEER || kind == MIX_PROJECT || (kind == MIX_PROBE && e.n_classes == 1))) {
    __nv_bfloat16* dst = c->d_vec_arena + (size_t)slot * c->cfg.d_model;
    MIX_CUDA(c, cudaMemcpyAsync(dst, e.W, (size_t)c->cfg.d_model * sizeof(__nv_bfloat16), cudaMemcpyDeviceToDevice, s));
    e.W = dst;
  }
  const AppEntry old = c->h_apps[slot];
  const int old_next = c->h_chain_next[slot];
  c->h_apps[slot] = e;
  c->h_chain_next[slot] = -1;                       // a new app starts without a successor
  if (c->cfg.flags & MIX_FLAG_SLOT_CHAINS) {
    rc = validate_chains(c);                        // chains that END in or pass through this slot must still fit
    if (rc != MIX_OK) {
      c->h_apps[slot] = old;
      c->h_chain_next[slot] = old_next;
      return rc;
    }
    if (old_next >= 0) MIX_CUDA(c, cudaMemcpyAsync(c->d_chain_next + slot, c->h_chain_next + slot, sizeof(int), cudaMemcpyHostToDevice, s));
  }
  // The bias of a one-class probe travels in the entry itself (its `alpha` word is otherwise unused): the
  // one-CTA-per-row kernel then has it with the entry instead of one dependent load later.
  const float* bias_src = (c->d_vec_arena && kind == MIX_PROBE && e.n_classes == 1) ? e.b : nullptr;
  return publish_app(c, slot, s, bias_src);
}

int mix_unregister_app(mix_ctx* c, int slot, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  int rc = check_slot(c, slot);
  if (rc != MIX_OK) return rc;
  memset(&c->h_apps[slot], 0, sizeof(AppEntry));
  const int zero = 0;
  MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].valid, &zero, sizeof(int), cudaMemcpyHostToDevice,
                              static_cast<cudaStream_t>(stream)));
  if (c->cfg.flags & MIX_FLAG_SLOT_CHAINS) {        // links from and to the slot go with it
    for (int p = 0; p < c->cfg.n_slots_max; ++p) {
      if (p != slot && c->h_chain_next[p] != slot) continue;
      if (c->h_chain_next[p] < 0) continue;
      c->h_chain_next[p] = -1;
      rc = upload_chain(c, p, static_cast<cudaStream_t>(stream));
      if (rc != MIX_OK) return rc;
    }
  }
  return MIX_OK;
}

int mix_set_chain(mix_ctx* c, int slot, int next_slot, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!(c->cfg.flags & MIX_FLAG_SLOT_CHAINS)) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "the context was created without MIX_FLAG_SLOT_CHAINS");
  int rc = check_slot(c, slot);
  if (rc != MIX_OK) return rc;
  if (next_slot < -1 || next_slot >= c->cfg.n_slots_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "next_slot %d outside [-1, %d)", next_slot, c->cfg.n_slots_max);
  if (!c->h_apps[slot].valid) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "slot %d has no app", slot);
  const int old_next = c->h_chain_next[slot];
  c->h_chain_next[slot] = next_slot;
  rc = validate_chains(c);
  if (rc != MIX_OK) {
    c->h_chain_next[slot] = old_next;
    return rc;
  }
  return upload_chain(c, slot, s);
}

int mix_set_gate(mix_ctx* c, int slot, const float* scores, int row_stride, int column, int cmp, float threshold,
                 void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = check_slot(c, slot);
  if (rc != MIX_OK) return rc;
  if (!c->h_apps[slot].valid) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "slot %d has no app to gate", slot);
  int kind = c->h_apps[slot].kind & ~kKindGated;
  if (!scores) {                      // remove: drop the flag first, the entry may then go stale
    c->h_apps[slot].kind = kind;
    MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].kind, &kind, sizeof(int), cudaMemcpyHostToDevice, s));
    return MIX_OK;
  }
  if (cmp != MIX_GATE_GE && cmp != MIX_GATE_LT) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "bad gate comparison %d", cmp);
  if (row_stride < 1 || column < 0 || column >= row_stride)
    MIX_FAIL(c, MIX_ERR_INVALID_ARG, "gate column %d outside [0, row_stride=%d)", column, row_stride);
  GateEntry g;
  memset(&g, 0, sizeof(g));
  g.scores = scores;
  g.stride = row_stride;
  g.col = column;
  g.cmp = cmp;
  g.thr = threshold;
  // replacing a live gate: close the flag, rewrite the entry, raise the flag again
  if (c->h_apps[slot].kind & kKindGated)
    MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].kind, &kind, sizeof(int), cudaMemcpyHostToDevice, s));
  MIX_CUDA(c, cudaMemcpyAsync(c->d_gates + slot, &g, sizeof(g), cudaMemcpyHostToDevice, s));
  kind |= kKindGated;
  c->h_apps[slot].kind = kind;
  MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].kind, &kind, sizeof(int), cudaMemcpyHostToDevice, s));
  return MIX_OK;
}

int mix_update_steer_alpha(mix_ctx* c, int slot, float alpha, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  int rc = check_slot(c, slot);
  if (rc != MIX_OK) return rc;
  const int kind_ = c->h_apps[slot].kind & kKindMask;
  if (!c->h_apps[slot].valid || (kind_ != MIX_STEER && kind_ != MIX_PROJECT))
    MIX_FAIL(c, MIX_ERR_INVALID_ARG, "slot %d is not a steering or projection app", slot);
  c->h_apps[slot].alpha = alpha;
  MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].alpha, &alpha, sizeof(float), cudaMemcpyHostToDevice,
                              static_cast<cudaStream_t>(stream)));
  return MIX_OK;
}

int mix_update_sae_edits(mix_ctx* c, int slot, int n_edit, const int* idx, const float* val,
                         const unsigned char* mode, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = check_slot(c, slot);
  if (rc != MIX_OK) return rc;
  if (!c->h_apps[slot].valid || (c->h_apps[slot].kind & kKindMask) != MIX_SAE) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "slot %d is not an SAE app", slot);
  // validate before anything is enqueued: a failed call changes nothing, on the host or on the device
  rc = check_edits(c, c->h_apps[slot].group, n_edit, idx, val, mode);
  if (rc != MIX_OK) return rc;
  // shrink first, grow last, so a concurrent reader never sees a count beyond valid entries
  const int old_n = c->h_apps[slot].n_edit;
  if (n_edit < old_n)
    MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].n_edit, &n_edit, sizeof(int), cudaMemcpyHostToDevice, s));
  rc = upload_edits(c, slot, n_edit, idx, val, mode, s);
  if (rc != MIX_OK) return rc;
  c->h_apps[slot].n_edit = n_edit;
  MIX_CUDA(c, cudaMemcpyAsync(&c->d_apps[slot].n_edit, &n_edit, sizeof(int), cudaMemcpyHostToDevice, s));
  return MIX_OK;
}

int mix_set_slot_map(mix_ctx* c, const int* token_slot, int T_live, int src_is_device, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (T_live < 0 || T_live > c->cfg.T_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "T_live %d outside [0, T_max=%d]", T_live, c->cfg.T_max);
  if (T_live > 0 && !token_slot) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "token_slot is NULL");
  if (T_live > 0)
    MIX_CUDA(c, cudaMemcpyAsync(c->d_token_slot, token_slot, (size_t)T_live * sizeof(int),
                                src_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, s));
  MIX_CUDA(c, cudaMemcpyAsync(c->d_n_live, &T_live, sizeof(int), cudaMemcpyHostToDevice, s));
  return MIX_OK;
}

int mix_set_request_map(mix_ctx* c, const int* token_req, int T_live, const int* req_slot, int n_req,
                        int src_is_device, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (T_live < 0 || T_live > c->cfg.T_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "T_live %d outside [0, T_max=%d]", T_live, c->cfg.T_max);
  if (n_req < 0 || n_req > c->cfg.T_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "n_req %d outside [0, T_max=%d]", n_req, c->cfg.T_max);
  if (T_live > 0 && (!token_req || (n_req > 0 && !req_slot))) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "map arrays are NULL");
  const cudaMemcpyKind kind = src_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  if (T_live > 0) {
    MIX_CUDA(c, cudaMemcpyAsync(c->d_tmp_req, token_req, (size_t)T_live * sizeof(int), kind, s));
    if (n_req > 0) MIX_CUDA(c, cudaMemcpyAsync(c->d_tmp_req_slot, req_slot, (size_t)n_req * sizeof(int), kind, s));
    MIX_CUDA(c, launch_compose_map(c, T_live, n_req, s));
    c->map_from_kernel = 1;
  }
  MIX_CUDA(c, cudaMemcpyAsync(c->d_n_live, &T_live, sizeof(int), cudaMemcpyHostToDevice, s));
  return MIX_OK;
}

int mix_set_feature_out(mix_ctx* c, int* topk_idx, float* topk_val, int* n_active) {
  if (!c) return MIX_ERR_INVALID_ARG;
  c->out_topk_idx = topk_idx;
  c->out_topk_val = topk_val;
  c->out_n_active = n_active;
  return MIX_OK;
}

extern "C++" {
namespace {

// The SAE chain behind the front kernel: encode ... write-back.  `tap` records a stage event after each launch.
template <class Tap>
int sae_chain(mix_ctx* c, __nv_bfloat16* h, cudaStream_t s, Tap&& tap) {
  if (c->cfg.flags & MIX_FLAG_ENCODE_SIMT) {
    MIX_CUDA(c, launch_encode_simt(c, s));
    MIX_CUDA(c, tap());
    MIX_CUDA(c, launch_tail(c, h, 1, s));        // TopK from Z, edits, decode
    MIX_CUDA(c, tap());
  } else {
    // TopK sets -> candidates, other sets -> Z.  Two kernels, of which the one the front kernel chose for this
    // call does the work: single CTAs on 128-row tiles, CTA pairs on 256-row tiles (contexts of more than 128 rows)
    if (encode_pair_mode(-1) != 1 || c->cfg.T_max <= kTileM) MIX_CUDA(c, launch_encode_tc(c, 0, false, s));
    MIX_CUDA(c, tap());
    if (encode_pair_possible(c)) MIX_CUDA(c, launch_encode_tc(c, 0, true, s));
    MIX_CUDA(c, tap());
    MIX_CUDA(c, launch_tail(c, h, 0, s));        // exact TopK from candidates (or a flag), edits, decode
    MIX_CUDA(c, tap());
    MIX_CUDA(c, launch_encode_tc(c, 1, false, s));   // flagged row tiles -> Z (returns at once if none)
    MIX_CUDA(c, tap());
    MIX_CUDA(c, launch_tail(c, h, 2, s));        // the flagged rows (returns at once if none)
    MIX_CUDA(c, tap());
  }
  return MIX_OK;
}

// Puts the SAE chain into the body of an IF node of the graph that `s` is capturing; the node
// depends on whatever `s` has captured so far (the route kernel, which sets the condition), and
// the capture continues after it.
int sae_chain_conditional(mix_ctx* c, __nv_bfloat16* h, cudaStream_t s, cudaGraph_t graph,
                          cudaGraphConditionalHandle handle) {
  cudaStreamCaptureStatus st;
  const cudaGraphNode_t* deps = nullptr;
  size_t n_deps = 0;
  MIX_CUDA(c, cudaStreamGetCaptureInfo_v2(s, &st, nullptr, nullptr, &deps, &n_deps));
  cudaGraphNodeParams np = {cudaGraphNodeTypeConditional};   // zero-initialises the rest
  np.conditional.handle = handle;
  np.conditional.type = cudaGraphCondTypeIf;
  np.conditional.size = 1;
  cudaGraphNode_t node;
  MIX_CUDA(c, cudaGraphAddNode(&node, graph, deps, n_deps, &np));
  cudaGraph_t body = np.conditional.phGraph_out[0];
  MIX_CUDA(c, cudaStreamBeginCaptureToGraph(c->body_stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed));
  const int rc = sae_chain(c, h, c->body_stream, [] { return cudaSuccess; });
  cudaGraph_t ended = nullptr;
  const cudaError_t e_end = cudaStreamEndCapture(c->body_stream, &ended);
  if (rc != MIX_OK) return rc;
  MIX_CUDA(c, e_end);
  MIX_CUDA(c, cudaStreamUpdateCaptureDependencies(s, &node, 1, cudaStreamSetCaptureDependencies));
  return MIX_OK;
}

int apply_impl(mix_ctx* c, void* hidden, int T, float* scores_out, void* stream, bool conditional) {
  if (!c) return MIX_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!hidden || !aligned16(hidden)) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "hidden is NULL or not 16-byte aligned");
  if (T < 0 || T > c->cfg.T_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "T %d outside [0, T_max=%d]", T, c->cfg.T_max);
  __nv_bfloat16* h = static_cast<__nv_bfloat16*>(hidden);
  cudaGraph_t graph = nullptr;
  cudaGraphConditionalHandle handle = 0;
  conditional = conditional && c->cfg.n_groups_max > 0;     // without weight sets there is no SAE chain to skip
  if (conditional) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    MIX_CUDA(c, cudaStreamGetCaptureInfo_v2(s, &st, nullptr, &graph, nullptr, nullptr));
    if (st != cudaStreamCaptureStatusActive || !graph)
      MIX_FAIL(c, MIX_ERR_INVALID_ARG, "mix_apply_conditional needs a stream that is being captured (status %d)", (int)st);
    if (c->stage_events_on) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "stage events cannot be recorded inside a conditional body");
    MIX_CUDA(c, cudaGraphConditionalHandleCreate(&handle, graph, 0, cudaGraphCondAssignDefault));
  }
  int stage = 0;
  auto tap = [&]() -> cudaError_t {
    return c->stage_events_on ? cudaEventRecord(c->stage_events[stage++], s) : cudaSuccess;
  };
  // Probes and steering touch rows the SAE path never touches, so when both are present they
  // run side by side: the probe/steer kernels on the context's side stream (forked from and
  // joined back into the caller's stream with events, which stream capture turns into graph
  // edges), the SAE chain on the caller's stream.  With the timing taps on, everything runs in
  // order on the caller's stream so that the per-stage times mean something.
  const bool fork = c->cfg.n_groups_max > 0 && !c->stage_events_on;
  cudaStream_t ps = fork ? c->side_stream : s;
  if (fork) {
    MIX_CUDA(c, cudaEventRecord(c->ev_fork, s));
    MIX_CUDA(c, cudaStreamWaitEvent(ps, c->ev_fork, 0));
  }
  MIX_CUDA(c, tap());
  // Multi-class probes of a large batch have two kernels of which exactly one does the work: the 16-row
  // kernel takes batches sparse in such rows (and every batch of a context with SAE weight sets), the
  // tensor-core kernel dense ones.  Where both exist, a one-CTA kernel makes the choice first and the
  // tensor-core kernel -- whose rows no other kernel of this call touches -- runs on the context's side
  // stream, beside the streaming kernel's pass over the batch.
  const bool tc = has_tc_probe_stage(c);
  const bool tc_fork = tc && !c->stage_events_on;
  CUtensorMap tm_hidden;                         // host-side encoding only: no device work, fine under capture
  if (tc) {
    if (make_tmap(&tm_hidden, h, (unsigned long long)c->cfg.T_max, c->cfg.d_model, kTileM) != MIX_OK)
      MIX_FAIL(c, MIX_ERR_CUDA, "cuTensorMapEncodeTiled failed for hidden");
    MIX_CUDA(c, launch_mc_census(c, T, ps));
    MIX_CUDA(c, tap());
    if (tc_fork) {
      MIX_CUDA(c, cudaEventRecord(c->ev_fork, ps));
      MIX_CUDA(c, cudaStreamWaitEvent(c->side_stream, c->ev_fork, 0));
      MIX_CUDA(c, launch_probe_tc(c, tm_hidden, T, scores_out, c->side_stream));
      MIX_CUDA(c, cudaEventRecord(c->ev_join, c->side_stream));
    }
  }
  // (programmatic launch only where this kernel directly follows the caller's work in the caller's stream)
  const bool hook_pdl = !fork && !tc && !c->stage_events_on && !c->map_from_kernel;
  c->map_from_kernel = 0;
  MIX_CUDA(c, launch_probe_steer(c, h, T, scores_out, ps, hook_pdl));
  MIX_CUDA(c, tap());
  if (has_multiclass_stage(c)) {
    MIX_CUDA(c, launch_probe_multiclass(c, h, T, scores_out, ps));
    MIX_CUDA(c, tap());
  }
  if (tc && !tc_fork) {
    MIX_CUDA(c, launch_probe_tc(c, tm_hidden, T, scores_out, ps));
    MIX_CUDA(c, tap());
  }
  if (tc_fork) MIX_CUDA(c, cudaStreamWaitEvent(ps, c->ev_join, 0));
  if (fork) MIX_CUDA(c, cudaEventRecord(c->ev_join, ps));
  if (c->cfg.n_groups_max > 0) {
    // with slot chains a steering app may precede an SAE app on the same row: the SAE chain reads
    // the hidden state (first in the front kernel's row pack) only after the probe / steering kernel is done
    if (fork && (c->cfg.flags & MIX_FLAG_SLOT_CHAINS)) MIX_CUDA(c, cudaStreamWaitEvent(s, c->ev_join, 0));
    MIX_CUDA(c, launch_front(c, h, T, s, handle, conditional ? 1 : 0));   // routing + row pack
    MIX_CUDA(c, tap());
    const int rc = conditional ? sae_chain_conditional(c, h, s, graph, handle) : sae_chain(c, h, s, tap);
    if (rc != MIX_OK) return rc;
    if (c->cfg.flags & MIX_FLAG_SAE_EDIT_ONLY) {
      MIX_CUDA(c, launch_edit_only(c, h, T, s));
      MIX_CUDA(c, tap());
      MIX_CUDA(c, launch_edit_only_delta(c, h, s));
      MIX_CUDA(c, tap());
    }
  }
  if (fork) MIX_CUDA(c, cudaStreamWaitEvent(s, c->ev_join, 0));
  return MIX_OK;
}

}  // namespace
}  // extern "C++"

int mix_apply(mix_ctx* c, void* hidden, int T, float* scores_out, void* stream) {
  return apply_impl(c, hidden, T, scores_out, stream, false);
}

int mix_apply_conditional(mix_ctx* c, void* hidden, int T, float* scores_out, void* stream) {
  return apply_impl(c, hidden, T, scores_out, stream, true);
}

int mix_apply_router(mix_ctx* c, float* logits, int n_experts, int T, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (!logits || n_experts < 1) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "logits is NULL or n_experts < 1");
  if (T < 0 || T > c->cfg.T_max) MIX_FAIL(c, MIX_ERR_OUT_OF_RANGE, "T %d outside [0, T_max=%d]", T, c->cfg.T_max);
  MIX_CUDA(c, launch_router(c, logits, n_experts, T, static_cast<cudaStream_t>(stream)));
  return MIX_OK;
}

int mix_launches_per_apply(const mix_ctx* c) {
  if (!c) return 0;
  const int front = 1 + (has_multiclass_stage(c) ? 1 : 0) + (has_tc_probe_stage(c) ? 2 : 0);
  if (c->cfg.n_groups_max == 0) return front;
  return front + ((c->cfg.flags & MIX_FLAG_ENCODE_SIMT) ? 3 : 6) + ((c->cfg.flags & MIX_FLAG_SAE_EDIT_ONLY) ? 2 : 0);   // coefficient kernel + delta kernel
}

int mix_get_status(mix_ctx* c, unsigned* bits, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (!bits) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "bits is NULL");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  MIX_CUDA(c, cudaMemcpyAsync(bits, c->d_status, sizeof(unsigned), cudaMemcpyDeviceToHost, s));
  MIX_CUDA(c, cudaMemsetAsync(c->d_status, 0, sizeof(unsigned), s));
  MIX_CUDA(c, cudaStreamSynchronize(s));
  return MIX_OK;
}

int mix_set_stage_events(mix_ctx* c, void* const* events) {
  if (!c) return MIX_ERR_INVALID_ARG;
  c->stage_events_on = 0;
  if (events) {
    const int n = mix_launches_per_apply(c) + 1;
    for (int i = 0; i < n; ++i) {
      if (!events[i]) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "stage event %d is NULL", i);
      c->stage_events[i] = static_cast<cudaEvent_t>(events[i]);
    }
    c->stage_events_on = 1;
  }
  return MIX_OK;
}

int mix_bench_param_update(mix_ctx* c, int iters, float* us_table, float* us_node, void* stream) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (!us_table || !us_node || iters < 1) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "NULL output or iters < 1");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* d = nullptr;                                   // d[0]: table entry / unused, d[1]: accumulator
  MIX_CUDA(c, cudaMalloc(reinterpret_cast<void**>(&d), 2 * sizeof(float)));
  cudaGraph_t graph[2] = {nullptr, nullptr};
  cudaGraphExec_t exec[2] = {nullptr, nullptr};
  cudaGraphNode_t node[2];
  float sums[2] = {0.f, 0.f};
  double us[2] = {0.0, 0.0};
  cudaError_t e = cudaSuccess;
  for (int v = 0; v < 2 && e == cudaSuccess; ++v) {
    const float* table = d;
    float* acc = d + 1;
    float value = 0.f;
    void* args_table[2] = {&table, &acc};
    void* args_param[2] = {&value, &acc};
    cudaKernelNodeParams kp;
    memset(&kp, 0, sizeof(kp));
    kp.func = v == 0 ? reinterpret_cast<void*>(bench_add_from_table) : reinterpret_cast<void*>(bench_add_from_param);
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(32);
    kp.kernelParams = v == 0 ? args_table : args_param;
    e = cudaGraphCreate(&graph[v], 0);
    if (e == cudaSuccess) e = cudaGraphAddKernelNode(&node[v], graph[v], nullptr, 0, &kp);
    if (e == cudaSuccess) e = cudaGraphInstantiate(&exec[v], graph[v], 0);
    if (e == cudaSuccess) e = cudaMemsetAsync(d, 0, 2 * sizeof(float), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) break;
    timespec t0, t1;
    clock_gettime(CLOCK_MONOTONIC, &t0);
    for (int i = 0; i < iters && e == cudaSuccess; ++i) {
      value = (float)(i % 7);                           // small integers: the sums are exact in fp32
      if (v == 0) {
        e = cudaMemcpyAsync(d, &value, sizeof(float), cudaMemcpyHostToDevice, s);   // pageable source: staged at once
      } else {
        e = cudaGraphExecKernelNodeSetParams(exec[v], node[v], &kp);
      }
      if (e == cudaSuccess) e = cudaGraphLaunch(exec[v], s);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    clock_gettime(CLOCK_MONOTONIC, &t1);
    us[v] = ((t1.tv_sec - t0.tv_sec) * 1e9 + (t1.tv_nsec - t0.tv_nsec)) / 1e3 / iters;
    if (e == cudaSuccess) e = cudaMemcpy(&sums[v], d + 1, sizeof(float), cudaMemcpyDeviceToHost);
  }
  for (int v = 0; v < 2; ++v) {
    if (exec[v]) cudaGraphExecDestroy(exec[v]);
    if (graph[v]) cudaGraphDestroy(graph[v]);
  }
  cudaFree(d);
  MIX_CUDA(c, e);
  if (sums[0] != sums[1]) MIX_FAIL(c, MIX_ERR_CUDA, "the two mechanisms disagree: %g vs %g", (double)sums[0], (double)sums[1]);
  *us_table = (float)us[0];
  *us_node = (float)us[1];
  return MIX_OK;
}

int mix_debug_phase_clocks(mix_ctx* c, unsigned long long* out32) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (!out32) MIX_FAIL(c, MIX_ERR_INVALID_ARG, "out32 is NULL");
  memset(out32, 0, 32 * sizeof(unsigned long long));
  if (c->d_phase_clk) MIX_CUDA(c, cudaMemcpy(out32, c->d_phase_clk, 32 * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  return MIX_OK;
}

int mix_debug_workspace(mix_ctx* c, const int** panel_rows, const float** z, long long* ld_z, int* n_panel_rows) {
  if (!c) return MIX_ERR_INVALID_ARG;
  if (panel_rows) *panel_rows = c->d_panel_row;
  if (z) *z = c->d_z;
  if (ld_z) *ld_z = c->cfg.d_sae_max;
  if (n_panel_rows) *n_panel_rows = c->panel_rows_cap;
  return MIX_OK;
}

}  // extern "C"
