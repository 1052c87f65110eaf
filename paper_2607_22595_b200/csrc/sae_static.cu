// mix_sae_apply_static(): the SAE function of the hook for callers that must not allocate.
//
// Everything mix_create() would cudaMalloc for the SAE path (slot map, app / weight-set
// tables, edit lists, routing state, the packed bf16 panel and the fp32 pre-activation
// scratch) lives here in ONE file-scope device array of fixed size.  The array is
// part of the library image: every GPU that loads libmix.so holds it until the process exits.
// The call then runs the same routing / pack, encode (CUDA-core kernel) and selection / decode
// kernels as mix_apply(), pointed at that array.
#include <stdio.h>
#include <string.h>

#include "mix_internal.h"

using namespace mix;

namespace {

constexpr int kStaticRows = MIX_STATIC_MAX_ROWS;        // one 128-row tile
constexpr int kStaticD = MIX_STATIC_MAX_D_MODEL;
constexpr long long kStaticDsae = MIX_STATIC_MAX_D_SAE;
constexpr int kStaticK = MIX_STATIC_MAX_K;
static_assert(kStaticRows == kTileM, "the static panel is exactly one row tile");

constexpr size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// byte offsets inside the scratch array (each 256-byte aligned)
constexpr size_t kOffTokenSlot = 0;
constexpr size_t kOffNLive = kOffTokenSlot + align256(kStaticRows * sizeof(int));
constexpr size_t kOffStatus = kOffNLive + 256;
constexpr size_t kOffApp = kOffStatus + 256;
constexpr size_t kOffGate = kOffApp + align256(sizeof(AppEntry));
constexpr size_t kOffGroup = kOffGate + align256(sizeof(GateEntry));
constexpr size_t kOffEditIdx = kOffGroup + align256(sizeof(GroupEntry));
constexpr size_t kOffEditVal = kOffEditIdx + align256(kMaxEdits * sizeof(int));
constexpr size_t kOffEditMode = kOffEditVal + align256(kMaxEdits * sizeof(float));
constexpr size_t kOffRoute = kOffEditMode + align256(kMaxEdits);
constexpr size_t kOffPanelRow = kOffRoute + align256(sizeof(RouteState));
constexpr size_t kOffMtileGroup = kOffPanelRow + align256(kStaticRows * sizeof(int));
constexpr size_t kOffRowMeta = kOffMtileGroup + 256;
constexpr size_t kOffFrontCounts = kOffRowMeta + align256(kStaticRows * sizeof(int2));
constexpr size_t kOffFrontSync = kOffFrontCounts + 256;      // one chunk: a count per weight set + one, then epoch words
constexpr size_t kOffChainNext = kOffFrontSync + 256;
constexpr size_t kOffRowRec = kOffChainNext + 256;
constexpr size_t kOffPanel = kOffRowRec + align256(kStaticRows * sizeof(RowRec));
constexpr size_t kOffZ = kOffPanel + align256((size_t)kStaticRows * kStaticD * sizeof(__nv_bfloat16));
constexpr size_t kScratchBytes = kOffZ + align256((size_t)kStaticRows * kStaticDsae * sizeof(float));
static_assert(kScratchBytes < (6u << 20), "the header promises less than 6 MiB");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress();
// it is NOT a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices];     // device address of the array, per device, once resolved

// Everything the call's tables need, passed to the set-up kernel BY VALUE (well under the 4 KiB of kernel
// parameters): no host pointer is handed to the stream, so nothing the stream does later depends on the
// caller's stack or on the caller's edit arrays staying alive.
struct StaticSetup {
  int n_rows;
  int n_edit;
  AppEntry app;
  GroupEntry group;
  int edit_idx[kMaxEdits];
  float edit_val[kMaxEdits];
  unsigned char edit_mode[kMaxEdits];
};

// Rewrites every table of the scratch array that this call's kernels read before writing.
__global__ void __launch_bounds__(128)
static_setup_kernel(const StaticSetup su, int* __restrict__ token_slot, int* __restrict__ n_live,
                    unsigned* __restrict__ status, AppEntry* __restrict__ app, GroupEntry* __restrict__ group,
                    int* __restrict__ edit_idx, float* __restrict__ edit_val, unsigned char* __restrict__ edit_mode) {
  const int tid = threadIdx.x;
  if (tid < su.n_rows) token_slot[tid] = 0;             // every row -> slot 0 (n_rows <= 128 = blockDim.x)
  if (tid < su.n_edit) {
    edit_idx[tid] = su.edit_idx[tid];
    edit_val[tid] = su.edit_val[tid];
    edit_mode[tid] = su.edit_mode[tid];
  }
  if (tid == 0) {
    *n_live = su.n_rows;
    *status = 0u;
    *app = su.app;
    *group = su.group;
  }
}
static_assert(kStaticRows <= 128 && kMaxEdits <= 128, "one thread per row / per edit entry in the set-up kernel");

int fail(char* errbuf, int errbuf_len, int code, const char* fmt, long long a = 0, long long b = 0) {
  if (errbuf && errbuf_len > 0) snprintf(errbuf, (size_t)errbuf_len, fmt, a, b);
  return code;
}

}  // namespace

extern "C" int mix_sae_apply_static(void* hidden, int n_rows, int d_model, const mix_sae_weights* w,
                                    const mix_sae_app* app, int* topk_idx, float* topk_val, void* stream,
                                    char* errbuf, int errbuf_len) {
  if (!hidden || !w || !app) return fail(errbuf, errbuf_len, MIX_ERR_INVALID_ARG, "hidden, weights and app are required");
  if (n_rows < 0 || n_rows > kStaticRows)
    return fail(errbuf, errbuf_len, MIX_ERR_OUT_OF_RANGE, "n_rows %lld exceeds the static limit of %lld rows", n_rows, kStaticRows);
  if (d_model <= 0 || d_model > kStaticD)
    return fail(errbuf, errbuf_len, MIX_ERR_OUT_OF_RANGE, "d_model %lld exceeds the static limit of %lld", d_model, kStaticD);
  if (d_model % 64) return fail(errbuf, errbuf_len, MIX_ERR_UNSUPPORTED, "d_model %lld is not a multiple of 64", d_model);
  if (w->d_sae <= 0 || w->d_sae > kStaticDsae)
    return fail(errbuf, errbuf_len, MIX_ERR_OUT_OF_RANGE, "d_sae %lld exceeds the static limit of %lld", w->d_sae, kStaticDsae);
  if (w->d_sae % kTileN) return fail(errbuf, errbuf_len, MIX_ERR_UNSUPPORTED, "d_sae %lld is not a multiple of %lld", w->d_sae, kTileN);
  if (w->act != MIX_SAE_RELU && w->act != MIX_SAE_JUMPRELU && w->act != MIX_SAE_TOPK)
    return fail(errbuf, errbuf_len, MIX_ERR_INVALID_ARG, "bad SAE activation %lld", w->act);
  if (w->act == MIX_SAE_TOPK && (w->k < 1 || w->k > kStaticK || w->k > w->d_sae))
    return fail(errbuf, errbuf_len, MIX_ERR_OUT_OF_RANGE, "k %lld outside [1, %lld]", w->k, kStaticK);
  if (!w->W_enc || !w->b_enc || !w->W_dec || (w->act == MIX_SAE_JUMPRELU && !w->theta))
    return fail(errbuf, errbuf_len, MIX_ERR_INVALID_ARG, "W_enc, b_enc, W_dec (and theta for JumpReLU) are required");
  if (w->center_input)
    return fail(errbuf, errbuf_len, MIX_ERR_UNSUPPORTED, "input centring needs a folded bias, which would have to be allocated");
  if (app->n_edit < 0 || app->n_edit > kMaxEdits)
    return fail(errbuf, errbuf_len, MIX_ERR_OUT_OF_RANGE, "n_edit %lld exceeds the limit of %lld", app->n_edit, kMaxEdits);
  if (app->n_edit > 0 && (!app->idx || !app->val || !app->mode))
    return fail(errbuf, errbuf_len, MIX_ERR_INVALID_ARG, "edit arrays are NULL");
  for (int e = 0; e < app->n_edit; ++e) {
    if (app->idx[e] < 0 || app->idx[e] >= w->d_sae)
      return fail(errbuf, errbuf_len, MIX_ERR_OUT_OF_RANGE, "edit %lld names feature %lld outside the SAE", e, app->idx[e]);
    if (app->mode[e] != MIX_EDIT_CLAMP && app->mode[e] != MIX_EDIT_ABLATE)
      return fail(errbuf, errbuf_len, MIX_ERR_INVALID_ARG, "edit %lld has bad mode %lld", e, app->mode[e]);
  }
  const uintptr_t align_or = (uintptr_t)hidden | (uintptr_t)w->W_enc | (uintptr_t)w->W_dec;
  if (align_or & 15u) return fail(errbuf, errbuf_len, MIX_ERR_INVALID_ARG, "hidden, W_enc and W_dec must be 16-byte aligned");
  if (n_rows == 0) return MIX_OK;

  // Set-up, once per device, with that device current: resolve the device address of the
  // scratch array.  (Passing the symbol itself to a kernel would hand it a host-side stand-in.)
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fail(errbuf, errbuf_len, MIX_ERR_CUDA, "cannot identify the current device");
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) return fail(errbuf, errbuf_len, MIX_ERR_CUDA, "cudaGetSymbolAddress failed (%lld)", (long long)e);
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  unsigned char* base = g_scratch_addr[dev];
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // A context that owns nothing: every pointer aims into the static array.
  Ctx c;
  memset(&c, 0, sizeof(c));
  c.cfg.d_model = d_model;
  c.cfg.T_max = n_rows;
  c.cfg.n_slots_max = 1;
  c.cfg.n_groups_max = 1;
  c.cfg.C_max = 1;
  c.cfg.k_max = w->act == MIX_SAE_TOPK ? w->k : 1;
  c.cfg.r_max = kMaxEdits;
  c.cfg.d_sae_max = w->d_sae;
  c.cfg.flags = MIX_FLAG_ENCODE_SIMT;
  c.device = dev;
  c.d_token_slot = reinterpret_cast<int*>(base + kOffTokenSlot);
  c.d_n_live = reinterpret_cast<int*>(base + kOffNLive);
  c.d_status = reinterpret_cast<unsigned*>(base + kOffStatus);
  c.d_apps = reinterpret_cast<AppEntry*>(base + kOffApp);
  c.d_gates = reinterpret_cast<GateEntry*>(base + kOffGate);     // never read: the app entry carries no gate flag
  c.d_groups = reinterpret_cast<GroupEntry*>(base + kOffGroup);
  c.d_edit_idx = reinterpret_cast<int*>(base + kOffEditIdx);
  c.d_edit_val = reinterpret_cast<float*>(base + kOffEditVal);
  c.d_edit_mode = base + kOffEditMode;
  c.d_route = reinterpret_cast<RouteState*>(base + kOffRoute);
  c.d_panel_row = reinterpret_cast<int*>(base + kOffPanelRow);
  c.d_mtile_group = reinterpret_cast<int*>(base + kOffMtileGroup);
  c.d_row_meta = reinterpret_cast<int2*>(base + kOffRowMeta);
  c.d_front_counts = reinterpret_cast<int*>(base + kOffFrontCounts);
  c.d_front_sync = reinterpret_cast<int*>(base + kOffFrontSync);   // two counters: zero when the library is loaded, and put back
                                                                   // to zero by the routing kernel itself at the end of every call
  c.d_chain_next = reinterpret_cast<int*>(base + kOffChainNext);   // never read: the app entry carries no chain flag
  c.d_row_rec = reinterpret_cast<RowRec*>(base + kOffRowRec);
  c.d_panel = reinterpret_cast<__nv_bfloat16*>(base + kOffPanel);
  c.d_z = reinterpret_cast<float*>(base + kOffZ);
  c.panel_rows_cap = kStaticRows;
  c.out_topk_idx = topk_idx;
  c.out_topk_val = topk_val;

  AppEntry ae;
  memset(&ae, 0, sizeof(ae));
  ae.valid = 1;
  ae.kind = MIX_SAE;
  ae.group = 0;
  ae.n_edit = app->n_edit;
  ae.add_error = app->add_error ? 1 : 0;
  GroupEntry ge;
  memset(&ge, 0, sizeof(ge));
  ge.valid = 1;
  ge.act = w->act;
  ge.k = w->act == MIX_SAE_TOPK ? w->k : 0;
  ge.d_sae = w->d_sae;
  ge.W_enc = static_cast<const __nv_bfloat16*>(w->W_enc);
  ge.b_eff = w->b_enc;
  ge.theta = w->theta;
  ge.W_dec = static_cast<const __nv_bfloat16*>(w->W_dec);
  ge.b_dec = w->b_dec;

  // The array keeps whatever the previous call left: one small kernel rewrites every table this call reads,
  // from values it received as kernel parameters.  (Routing rewrites the row lists and counters itself; the
  // panel, Z and TopK lists are fully rewritten for the rows in use before they are read.)
  StaticSetup su;
  memset(&su, 0, sizeof(su));
  su.n_rows = n_rows;
  su.n_edit = app->n_edit;
  su.app = ae;
  su.group = ge;
  for (int i = 0; i < app->n_edit; ++i) {
    su.edit_idx[i] = app->idx[i];
    su.edit_val[i] = app->val[i];
    su.edit_mode[i] = app->mode[i];
  }
  static_setup_kernel<<<1, 128, 0, s>>>(su, c.d_token_slot, c.d_n_live, c.d_status, c.d_apps, c.d_groups, c.d_edit_idx,
                                        c.d_edit_val, c.d_edit_mode);
  cudaError_t e = cudaGetLastError();
  __nv_bfloat16* h = static_cast<__nv_bfloat16*>(hidden);
  if (e == cudaSuccess) e = launch_front(&c, h, n_rows, s);       // routing + row pack
  if (e == cudaSuccess) e = launch_encode_simt(&c, s);
  if (e == cudaSuccess) e = launch_tail(&c, h, 1, s);             // selection, edits, decode, write-back
  if (e != cudaSuccess) return fail(errbuf, errbuf_len, MIX_ERR_CUDA, "CUDA error %lld while enqueuing the static SAE call", (long long)e);
  return MIX_OK;
}
