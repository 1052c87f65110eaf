// The plain CUDA-core SAE encode (the in-library cross-check of the tensor-core encode, MIX_FLAG_ENCODE_SIMT)
// and the edit-only shortcut (MIX_FLAG_SAE_EDIT_ONLY):
//
//   encode_simt_kernel   : Z = panel W_enc^T + b, fp32 FMA on a shared-memory tile.
//   sae_edit_only_kernel : for ReLU / JumpReLU rows that keep the error term, only the pre-activations of the
//                          edited features (warp-level MMA), leaving per token row the coefficients f'_j - f_j;
//   decode_delta_kernel  : adds sum_j (f'_j - f_j) W_dec[j] to those rows, eight rows per CTA.
#include "mix_internal.h"

namespace mix {

namespace {

// ---------------------------------------------------------------------------------------
// cross-check encode: Z[p, j] = sum_i panel[p, i] * W_enc[j, i] + b_eff[j], fp32 FMA
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
encode_simt_kernel(const __nv_bfloat16* __restrict__ panel, const int* __restrict__ mtile_group,
                   const RouteState* __restrict__ rs, const GroupEntry* __restrict__ groups, float* __restrict__ Z,
                   long long ldz, int d) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int BM = 64, BN = 64, BK = 32;
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  const int p0 = blockIdx.y * BM;
  if (p0 >= rs->n_panel_rows) return;
  const int g = mtile_group[p0 / kTileM];
  if (g < 0) return;
  const GroupEntry ge = groups[g];
  const long long j0 = (long long)blockIdx.x * BN;
  if (j0 >= ge.d_sae) return;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int lr = tid >> 2, lk = (tid & 3) * 8;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < d; k0 += BK) {
    {
      const uint4 qa = *reinterpret_cast<const uint4*>(panel + (size_t)(p0 + lr) * d + k0 + lk);
      const uint4 qb = *reinterpret_cast<const uint4*>(ge.W_enc + (size_t)(j0 + lr) * d + k0 + lk);
      const __nv_bfloat16* a = reinterpret_cast<const __nv_bfloat16*>(&qa);
      const __nv_bfloat16* b = reinterpret_cast<const __nv_bfloat16*>(&qb);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        As[lk + e][lr] = __bfloat162float(a[e]);
        Bs[lk + e][lr] = __bfloat162float(b[e]);
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = As[k][ty * 4 + i];
        b[i] = Bs[k][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const long long col = j0 + tx * 4 + j;
      Z[(size_t)(p0 + ty * 4 + i) * ldz + col] = acc[i][j] + ge.b_eff[col];
    }
}

__device__ __forceinline__ void axpy8(float* acc, float c, const uint4& q) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    acc[2 * i] = fmaf(c, t.x, acc[2 * i]);
    acc[2 * i + 1] = fmaf(c, t.y, acc[2 * i + 1]);
  }
}

// ---------------------------------------------------------------------------------------
// decode of rows with the error term: h' = h + sum over edited j of (f'_j - f_j) W_dec[j]
// ---------------------------------------------------------------------------------------
// A CTA owns kDdRows consecutive packed rows and a slice of 1024 columns.  Consecutive packed rows
// usually belong to one request, i.e. one slot and one edit list, so every edited W_dec row is
// loaded once per CTA and applied to all of its rows with per-row coefficients (f_j differs by
// row): the gather's L2 traffic drops by up to kDdRows.  Rows of different slots in one CTA are
// handled by listing the edits of every distinct slot, with zero coefficients for foreign rows.
constexpr int kDdRows = 8;
constexpr int kDdThreads = 128;
constexpr int kDdBatch = 8;
constexpr int kDdEntries = kDdRows * kMaxEdits;

__device__ __forceinline__ void decode_delta_fma(float (&acc)[kDdRows][8], const float* coef, const uint4& q) {
  const float4 c0 = *reinterpret_cast<const float4*>(coef);
  const float4 c1 = *reinterpret_cast<const float4*>(coef + 4);
  axpy8(acc[0], c0.x, q);
  axpy8(acc[1], c0.y, q);
  axpy8(acc[2], c0.z, q);
  axpy8(acc[3], c0.w, q);
  axpy8(acc[4], c1.x, q);
  axpy8(acc[5], c1.y, q);
  axpy8(acc[6], c1.z, q);
  axpy8(acc[7], c1.w, q);
}

// The kernel in front has already left, per row, the slot (or -1 when there is nothing to add), the
// decoder matrix and one coefficient f'_j - f_j per edit entry, so the chain of dependent loads here
// is short: row records -> (residual rows, edit lists, coefficients) -> decoder rows -> store.
__global__ void __launch_bounds__(kDdThreads, 4)
decode_delta_kernel(__nv_bfloat16* __restrict__ hidden, int d, const int* __restrict__ panel_row,
                    const RouteState* __restrict__ rs, const RowDelta* __restrict__ row_delta,
                    const float* __restrict__ edit_coef, const int* __restrict__ edit_idx, int r_max, int n_token_rows) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ __align__(16) float s_coef[kDdEntries + kDdBatch][kDdRows];
  __shared__ const uint4* s_wrow[kDdEntries + kDdBatch];
  __shared__ int s_t[kDdRows], s_slot[kDdRows], s_nedit[kDdRows];
  __shared__ const __nv_bfloat16* s_wdec[kDdRows];
  const int p0 = blockIdx.x * kDdRows;
  const int tid = threadIdx.x;
  // panel_row == nullptr: the records are indexed by token row (the edit-only shortcut), n_token_rows of them
  const int n_rows = panel_row ? rs->n_panel_rows : n_token_rows;
  if (tid < kDdRows) {
    const int p = p0 + tid;                              // packed rows are in bounds: the panel capacity is a multiple of 128
    const bool in = panel_row != nullptr || p < n_rows;
    const int t = !in ? -1 : (panel_row ? panel_row[p] : p);
    RowDelta rd;
    rd.slot = -1;
    rd.n_edit = 0;
    rd.W_dec = nullptr;
    if (in) rd = row_delta[p];
    const bool on = p < n_rows && t >= 0 && rd.slot >= 0;
    s_t[tid] = on ? t : -1;
    s_slot[tid] = on ? rd.slot : -1;
    s_nedit[tid] = rd.n_edit;
    s_wdec[tid] = rd.W_dec;
  }
  if (p0 >= n_rows) return;
  __syncthreads();
  bool any = false;
#pragma unroll
  for (int r = 0; r < kDdRows; ++r) any = any || s_slot[r] >= 0;
  if (!any) return;
  const int v = blockIdx.y * kDdThreads + tid;          // this thread's 16-byte column vector
  const bool in_cols = v < (d >> 3);
  uint4 hraw[kDdRows];
#pragma unroll
  for (int r = 0; r < kDdRows; ++r) {
    const int t = s_t[r];
    hraw[r] = make_uint4(0u, 0u, 0u, 0u);
    if (t >= 0 && in_cols) hraw[r] = reinterpret_cast<const uint4*>(hidden + (size_t)t * d)[v];
  }
  // entries: the edit lists of the distinct slots, one after the other; thread e of a slot fills
  // entry e for all rows (the coefficient of a row of another slot is zero)
  int n_entries = 0;                                    // CTA-uniform
  for (int r = 0; r < kDdRows; ++r) {
    const int slot = s_slot[r];
    bool first = slot >= 0;
    for (int r2 = 0; r2 < r; ++r2) first = first && s_slot[r2] != slot;
    if (!first) continue;
    const int n_edit = s_nedit[r];
    if (tid < n_edit) {
      const int j = edit_idx[slot * r_max + tid];
      float c[kDdRows];
#pragma unroll
      for (int r2 = 0; r2 < kDdRows; ++r2)
        c[r2] = s_slot[r2] == slot ? edit_coef[(size_t)(p0 + r2) * r_max + tid] : 0.f;
#pragma unroll
      for (int r2 = 0; r2 < kDdRows; ++r2) s_coef[n_entries + tid][r2] = c[r2];
      s_wrow[n_entries + tid] = reinterpret_cast<const uint4*>(s_wdec[r] + (size_t)j * d);
    }
    n_entries += n_edit;
  }
  __syncthreads();
  // pad to a whole batch: repeats of the last decoder row with zero coefficients
  if (tid < kDdBatch) {
    s_wrow[n_entries + tid] = s_wrow[n_entries - 1];
#pragma unroll
    for (int r2 = 0; r2 < kDdRows; ++r2) s_coef[n_entries + tid][r2] = 0.f;
  }
  __syncthreads();
  if (!in_cols) return;
  float acc[kDdRows][8];
#pragma unroll
  for (int r = 0; r < kDdRows; ++r) {
    const __nv_bfloat162* pp = reinterpret_cast<const __nv_bfloat162*>(&hraw[r]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f2 = __bfloat1622float2(pp[i]);
      acc[r][2 * i] = f2.x;
      acc[r][2 * i + 1] = f2.y;
    }
  }
  // kDdBatch decoder rows in flight per thread: the loop is bound by load latency, not arithmetic
  for (int e0 = 0; e0 < n_entries; e0 += kDdBatch) {
    uint4 q[kDdBatch];
#pragma unroll
    for (int u = 0; u < kDdBatch; ++u) q[u] = __ldg(s_wrow[e0 + u] + v);
#pragma unroll
    for (int u = 0; u < kDdBatch; ++u) decode_delta_fma(acc, &s_coef[e0 + u][0], q[u]);
  }
#pragma unroll
  for (int r = 0; r < kDdRows; ++r) {
    if (s_slot[r] < 0) continue;
    uint4 o;
    __nv_bfloat162* pp = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) pp[i] = __floats2bfloat162_rn(acc[r][2 * i], acc[r][2 * i + 1]);
    reinterpret_cast<uint4*>(hidden + (size_t)s_t[r] * d)[v] = o;
  }
}

// ---------------------------------------------------------------------------------------
// edit-only shortcut (MIX_FLAG_SAE_EDIT_ONLY)
// ---------------------------------------------------------------------------------------
// With the error term on, h' = h + sum over edited j of (f'_j - f_j) W_dec[j]: for ReLU and JumpReLU
// sets f_j depends on z_j alone, so a row needs just the |edits| pre-activations
// z_j = W_enc[j] . h + b_eff[j] -- 16 dot products instead of the d_sae-wide encode.  (TopK rows
// still need every pre-activation to know which features are kept.)
// Two launches.  sae_edit_only_kernel: a CTA owns kEoRows consecutive TOKEN rows, straight from the slot map,
// and keeps them in shared memory.  Consecutive rows mostly belong to one request, i.e. one slot and one edit
// list, so every edited W_enc row is fetched once per CTA and contracted with all of its rows on the warp-level
// tensor-core MMA; rows of different slots in one CTA are handled by listing the edits of every distinct slot (a
// row takes no part in the entries of another slot).  It leaves, per token row, the record decode_delta_kernel
// reads -- slot or -1, decoder, one coefficient f'_j - f_j per edit entry -- and that kernel, launched next with
// token-indexed records, adds the deltas (8 rows x 1024 columns per CTA, decoder rows shared likewise).
constexpr int kEoRows = 8;
constexpr int kEoThreads = 256;
constexpr int kEoEntries = kEoRows * kMaxEdits;
constexpr int kEoLoads = 4;      // 32-column chunks in flight per warp in the dot-product pass

struct EoRow {
  int t;                 // token row, or -1 when the row takes no part
  int slot, n_edit, act;
  const __nv_bfloat16* W_enc;
  const __nv_bfloat16* W_dec;
  const float* b_eff;
  const float* theta;
};

__global__ void __launch_bounds__(kEoThreads)
sae_edit_only_kernel(__nv_bfloat16* __restrict__ hidden, int d, const int* __restrict__ token_slot,
                     const int* __restrict__ n_live_p, int T, const AppEntry* __restrict__ apps,
                     const GateEntry* __restrict__ gates, int n_slots, const GroupEntry* __restrict__ groups,
                     int n_groups, const int* __restrict__ edit_idx, const float* __restrict__ edit_val,
                     const unsigned char* __restrict__ edit_mode, int r_max, RowDelta* __restrict__ row_delta,
                     float* __restrict__ edit_coef, int T_max) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ uint4 s_h[];                                   // [kEoRows][nvec]: the CTA's rows
  __shared__ EoRow s_row[kEoRows];
  __shared__ const uint4* s_wenc[kEoEntries];
  __shared__ int s_feat[kEoEntries], s_owner[kEoEntries], s_pos[kEoEntries];   // feature id, owning row, position in its slot's list
  __shared__ int s_changed[kEoRows];
  __shared__ float s_part[kEoThreads / 32][kEoRows][16];            // per-warp partial pre-activations of a pass
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nvec = d >> 3;
  const int t0 = blockIdx.x * kEoRows;
  if (tid < kEoRows) {
    EoRow r;
    r.t = -1;
    r.slot = -1;
    r.n_edit = 0;
    const int t = t0 + tid;
    if (t < min(T, *n_live_p)) {
      const int slot = token_slot[t];
      if (slot >= 0 && slot < n_slots) {
        const AppEntry app = apps[slot];
        bool on = app.valid && (app.kind & kKindMask) == MIX_SAE && app.add_error && app.group >= 0 && app.group < n_groups &&
                  app.n_edit > 0;
        GroupEntry ge;
        if (on) {
          ge = groups[app.group];
          on = ge.valid && ge.act != MIX_SAE_TOPK;
        }
        if (on && (app.kind & kKindGated)) {
          const GateEntry gt = gates[slot];
          const float v = gt.scores[(size_t)t * gt.stride + gt.col];
          on = gt.cmp == MIX_GATE_GE ? v >= gt.thr : v < gt.thr;
        }
        if (on) {
          r.t = t;
          r.slot = slot;
          r.n_edit = app.n_edit;
          r.act = ge.act;
          r.W_enc = ge.W_enc;
          r.W_dec = ge.W_dec;
          r.b_eff = ge.b_eff;
          r.theta = ge.theta;
        }
      }
    }
    s_row[tid] = r;
    s_changed[tid] = 0;
  }
  __syncthreads();
  bool any = false;
#pragma unroll
  for (int r = 0; r < kEoRows; ++r) any = any || s_row[r].t >= 0;
  if (!any) {                                                      // every row of the CTA: nothing to add
    if (tid < kEoRows && t0 + tid < T_max) row_delta[t0 + tid].slot = -1;
    return;
  }
  // the rows into shared memory
  for (int r = 0; r < kEoRows; ++r) {
    const int t = s_row[r].t;
    if (t < 0) continue;
    const uint4* hrow = reinterpret_cast<const uint4*>(hidden + (size_t)t * d);
    for (int v = tid; v < nvec; v += kEoThreads) s_h[(size_t)r * nvec + v] = hrow[v];
  }
  // entries: the edit lists of the distinct slots, one after the other (n_entries is uniform across the CTA)
  int n_entries = 0;
  for (int r = 0; r < kEoRows; ++r) {
    const int slot = s_row[r].slot;
    bool first = s_row[r].t >= 0;
    for (int r2 = 0; r2 < r; ++r2) first = first && s_row[r2].slot != slot;
    if (!first) continue;
    const int n_edit = s_row[r].n_edit;
    if (tid < n_edit) {
      const int j = edit_idx[slot * r_max + tid];
      s_feat[n_entries + tid] = j;
      s_owner[n_entries + tid] = r;
      s_pos[n_entries + tid] = tid;
      s_wenc[n_entries + tid] = reinterpret_cast<const uint4*>(s_row[r].W_enc + (size_t)j * d);
    }
    n_entries += n_edit;
  }
  __syncthreads();
  // pre-activations Z[8 rows x entries] = H[8 x d] W_enc[entries x d]^T on the warp-level tensor-core MMA
  // (m16n8k16, bf16 -> fp32; rows 8..15 of the A tile are zero), 16 entries per pass, the warps splitting d
  // between them.  Fragments as in probe_multiclass_kernel: lane (g, q) takes 16 contiguous bytes, columns
  // 8q..8q+7 of a 32-column chunk, of row g (from shared memory) and of the encoder rows of entries g and g + 8
  // (from global memory); which columns a fragment slot holds is immaterial as long as A and B agree.
  {
    const int g = lane >> 2, q = lane & 3;
    const int n_chunks = d >> 5;
    for (int e0 = 0; e0 < n_entries; e0 += 16) {                   // uniform
      const uint4* w0 = e0 + g < n_entries ? s_wenc[e0 + g] : nullptr;
      const uint4* w1 = e0 + 8 + g < n_entries ? s_wenc[e0 + 8 + g] : nullptr;
      float acc[2][4];
#pragma unroll
      for (int ct = 0; ct < 2; ++ct) acc[ct][0] = acc[ct][1] = acc[ct][2] = acc[ct][3] = 0.f;
      for (int ch0 = warp; ch0 < n_chunks; ch0 += (kEoThreads / 32) * kEoLoads) {
        uint4 ha[kEoLoads], b0[kEoLoads], b1[kEoLoads];
#pragma unroll
        for (int u = 0; u < kEoLoads; ++u) {
          const int ch = ch0 + u * (kEoThreads / 32);
          const bool in = ch < n_chunks;
          const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
          ha[u] = in ? s_h[(size_t)g * nvec + ch * 4 + q] : zero;
          b0[u] = (in && w0) ? __ldg(w0 + ch * 4 + q) : zero;
          b1[u] = (in && w1) ? __ldg(w1 + ch * 4 + q) : zero;
        }
#pragma unroll
        for (int u = 0; u < kEoLoads; ++u) {
#pragma unroll
          for (int ct = 0; ct < 2; ++ct) {
            const uint4& bb = ct == 0 ? b0[u] : b1[u];
            asm volatile(
                "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                "{%0, %1, %2, %3};"
                : "+f"(acc[ct][0]), "+f"(acc[ct][1]), "+f"(acc[ct][2]), "+f"(acc[ct][3])
                : "r"(ha[u].x), "r"(0u), "r"(ha[u].y), "r"(0u), "r"(bb.x), "r"(bb.y));
            asm volatile(
                "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                "{%0, %1, %2, %3};"
                : "+f"(acc[ct][0]), "+f"(acc[ct][1]), "+f"(acc[ct][2]), "+f"(acc[ct][3])
                : "r"(ha[u].z), "r"(0u), "r"(ha[u].w), "r"(0u), "r"(bb.z), "r"(bb.w));
          }
        }
      }
      // lane (g, q): row g, entries e0 + 8 ct + 2q and + 1
#pragma unroll
      for (int ct = 0; ct < 2; ++ct) {
        s_part[warp][g][ct * 8 + 2 * q] = acc[ct][0];
        s_part[warp][g][ct * 8 + 2 * q + 1] = acc[ct][1];
      }
      __syncthreads();
      if (tid < kEoRows * 16) {                                      // one thread per (row, entry of the pass)
        const int r = tid >> 4, e = e0 + (tid & 15);
        if (e < n_entries) {
          const int owner = s_owner[e], slot = s_row[owner].slot, j = s_feat[e];
          float delta = 0.f;
          if (s_row[r].t >= 0 && s_row[r].slot == slot) {
            float z = s_row[owner].b_eff[j];
#pragma unroll
            for (int w = 0; w < kEoThreads / 32; ++w) z += s_part[w][r][tid & 15];
            const int pos = s_pos[e], n_edit = s_row[owner].n_edit;
            const float f = s_row[owner].act == MIX_SAE_RELU ? fmaxf(z, 0.f) : (z > s_row[owner].theta[j] ? z : 0.f);
            bool alive = true;                                       // a later entry for the same feature wins
            for (int e2 = pos + 1; e2 < n_edit; ++e2) alive = alive && (s_feat[e - pos + e2] != j);
            const float fnew = edit_mode[slot * r_max + pos] == MIX_EDIT_CLAMP ? edit_val[slot * r_max + pos] : 0.f;
            delta = alive ? fnew - f : 0.f;
            if (delta != 0.f) s_changed[r] = 1;
            edit_coef[(size_t)(t0 + r) * r_max + pos] = delta;      // the record decode_delta_kernel reads (token-indexed)
          }
        }
      }
      __syncthreads();
    }
  }
  // per token row: the slot (-1 when no edit changes anything: the row then stays bit-exact), the length of its
  // edit list and the decoder; decode_delta_kernel, launched next, adds the deltas
  if (tid < kEoRows && t0 + tid < T_max) {
    RowDelta rd;
    rd.slot = (s_row[tid].t >= 0 && s_changed[tid]) ? s_row[tid].slot : -1;
    rd.n_edit = s_row[tid].n_edit;
    rd.W_dec = s_row[tid].W_dec;
    row_delta[t0 + tid] = rd;
  }
}

}  // namespace

cudaError_t launch_encode_simt(const Ctx* c, cudaStream_t s) {
  dim3 grid((unsigned)(c->cfg.d_sae_max / 64), (unsigned)(c->panel_rows_cap / 64));
  return launch_pdl(kPdlEncode, encode_simt_kernel, dim3(grid), dim3(256), 0, s, c->d_panel, c->d_mtile_group, c->d_route, c->d_groups, c->d_z,
                                          c->cfg.d_sae_max, c->cfg.d_model);
}

cudaError_t edit_only_prepare() {
  return cudaFuncSetAttribute(sae_edit_only_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kEoRows * 8192 * 2);
}

cudaError_t launch_edit_only(const Ctx* c, __nv_bfloat16* hidden, int T, cudaStream_t s) {
  const size_t smem = (size_t)kEoRows * c->cfg.d_model * sizeof(__nv_bfloat16);
  cudaError_t e = launch_pdl(kPdlTail, sae_edit_only_kernel, dim3((c->cfg.T_max + kEoRows - 1) / kEoRows), dim3(kEoThreads), smem, s,
                             hidden, c->cfg.d_model, c->d_token_slot, c->d_n_live, T, c->d_apps, c->d_gates, c->cfg.n_slots_max,
                             c->d_groups, c->cfg.n_groups_max, c->d_edit_idx, c->d_edit_val, c->d_edit_mode, c->cfg.r_max,
                             c->d_eo_row_delta, c->d_eo_coef, c->cfg.T_max);
  return e;
}

cudaError_t launch_edit_only_delta(const Ctx* c, __nv_bfloat16* hidden, cudaStream_t s) {
  dim3 grid((unsigned)((c->cfg.T_max + kDdRows - 1) / kDdRows), (unsigned)((c->cfg.d_model / 8 + kDdThreads - 1) / kDdThreads));
  return launch_pdl(kPdlTail, decode_delta_kernel, dim3(grid), dim3(kDdThreads), 0, s, hidden, c->cfg.d_model,
                    static_cast<const int*>(nullptr), c->d_route, c->d_eo_row_delta, c->d_eo_coef, c->d_edit_idx, c->cfg.r_max,
                    c->cfg.T_max);
}

}  // namespace mix
