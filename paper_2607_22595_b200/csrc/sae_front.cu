// Front of the SAE chain: slot routing and the row pack in ONE launch.
//
// Routing is integer work on the slot map: which rows carry an SAE app, of which weight set, and where each of
// them goes in the packed panel (weight set by weight set, ascending token order inside a set, every set
// starting on a 128-row tile).  It used to be a one-CTA kernel followed by a pack kernel that waited for it.
// Here EVERY CTA repeats the routing for itself -- the slot map and the small tables are a few tens of KiB, L2
// hits after the first CTA -- and then packs its own 32 panel rows, one per warp: no CTA waits for another, and
// one launch and one dependent kernel boundary disappear from the front of every SAE call.  CTA 0 alone writes
// what exists once (the routing result the encode reads, the tile -> weight-set map, the conditional handle).
//
// Pack forms: the bf16 row as it is; with an 8-bit encoder the row as E4M3 codes with a power-of-two row
// scale -- quantised (MIX_FLAG_FP8_ACT), or split exactly into two E4M3 operands hi + lo.
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "mix_internal.h"
#include "row_lookup.cuh"

namespace mix {

namespace {

constexpr int kFrontThreads = 1024;
constexpr int kFrontWarps = kFrontThreads / 32;
constexpr int kFrontRowsMax = 512;        // most panel rows one CTA packs (a multiple of 32: whole rounds of one row per warp)
constexpr int kRouteBatch = 8;            // chunks of 1024 rows whose look-ups are in flight together

// bf16 row -> panel row (or zeros for the padding rows of a tile: they must be finite).
__device__ __forceinline__ void pack_row_bf16(const __nv_bfloat16* __restrict__ hidden, int t, __nv_bfloat16* __restrict__ panel,
                                              size_t p, int d, int lane) {
  uint4* dst = reinterpret_cast<uint4*>(panel + p * d);
  const int nvec = d >> 3;
  if (t < 0) {
    for (int i = lane; i < nvec; i += 32) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)t * d);
  int i = lane;
  for (; i + 224 < nvec; i += 256) {                     // eight loads in flight per lane
    uint4 q[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) q[u] = __ldg(src + i + 32 * u);
#pragma unroll
    for (int u = 0; u < 8; ++u) dst[i + 32 * u] = q[u];
  }
  for (; i < nvec; i += 32) dst[i] = __ldg(src + i);
}

// 8-bit encoder: the row goes into the panel as E4M3 codes with a power-of-two row scale.
// s = the smallest power of two with max|h_i| / s <= 448 (never below 2^-100; 1 for a row of zeros); h_i / s is
// exact in fp32, the conversion rounds to nearest even.  A first pass finds the largest magnitude, a second
// one (the row is in L1 by then) writes the codes.
//   kSplit = false (MIX_FLAG_FP8_ACT): code_i = E4M3 nearest to h_i / s -- the encoder's input IS quantised.
//   kSplit = true  (MIX_FLAG_FP8_W_ENC alone): the bf16 row is kept, as the sum of two E4M3 operands with the same
//     scale: hi_i = E4M3 nearest to x = h_i / s, lo_i = E4M3 nearest to x - hi_i (exact subtraction).  A bf16 value
//     has 8 significant bits, hi takes the leading 4 and the remainder has at most 4, so hi + lo = x exactly
//     unless bits of x lie below 2^-9 (the subnormal step of E4M3), i.e. the error per element is at most
//     2^-10 s <= 4.4e-6 max|h_i| and zero for |h_i| >= 2^-2 s.  The lo codes go to rows [lo_row0 + p] of the panel.
template <bool kSplit>
__device__ __forceinline__ void pack_row_e4m3(const __nv_bfloat16* __restrict__ hidden, int t, unsigned char* __restrict__ panel,
                                              float* __restrict__ act_scale, size_t p, int d, int lo_row0, int lane) {
  uint2* dst = reinterpret_cast<uint2*>(panel + p * d);
  uint2* dst_lo = reinterpret_cast<uint2*>(panel + ((size_t)lo_row0 + p) * d);
  const int nvec = d >> 3;
  if (t < 0) {   // padding rows of a tile
    for (int i = lane; i < nvec; i += 32) {
      dst[i] = make_uint2(0u, 0u);
      if (kSplit) dst_lo[i] = make_uint2(0u, 0u);
    }
    if (lane == 0) act_scale[p] = 0.f;
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)t * d);
  unsigned m2 = 0u;                                     // two 15-bit magnitudes, compared as integers
  for (int i = lane; i < nvec; i += 32) {
    const uint4 q = __ldg(src + i);
    m2 = __vmaxu2(m2, __vmaxu2(__vmaxu2(q.x & 0x7fff7fffu, q.y & 0x7fff7fffu), __vmaxu2(q.z & 0x7fff7fffu, q.w & 0x7fff7fffu)));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m2 = __vmaxu2(m2, __shfl_xor_sync(0xffffffffu, m2, o));
  const unsigned a = max(m2 & 0xffffu, m2 >> 16);       // bf16 bits of max|h_i|: (1 + frac / 128) * 2^(E - 127)
  int e = 0;
  if (a != 0u) {
    const int E = (int)(a >> 7) - 127, frac = (int)(a & 0x7fu);
    e = max(E - (frac <= 96 ? 8 : 7), -100);            // 448 = 1.75 * 2^8, and 1.75 = 1 + 96 / 128
  }
  const float inv = __uint_as_float((unsigned)(127 - e) << 23);
  if (lane == 0) act_scale[p] = __uint_as_float((unsigned)(127 + e) << 23);
  for (int i = lane; i < nvec; i += 32) {
    const uint4 q = __ldg(src + i);
    const unsigned w[4] = {q.x, q.y, q.z, q.w};
    unsigned short c[4], cl[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float lo = __uint_as_float(w[u] << 16) * inv, hi = __uint_as_float(w[u] & 0xffff0000u) * inv;
      c[u] = __nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, __NV_E4M3);
      if (kSplit) {
        const float2 back = __half22float2(__half2(__nv_cvt_fp8x2_to_halfraw2(c[u], __NV_E4M3)));   // exact: E4M3 fits fp16
        cl[u] = __nv_cvt_float2_to_fp8x2(make_float2(lo - back.x, hi - back.y), __NV_SATFINITE, __NV_E4M3);
      }
    }
    dst[i] = make_uint2((unsigned)c[0] | ((unsigned)c[1] << 16), (unsigned)c[2] | ((unsigned)c[3] << 16));
    if (kSplit) dst_lo[i] = make_uint2((unsigned)cl[0] | ((unsigned)cl[1] << 16), (unsigned)cl[2] | ((unsigned)cl[3] << 16));
  }
}

struct FrontArgs {
  // slot map and tables (read)
  const int* token_slot;
  const int* n_live_p;
  int T;
  const AppEntry* apps;
  const GateEntry* gates;
  int n_slots;
  const GroupEntry* groups;
  int n_groups;
  const int* chain_next;
  int edit_only;
  // routing results (written)
  int* panel_row;
  RowRec* row_rec;
  int panel_cap;
  int rows_per_cta;        // panel rows packed by one CTA: a multiple of 32, <= kFrontRowsMax
  int* mtile_group;
  RouteState* rs;
  unsigned* status;
  int* row_flag;
  int* mtile_flag;
  int* n_flagged;
  int* row_group;          // scratch, used only by batches beyond the first 8192 rows
  int* row_slot;           // scratch, likewise
  cudaGraphConditionalHandle cond;
  int use_cond;
  // pack
  const __nv_bfloat16* hidden;
  void* panel;
  float* act_scale;
  int d;
  unsigned* tau_slots;
  unsigned* tau_min;
  int lo_row0;
  unsigned long long* clk;   // profiling aid or null
};

// kPack: 0 the bf16 row, 1 E4M3 hi + lo (exact split), 2 E4M3 quantised.
template <int kPack>
__global__ void __launch_bounds__(kFrontThreads)
front_kernel(const FrontArgs a) {
  extern __shared__ int s_cnt[];                      // [n_chunks * kFrontWarps][n_groups]
  __shared__ int s_total[kMaxGroups], s_base[kMaxGroups + 1];
  __shared__ int s_tok[kFrontRowsMax], s_slot[kFrontRowsMax], s_grp[kFrontRowsMax];
  __shared__ int s_n_panel_rows;
  __shared__ int s_gact[kMaxGroups], s_gtiles[kMaxGroups];   // per weight set: activation, feature tiles (0: not registered)
  __shared__ int s_n_delta;
  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool first_cta = blockIdx.x == 0;
  const int n_groups = a.n_groups, n_slots = a.n_slots;
  const int n_live = min(a.T, __ldg(a.n_live_p));
  const int n_chunks = (n_live + kFrontThreads - 1) / kFrontThreads;
  phase_stamp(a.clk, 0, first_cta && tid == 0);
  const int n_own = a.rows_per_cta;
  const int p0 = blockIdx.x * n_own;
  if (tid < n_own) s_tok[tid] = -1;
  if (tid == 0) s_n_delta = 0;
  if (tid < n_groups) {                                // requested now, needed after the scan
    const bool valid = __ldg(&a.groups[tid].valid) != 0;
    s_gact[tid] = __ldg(&a.groups[tid].act);
    s_gtiles[tid] = valid ? (int)(__ldg(&a.groups[tid].d_sae) / kTileN) : 0;
  }

  // phase A: the weight set (or -1) of every row this thread owns (row c * 1024 + tid of chunk c), resolved
  // stage by stage for kRouteBatch chunks at a time so that their loads are in flight together: the slot ids
  // (requested together with the live count), then bytes 0..31 of the app entries -- valid, kind, weight set,
  // edit count, error-term flag in one round trip; the weight sets' own entries were requested at the top of
  // the kernel.  Then per (chunk, warp) counts per set.  The first batch (8192 rows: every configuration in use)
  // stays in registers for phase C; later batches go through the row_group / row_slot scratch (every CTA writes
  // the same values there and reads back its own).
  // meta: (weight set + 1) | edit count << 8 | error-term flag << 16; 0 = not an SAE row of this call
  int meta0[kRouteBatch], slot0[kRouteBatch];
  const int T_cap = a.T;
  const int n_chunks_cap = (T_cap + kFrontThreads - 1) / kFrontThreads;
  bool groups_ready = false;
  for (int c0 = 0; c0 < n_chunks_cap; c0 += kRouteBatch) {
    int slot[kRouteBatch], meta[kRouteBatch];
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      const int t = (c0 + c) * kFrontThreads + tid;
      slot[c] = t < T_cap ? __ldg(a.token_slot + t) : -1;      // does not wait for the live count
    }
    if (c0 >= n_chunks) break;                                  // (uniform) nothing live from here on
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      const int t = (c0 + c) * kFrontThreads + tid;
      if (t >= n_live || slot[c] >= n_slots) slot[c] = -1;
    }
    int2 q0[kRouteBatch];                 // valid, kind
    int3 q1[kRouteBatch];                 // weight set, edit count, error-term flag
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      q0[c] = make_int2(0, 0);
      q1[c] = make_int3(0, 0, 0);
      if (slot[c] >= 0) {
        const AppEntry* e = a.apps + slot[c];
        q0[c] = __ldg(reinterpret_cast<const int2*>(e));
        q1[c].x = __ldg(&e->group);
        const int2 ne = __ldg(reinterpret_cast<const int2*>(&e->n_edit));
        q1[c].y = ne.x;
        q1[c].z = ne.y;
      }
    }
    // a row whose slot starts a chain is an SAE row if the chain ends in an SAE app: follow the
    // links (rare, so the dependent loads are not batched) and carry on with that app's slot
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      if (q0[c].x && (q0[c].y & kKindChained) && (q0[c].y & kKindMask) != MIX_SAE) {
        int s2 = slot[c];
        int2 h2 = q0[c];
        for (int depth = 1; depth < kMaxChain && s2 >= 0; ++depth) {
          s2 = (h2.y & kKindChained) ? __ldg(a.chain_next + s2) : -1;
          if (s2 < 0 || s2 >= n_slots) { s2 = -1; break; }
          h2 = __ldg(reinterpret_cast<const int2*>(a.apps + s2));
          if (!h2.x) { s2 = -1; break; }
          if ((h2.y & kKindMask) == MIX_SAE) break;
        }
        if (s2 >= 0 && (h2.y & kKindMask) != MIX_SAE) s2 = -1;
        slot[c] = s2;
        q0[c] = s2 >= 0 ? h2 : make_int2(0, 0);
        q1[c] = make_int3(0, 0, 0);
        if (s2 >= 0) {
          q1[c].x = __ldg(&a.apps[s2].group);
          q1[c].y = __ldg(&a.apps[s2].n_edit);
          q1[c].z = __ldg(&a.apps[s2].add_error);
        }
      }
    }
    if (!groups_ready) {                   // the weight-set table requested at the top has long arrived
      __syncthreads();
      groups_ready = true;
    }
    int n_delta = 0;
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      meta[c] = 0;
      if (q0[c].x && (q0[c].y & kKindMask) == MIX_SAE) {
        const int g = q1[c].x, n_edit = q1[c].y, add_error = q1[c].z != 0;
        if (g < 0 || g >= n_groups || s_gtiles[g] == 0) {
          if (first_cta) atomicOr(a.status, MIX_STATUS_BAD_GROUP);
        } else if (a.edit_only && add_error && s_gact[g] != MIX_SAE_TOPK) {
          // handled by sae_edit_only_kernel: with the error term on, a ReLU / JumpReLU row needs
          // only the pre-activations of its edited features, not the whole encode
        } else if (!(q0[c].y & kKindGated) || gate_open(a.gates, slot[c], (c0 + c) * kFrontThreads + tid)) {
          meta[c] = (g + 1) | (n_edit << 8) | (add_error << 16);
          n_delta += add_error && n_edit > 0 && s_gact[g] != MIX_SAE_TOPK;
        }
      }
    }
    n_delta = __reduce_add_sync(0xffffffffu, n_delta);
    if (lane == 0 && n_delta) atomicAdd(&s_n_delta, n_delta);
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      if (c0 == 0) {
        meta0[c] = meta[c];
        slot0[c] = slot[c];
      }
      if (c0 + c < n_chunks) {                       // uniform across the CTA
        const int t = (c0 + c) * kFrontThreads + tid;
        if (c0 > 0 && t < n_live) {
          a.row_group[t] = meta[c];
          a.row_slot[t] = slot[c];
        }
        const int grp = (meta[c] & 0xff) - 1;
        for (int q = 0; q < n_groups; ++q) {
          const unsigned m = __ballot_sync(0xffffffffu, grp == q);
          if (lane == 0) s_cnt[((c0 + c) * kFrontWarps + warp) * n_groups + q] = __popc(m);
        }
      }
    }
  }
  if (!groups_ready) __syncthreads();
  phase_stamp(a.clk, 1, first_cta && tid == 0);
  if (n_chunks == 0) {
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      meta0[c] = 0;
      slot0[c] = -1;
    }
  }
  __syncthreads();
  // phase B: exclusive scan over (chunk, warp) for each weight set; warp q owns set q
  const int n_seg = n_chunks * kFrontWarps;
  for (int q = warp; q < n_groups; q += kFrontWarps) {
    int carry = 0;
    for (int s0 = 0; s0 < n_seg; s0 += 32) {
      const int i = s0 + lane;
      const int v = i < n_seg ? s_cnt[i * n_groups + q] : 0;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      if (i < n_seg) s_cnt[i * n_groups + q] = carry + incl - v;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) s_total[q] = carry;
  }
  __syncthreads();
  if (tid == 0) {
    int mt = 0, tiles = 0, rows = 0, topk_rows = 0;
    for (int q = 0; q < n_groups; ++q) {
      s_base[q] = mt * kTileM;
      const int m_tiles = (s_total[q] + kTileM - 1) / kTileM;
      const int act = s_gact[q];
      if (first_cta) {
        a.rs->group_count[q] = s_total[q];
        a.rs->group_mtile0[q] = mt;
        a.rs->group_tile0[q] = tiles;
        for (int m = 0; m < m_tiles; ++m) a.mtile_group[mt + m] = q;
      }
      mt += m_tiles;
      rows += s_total[q];
      if (s_total[q] > 0 && act == MIX_SAE_TOPK) topk_rows += s_total[q];
      tiles += s_total[q] > 0 ? m_tiles * s_gtiles[q] : 0;
    }
    s_base[n_groups] = mt * kTileM;
    s_n_panel_rows = mt * kTileM;
    if (first_cta) {
      for (int q = n_groups; q <= kMaxGroups; ++q) {
        a.rs->group_mtile0[q] = mt;
        a.rs->group_tile0[q] = tiles;
        if (q < kMaxGroups) a.rs->group_count[q] = 0;
      }
      for (int m = mt; m < a.panel_cap / kTileM; ++m) a.mtile_group[m] = -1;
      a.rs->n_panel_rows = mt * kTileM;
      a.rs->n_mtiles = mt;
      a.rs->n_sae_rows = rows;
      a.rs->total_tiles = tiles;
      a.rs->n_topk_rows = topk_rows;
      a.rs->n_delta_rows = s_n_delta;
      if (a.n_flagged) *a.n_flagged = 0;       // fallback-selection flags of the fused TopK path start clear every call
      // graph-conditional form: the rest of the SAE chain sits in the body of an IF node that runs only when a row needs it
      if (a.use_cond) cudaGraphSetConditional(a.cond, rows > 0 ? 1u : 0u);
    }
  }
  if (first_cta && a.mtile_flag)
    for (int m = tid; m < a.panel_cap / kTileM; m += kFrontThreads) a.mtile_flag[m] = 0;
  __syncthreads();
  phase_stamp(a.clk, 2, first_cta && tid == 0);
  // phase C: stable positions; a row that lands in this CTA's share of the panel leaves its token here
  for (int c0 = 0; c0 < n_chunks; c0 += kRouteBatch) {
    int meta[kRouteBatch], slot[kRouteBatch];
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      const int t = (c0 + c) * kFrontThreads + tid;
      if (c0 == 0) {
        meta[c] = meta0[c];
        slot[c] = slot0[c];
      } else {
        meta[c] = (c0 + c < n_chunks && t < n_live) ? a.row_group[t] : 0;
        slot[c] = meta[c] ? a.row_slot[t] : -1;
      }
    }
#pragma unroll
    for (int c = 0; c < kRouteBatch; ++c) {
      if (c0 + c < n_chunks) {
        const int grp = (meta[c] & 0xff) - 1;
        for (int q = 0; q < n_groups; ++q) {
          const unsigned m = __ballot_sync(0xffffffffu, grp == q);
          if (grp == q) {
            const int pos = s_base[q] + s_cnt[((c0 + c) * kFrontWarps + warp) * n_groups + q] +
                            __popc(m & ((1u << lane) - 1u));
            if (pos >= p0 && pos < p0 + n_own) {
              s_tok[pos - p0] = (c0 + c) * kFrontThreads + tid;
              s_slot[pos - p0] = slot[c];
              s_grp[pos - p0] = meta[c];
            }
          }
        }
      }
    }
  }
  __syncthreads();
  phase_stamp(a.clk, 3, first_cta && tid == 0);
  // this CTA's panel rows, one per warp and round: the row's record for the kernels behind the encode, then the row itself
  for (int r = warp; r < n_own; r += kFrontWarps) {
    const int p = p0 + r;
    if (p >= a.panel_cap) break;
    const int t = s_tok[r];
    if (p < s_n_panel_rows) {
      if (a.tau_slots) {                                 // the encode's TopK bound starts empty
        reinterpret_cast<uint4*>(a.tau_slots + (size_t)p * kTauSlots)[lane] = make_uint4(0u, 0u, 0u, 0u);
        if (lane == 0) a.tau_min[p] = 0u;
      }
      if (kPack == 0)
        pack_row_bf16(a.hidden, t, static_cast<__nv_bfloat16*>(a.panel), (size_t)p, a.d, lane);
      else
        pack_row_e4m3<kPack == 1>(a.hidden, t, static_cast<unsigned char*>(a.panel), a.act_scale, (size_t)p, a.d, a.lo_row0, lane);
    }
    if (lane == 0) {
      RowRec rec;
      rec.t = t;
      rec.slot = t >= 0 ? s_slot[r] : -1;
      const int meta = t >= 0 ? s_grp[r] : 0, g = (meta & 0xff) - 1;
      rec.n_edit = (meta >> 8) & 0xff;
      rec.group_flags = t >= 0 ? (g | ((meta >> 16) & 1 ? kRecAddError : 0) | (s_gact[g] << kRecActShift)) : 0;
      a.row_rec[p] = rec;
      a.panel_row[p] = t;
      if (a.row_flag) a.row_flag[p] = 0;
    }
  }
  phase_stamp(a.clk, 4, first_cta && tid == 0);
}

}  // namespace

cudaError_t launch_front(const Ctx* c, const __nv_bfloat16* hidden, int T, cudaStream_t s, unsigned long long cond, int use_cond) {
  FrontArgs a;
  a.token_slot = c->d_token_slot;
  a.n_live_p = c->d_n_live;
  a.T = T;
  a.apps = c->d_apps;
  a.gates = c->d_gates;
  a.n_slots = c->cfg.n_slots_max;
  a.groups = c->d_groups;
  a.n_groups = c->cfg.n_groups_max;
  a.chain_next = c->d_chain_next;
  a.edit_only = (c->cfg.flags & MIX_FLAG_SAE_EDIT_ONLY) ? 1 : 0;
  a.panel_row = c->d_panel_row;
  a.row_rec = c->d_row_rec;
  a.panel_cap = c->panel_rows_cap;
  a.mtile_group = c->d_mtile_group;
  a.rs = c->d_route;
  a.status = c->d_status;
  a.row_flag = c->d_row_flag;
  a.mtile_flag = c->d_mtile_flag;
  a.n_flagged = c->d_n_flagged;
  a.row_group = c->d_row_group;
  a.row_slot = c->d_row_slot;
  a.cond = static_cast<cudaGraphConditionalHandle>(cond);
  a.use_cond = use_cond;
  a.hidden = hidden;
  a.panel = c->d_panel;
  a.act_scale = c->d_act_scale;
  a.d = c->cfg.d_model;
  a.tau_slots = c->d_tau;
  a.tau_min = c->d_tau_min;
  a.lo_row0 = c->panel_rows_cap;
  a.clk = c->d_phase_clk;
  const int n_chunks = (c->cfg.T_max + kFrontThreads - 1) / kFrontThreads;
  const size_t smem = (size_t)n_chunks * kFrontWarps * c->cfg.n_groups_max * sizeof(int);
  // one wave of CTAs where the panel allows it (a CTA of 1024 threads has an SM to itself)
  const int n_sms = c->n_sms > 0 ? c->n_sms : 148;
  int rows = ((c->panel_rows_cap + n_sms - 1) / n_sms + 31) / 32 * 32;
  rows = rows < 32 ? 32 : (rows > kFrontRowsMax ? kFrontRowsMax : rows);
  a.rows_per_cta = rows;
  const dim3 grid((c->panel_rows_cap + rows - 1) / rows);
  if (c->cfg.flags & MIX_FLAG_FP8_ACT)
    front_kernel<2><<<grid, kFrontThreads, smem, s>>>(a);
  else if (c->cfg.flags & MIX_FLAG_FP8_W_ENC)      // hi codes in rows [0, P), lo codes in rows [P, 2P) of the same buffer
    front_kernel<1><<<grid, kFrontThreads, smem, s>>>(a);
  else
    front_kernel<0><<<grid, kFrontThreads, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace mix
