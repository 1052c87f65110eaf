// The read (probe) and write (steering) primitives of the hook, and the small kernels around the slot map.
//
// probe_steer_kernel is the bandwidth kernel of the hook: one warp per token row, 16-byte
// loads, fp32 FMA, shuffle reductions.  A row whose slot is -1 costs one 4-byte load.
#include "mix_internal.h"
#include "row_lookup.cuh"

namespace mix {

namespace {

__device__ __forceinline__ void unpack8(const uint4& q, float* f) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

__device__ __forceinline__ uint4 pack8(const float* f) {
  uint4 q;
  __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return q;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// h + alpha v for one row; nvec = d / 8 16-byte vectors.  The `stride` threads that share the
// row start at `first` (a warp: lane, 32; a CTA team: threadIdx.x, blockDim.x).
__device__ __forceinline__ void steer_row(uint4* __restrict__ h, const uint4* __restrict__ v, float alpha,
                                          int nvec, int first, int stride) {
  constexpr int U = 4;
  int i = first;
  for (; i + (U - 1) * stride < nvec; i += U * stride) {
    uint4 hq[U], vq[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      hq[u] = __ldcs(h + i + u * stride);
      vq[u] = __ldg(v + i + u * stride);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float a[8], b[8];
      unpack8(hq[u], a);
      unpack8(vq[u], b);
#pragma unroll
      for (int e = 0; e < 8; ++e) a[e] = fmaf(alpha, b[e], a[e]);
      __stcs(h + i + u * stride, pack8(a));
    }
  }
  for (; i < nvec; i += stride) {
    float a[8], b[8];
    unpack8(__ldcs(h + i), a);
    unpack8(__ldg(v + i), b);
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = fmaf(alpha, b[e], a[e]);
    __stcs(h + i, pack8(a));
  }
}

// Partial logits of RB rows against NC consecutive probe rows over this thread's share of the
// columns; warp-reduced, so every lane of a warp returns the warp's sums.
template <int RB, int NC>
__device__ __forceinline__ void probe_dots(const uint4* const* __restrict__ h, const uint4* __restrict__ W, int nvec,
                                           int nc, int first, int stride, float (*out)[NC]) {
  float acc[RB][NC];
#pragma unroll
  for (int r = 0; r < RB; ++r)
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[r][c] = 0.f;
  constexpr int U = (NC == 1 && RB == 1) ? 4 : 1;
  int i = first;
  for (; i + (U - 1) * stride < nvec; i += U * stride) {
    uint4 hq[U][RB];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int r = 0; r < RB; ++r) hq[u][r] = __ldg(h[r] + i + u * stride);
    uint4 wq[U][NC];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int c = 0; c < NC; ++c)
        if (c < nc) wq[u][c] = __ldg(W + (size_t)c * nvec + i + u * stride);
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
      for (int c = 0; c < NC; ++c)
        if (c < nc) {
          float b[8];
          unpack8(wq[u][c], b);
#pragma unroll
          for (int r = 0; r < RB; ++r) {
            float a[8];
            unpack8(hq[u][r], a);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[r][c] = fmaf(a[e], b[e], acc[r][c]);
          }
        }
    }
  }
  if (U > 1) {
    for (; i < nvec; i += stride) {
      float a[8], b[8];
      unpack8(__ldg(h[0] + i), a);
      unpack8(__ldg(W + i), b);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[0][0] = fmaf(a[e], b[e], acc[0][0]);
    }
  }
#pragma unroll
  for (int r = 0; r < RB; ++r)
#pragma unroll
    for (int c = 0; c < NC; ++c) out[r][c] = warp_sum(acc[r][c]);
}

// 1 / (1 + e^-z) with the hardware exponential and reciprocal: a few instructions instead of the two library
// routines' hundred on the one-warp tail of a decode step (0.28 us of a 3 us step); the relative error stays
// below 1e-5 for |z| < 80, two orders under the 1e-3 the scores are held to.
__device__ __forceinline__ float fast_sigmoid(float z) { return __frcp_rn(1.f + __expf(-z)); }

// Logits (bias included) of one row in `logit` -> scores.  One warp; C <= 64.
__device__ __forceinline__ void finish_probe(const float* logit, int C, int act, float* __restrict__ out, int lane) {
  if (C == 1) {                                  // the decode step's case: one lane, no cross-lane work
    if (lane == 0) {
      const float z = logit[0];
      out[0] = act == MIX_ACT_NONE ? z : (act == MIX_ACT_SOFTMAX ? 1.f : fast_sigmoid(z));
    }
    return;
  }
  float z0 = lane < C ? logit[lane] : -INFINITY;
  float z1 = lane + 32 < C ? logit[lane + 32] : -INFINITY;
  if (act == MIX_ACT_SOFTMAX) {
    float m = fmaxf(z0, z1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float e0 = lane < C ? expf(z0 - m) : 0.f;
    const float e1 = lane + 32 < C ? expf(z1 - m) : 0.f;
    const float sum = warp_sum(e0 + e1);
    z0 = e0 / sum;
    z1 = e1 / sum;
  } else if (act == MIX_ACT_SIGMOID) {
    z0 = fast_sigmoid(z0);
    z1 = fast_sigmoid(z1);
  }
  if (lane < C) out[lane] = z0;
  if (lane + 32 < C) out[lane + 32] = z1;
}

constexpr int kWarpsPerBlock = 8;      // = rows per CTA of the large-batch kernel
constexpr int kCoopMaxClasses = 32;    // widest probe the cooperative tensor-core pass takes

// One row, one warp: steer, single-class probe, or multi-class probe.
__device__ __forceinline__ void warp_row(const RowApp& a, __nv_bfloat16* __restrict__ hidden, int t, int d,
                                         float* __restrict__ scores, int C_max, float* s_logit, int lane) {
  const int nvec = d >> 3;
  uint4* hrow = reinterpret_cast<uint4*>(hidden + (size_t)t * d);
  if (a.kind == MIX_STEER) {
    if (a.alpha != 0.f) steer_row(hrow, a.W, a.alpha, nvec, lane, 32);   // alpha = 0: row stays bit-exact
    return;
  }
  const uint4* h1[1] = {hrow};
  if (a.kind == MIX_PROJECT) {                 // h - beta (h . r) r: one pass for the dot, one for the update
    if (a.alpha == 0.f) return;
    float z[1][1];
    probe_dots<1, 1>(h1, a.W, nvec, 1, lane, 32, z);
    steer_row(hrow, a.W, -a.alpha * z[0][0], nvec, lane, 32);
    return;
  }
  if (a.kind != MIX_PROBE || scores == nullptr) return;
  float* out = scores + (size_t)t * C_max;
  if (a.C == 1) {
    float z[1][1];
    probe_dots<1, 1>(h1, a.W, nvec, 1, lane, 32, z);
    if (lane == 0) {
      const float zz = z[0][0] + (a.b ? __ldg(a.b) : 0.f);
      // one class: raw logit, sigmoid, or a softmax over a single entry (= 1)
      out[0] = a.act == MIX_ACT_NONE ? zz : (a.act == MIX_ACT_SOFTMAX ? 1.f : fast_sigmoid(zz));
    }
    return;
  }
  for (int c0 = 0; c0 < a.C; c0 += 4) {
    float z[1][4];
    const int nc = min(4, a.C - c0);
    probe_dots<1, 4>(h1, a.W + (size_t)c0 * nvec, nvec, nc, lane, 32, z);
    if (lane == 0) {
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (c < nc) s_logit[c0 + c] = z[0][c] + (a.b ? __ldg(a.b + c0 + c) : 0.f);
    }
  }
  __syncwarp();
  finish_probe(s_logit, a.C, a.act, out, lane);
}

// Large batches: a CTA owns 8 consecutive rows, one warp per row: streaming work (steering,
// single-class probes).  Multi-class probes up to kCoopMaxClasses classes are left to
// probe_tc_kernel (probe_tc.cu) when `multiclass_elsewhere` is set.
__global__ void __launch_bounds__(kWarpsPerBlock * 32, 3)
probe_steer_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
                   const AppEntry* __restrict__ apps, const GateEntry* __restrict__ gates, int n_slots,
                   __nv_bfloat16* __restrict__ hidden, int d,
                   float* __restrict__ scores, int C_max, unsigned* __restrict__ status, int multiclass_elsewhere) {
  __shared__ float s_logit[kWarpsPerBlock][kMaxClasses];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  const int n_live = __ldg(n_live_p);            // issued together with the slot id: one round trip, not two
  const int slot = t < T ? __ldg(token_slot + t) : -1;
  if (t >= min(T, n_live)) return;
  const RowApp a = lookup(slot, t, apps, gates, n_slots, status, lane == 0);
  if (a.kind == 0) return;
  if (multiclass_elsewhere && a.kind == MIX_PROBE && a.C > 1 && a.C <= kCoopMaxClasses) return;
  warp_row(a, hidden, t, d, scores, C_max, s_logit[warp], lane);
}

// 16-byte read-only load that the compiler may not sink below later volatile statements: keeps
// all loads of a batch in flight before the first MMA that consumes them.
__device__ __forceinline__ uint4 ldg128_early(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

constexpr int kMcRows = 16;            // rows per CTA of probe_multiclass_kernel (one m16 MMA tile)
constexpr int kMcWarps = 8;            // warps per CTA: they split d between them

// One warp's share of the contraction of 16 rows against one probe matrix on the warp-level
// tensor-core MMA (m16n8k16, bf16 -> fp32): every kMcWarps-th 32-column chunk of d, UB chunks in flight,
// KCT 8-class tiles.  Fragments come straight from global memory, 16 contiguous bytes per lane:
// lane (g, q) takes columns 8q..8q+7 of the chunk for rows g and g + 8 and for class g of each
// 8-class tile.  Which columns a fragment slot holds is immaterial as long as A and B agree,
// because the sum runs over all of them.  Partial logits go to part[row][class].
template <int KCT, int UB>
__device__ __forceinline__ void mc_contract(const uint4* __restrict__ h_lo, const uint4* __restrict__ h_hi,
                                            const uint4* __restrict__ W, int C, int n_chunks, int row_vecs,
                                            float (*part)[kCoopMaxClasses]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, q = lane & 3;
  float acc[KCT][4];
#pragma unroll
  for (int ct = 0; ct < KCT; ++ct) acc[ct][0] = acc[ct][1] = acc[ct][2] = acc[ct][3] = 0.f;
  for (int ch0 = warp; ch0 < n_chunks; ch0 += kMcWarps * UB) {
    uint4 lo[UB], hi[UB], wq[UB][KCT];
#pragma unroll
    for (int u = 0; u < UB; ++u) {
      const int ch = ch0 + u * kMcWarps;
      const bool in = ch < n_chunks;
      lo[u] = in ? ldg128_early(h_lo + ch * 4 + q) : make_uint4(0u, 0u, 0u, 0u);
      hi[u] = in ? ldg128_early(h_hi + ch * 4 + q) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int ct = 0; ct < KCT; ++ct) {
        const int cls = ct * 8 + g;
        wq[u][ct] = (in && cls < C) ? ldg128_early(W + (size_t)cls * row_vecs + ch * 4 + q) : make_uint4(0u, 0u, 0u, 0u);
      }
    }
#pragma unroll
    for (int u = 0; u < UB; ++u) {
#pragma unroll
      for (int ct = 0; ct < KCT; ++ct) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
            "{%0, %1, %2, %3};"
            : "+f"(acc[ct][0]), "+f"(acc[ct][1]), "+f"(acc[ct][2]), "+f"(acc[ct][3])
            : "r"(lo[u].x), "r"(hi[u].x), "r"(lo[u].y), "r"(hi[u].y), "r"(wq[u][ct].x), "r"(wq[u][ct].y));
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
            "{%0, %1, %2, %3};"
            : "+f"(acc[ct][0]), "+f"(acc[ct][1]), "+f"(acc[ct][2]), "+f"(acc[ct][3])
            : "r"(lo[u].z), "r"(hi[u].z), "r"(lo[u].w), "r"(hi[u].w), "r"(wq[u][ct].z), "r"(wq[u][ct].w));
      }
    }
  }
  // lane (g, q): rows g (acc 0, 1) and g + 8 (acc 2, 3), classes 8 ct + 2q and + 1
#pragma unroll
  for (int ct = 0; ct < KCT; ++ct) {
    if (ct * 8 < C) {
      part[g][ct * 8 + 2 * q] = acc[ct][0];
      part[g][ct * 8 + 2 * q + 1] = acc[ct][1];
      part[g + 8][ct * 8 + 2 * q] = acc[ct][2];
      part[g + 8][ct * 8 + 2 * q + 1] = acc[ct][3];
    }
  }
}

// What the CTA knows about each of its rows.
struct McRow {
  const uint4* W;
  const float* b;
  int C, act;
  int slot;      // slot id if the row is a multi-class probe this kernel takes and its gate is open, else -1
};

// Multi-class probes of large batches.  16 rows x C classes x d is a skinny dense contraction;
// consecutive rows usually belong to one request and share the probe.  For every distinct
// multi-class probe among the CTA's 16 rows, the warps split d between them and contract ALL
// 16 rows against that probe's matrix, which is therefore streamed from L2 once per 16 rows;
// only the rows that belong to the probe keep their result.
__global__ void __launch_bounds__(kMcWarps * 32, 2)
probe_multiclass_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
                        const AppEntry* __restrict__ apps, const GateEntry* __restrict__ gates, int n_slots,
                        const __nv_bfloat16* __restrict__ hidden, int d, float* __restrict__ scores, int C_max,
                        const McCensus* __restrict__ census) {
  __shared__ float s_part[kMcWarps][kMcRows][kCoopMaxClasses];   // [warp][row][class]
  __shared__ float s_logit[kMcWarps][kCoopMaxClasses];
  __shared__ McRow s_row[kMcRows];
  __shared__ int s_any;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t0 = blockIdx.x * kMcRows;
  const int n_live = min(T, __ldg(n_live_p));
  if (t0 >= n_live || scores == nullptr) return;
  if (census != nullptr && census->use_tc) return;          // this call's batch is probe_tc_kernel's
  if (threadIdx.x == 0) s_any = 0;
  __syncthreads();
  if (threadIdx.x < kMcRows) {           // one thread per row: slot -> entry -> gate
    const int t = t0 + threadIdx.x;
    McRow r;
    r.slot = -1;
    if (t < n_live) {
      const int s = __ldg(token_slot + t);
      const RowApp a = lookup(s, t, apps, gates, n_slots, nullptr, false);   // bad slots are flagged by probe_steer_kernel
      if (a.kind == MIX_PROBE && a.C > 1 && a.C <= kCoopMaxClasses) {
        r.W = a.W;
        r.b = a.b;
        r.C = a.C;
        r.act = a.act;
        r.slot = s;
        s_any = 1;
      }
    }
    s_row[threadIdx.x] = r;
  }
  __syncthreads();
  if (!s_any) return;                    // CTA-uniform
  const int g = lane >> 2;
  const uint4* h_lo = reinterpret_cast<const uint4*>(hidden + (size_t)min(t0 + g, n_live - 1) * d);
  const uint4* h_hi = reinterpret_cast<const uint4*>(hidden + (size_t)min(t0 + g + 8, n_live - 1) * d);
  const int n_chunks = d >> 5, row_vecs = d >> 3;
  for (int r = 0; r < kMcRows; ++r) {
    const McRow ci = s_row[r];
    if (ci.slot < 0) continue;
    bool first = true;
    for (int r2 = 0; r2 < r; ++r2) first = first && s_row[r2].slot != ci.slot;
    if (!first) continue;
    if (ci.C <= 16)
      mc_contract<2, 4>(h_lo, h_hi, ci.W, ci.C, n_chunks, row_vecs, s_part[warp]);
    else
      mc_contract<kCoopMaxClasses / 8, 2>(h_lo, h_hi, ci.W, ci.C, n_chunks, row_vecs, s_part[warp]);
    __syncthreads();
#pragma unroll 1
    for (int rr = warp; rr < kMcRows; rr += kMcWarps) {     // warp w finishes row w
      if (s_row[rr].slot != ci.slot) continue;
      for (int c = lane; c < ci.C; c += 32) {
        float z = ci.b ? __ldg(ci.b + c) : 0.f;
#pragma unroll
        for (int w = 0; w < kMcWarps; ++w) z += s_part[w][rr][c];
        s_logit[warp][c] = z;
      }
      __syncwarp();
      finish_probe(s_logit[warp], ci.C, ci.act, scores + (size_t)(t0 + rr) * C_max, lane);
      __syncwarp();
    }
    __syncthreads();                     // s_part is reused by the next probe
  }
}

// Small batches (decode): one CTA of NW warps per row, the row held in registers (up to kTeamVec
// 16-byte vectors per thread).  The row's loads are issued as soon as the slot id is known to be
// >= 0, in parallel with the app-table lookup, so a cold row costs two dependent round trips
// (slot, then entry + data) instead of three.  Control flow is uniform across the CTA.
constexpr int kTeamVec = 4;     // NW * 32 * kTeamVec * 8 >= d_model: 8192 columns at NW = 8

template <int NW>
__global__ void __launch_bounds__(NW * 32)
probe_steer_team_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
                        const AppEntry* __restrict__ apps, const GateEntry* __restrict__ gates, int n_slots,
                        __nv_bfloat16* __restrict__ hidden, int d, float* __restrict__ scores, int C_max,
                        unsigned* __restrict__ status, const uint4* __restrict__ vec_arena, int pdl) {
  __shared__ float s_part[NW][kMaxClasses];
  constexpr int NT = NW * 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x;                      // < T_max: the slot map has an entry for every row
  // Programmatic dependent launch (`pdl`: the launch asked for it): everything up to pdl_wait() reads only
  // tables the LIBRARY owns and that only copies write -- live count, slot map, app entry, vector arena -- so it
  // may run while the kernel in front of this one in the stream (the layer that produces `hidden`, or the
  // previous hook) is still running.  Memory the caller owns (`hidden`, multi-class probe weights, gate scores)
  // is read after the wait only, and every thread waits before it leaves, so that this grid cannot end -- and
  // release ITS successor -- before its predecessor has.  Launched the ordinary way, nothing has to wait: the
  // row is then requested together with the vector and the app entry, one round trip earlier.
  if (pdl) pdl_launch_dependents();
  const int n_live = __ldg(n_live_p);            // both loads issue together: one round trip, not two
  const int slot = __ldg(token_slot + t);
  if (t >= min(T, n_live) || slot == -1) {
    if (pdl) pdl_wait();
    return;
  }
  const int nvec = d >> 3;
  uint4* hrow = reinterpret_cast<uint4*>(hidden + (size_t)t * d);
  // Single-vector weights (steering, projection, one-class probe) were copied at registration
  // into row `slot` of the context's vector arena, so their address follows from the slot id
  // alone: the row AND its vector are requested together, before the app entry is known.
  uint4 hq[kTeamVec], vq[kTeamVec];
  const bool slot_ok = slot >= 0 && slot < n_slots;
  if (slot_ok) {
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) vq[u] = __ldg(vec_arena + (size_t)slot * nvec + v);
    }
  }
  if (!pdl && slot_ok) {
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) hq[u] = __ldcs(hrow + v);
    }
  }
  RowApp a = lookup(slot, t, apps, gates, n_slots, status, threadIdx.x == 0, /*eval_gate=*/false);
  if (pdl) {
    pdl_wait();
    if (slot_ok) {
#pragma unroll
      for (int u = 0; u < kTeamVec; ++u) {
        const int v = threadIdx.x + u * NT;
        if (v < nvec) hq[u] = __ldcs(hrow + v);
      }
    }
  }
  // A one-class probe's bias came with the entry (registration put it into the `alpha` word); the biases of a
  // wider probe are requested as soon as the entry is here, not after the dot products they are added to.
  float bias_lo = 0.f, bias_hi = 0.f;
  if (a.kind == MIX_PROBE && warp == 0) {
    if (a.C == 1) {
      bias_lo = a.alpha;
    } else if (a.b != nullptr) {
      if (lane < a.C) bias_lo = __ldg(a.b + lane);
      if (lane + 32 < a.C) bias_hi = __ldg(a.b + lane + 32);
    }
  }
  if (a.gated && a.kind != 0 && !gate_open(gates, slot, t)) return;       // gate closed: the row passes through
  if (a.kind == MIX_STEER) {
    if (a.alpha == 0.f) return;                  // identity; the row stays bit-exact
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) {
        float x[8], y[8];
        unpack8(hq[u], x);
        unpack8(vq[u], y);
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = fmaf(a.alpha, y[e], x[e]);
        __stcs(hrow + v, pack8(x));
      }
    }
    return;
  }
  if (a.kind == MIX_PROJECT) {                 // h - beta (h . r) r
    if (a.alpha == 0.f) return;
    float dot = 0.f;
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) {
        float x[8], y[8];
        unpack8(hq[u], x);
        unpack8(vq[u], y);
#pragma unroll
        for (int e = 0; e < 8; ++e) dot = fmaf(x[e], y[e], dot);
      }
    }
    dot = warp_sum(dot);
    if (lane == 0) s_part[warp][0] = dot;
    __syncthreads();
    float total = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) total += s_part[w][0];
    const float coef = -a.alpha * total;
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) {
        float x[8], y[8];
        unpack8(hq[u], x);
        unpack8(vq[u], y);
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = fmaf(coef, y[e], x[e]);
        __stcs(hrow + v, pack8(x));
      }
    }
    return;
  }
  if (a.kind != MIX_PROBE || scores == nullptr) return;
  if (a.C == 1) {                              // the probe vector is already here
    float acc = 0.f;
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) {
        float x[8], y[8];
        unpack8(hq[u], x);
        unpack8(vq[u], y);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fmaf(x[e], y[e], acc);
      }
    }
    acc = warp_sum(acc);
    if (lane == 0) s_part[warp][0] = acc;
  }
  for (int c0 = 0; c0 < (a.C == 1 ? 0 : a.C); c0 += 4) {
    const int nc = min(4, a.C - c0);
    uint4 wq[4][kTeamVec];
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
      for (int u = 0; u < kTeamVec; ++u) {
        const int v = threadIdx.x + u * NT;
        if (c < nc && v < nvec) wq[c][u] = __ldg(a.W + (size_t)(c0 + c) * nvec + v);
      }
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) {
        float x[8];
        unpack8(hq[u], x);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (c < nc) {
            float y[8];
            unpack8(wq[c][u], y);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[c] = fmaf(x[e], y[e], acc[c]);
          }
      }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float z = warp_sum(acc[c]);
      if (lane == 0 && c < nc) s_part[warp][c0 + c] = z;
    }
  }
  __syncthreads();
  if (warp == 0) {
    for (int c = lane; c < a.C; c += 32) {
      float z = c < 32 ? bias_lo : bias_hi;
#pragma unroll
      for (int w = 0; w < NW; ++w) z += s_part[w][c];
      s_part[0][c] = z;            // only this lane reads or writes column c from here on
    }
    __syncwarp();
    finish_probe(s_part[0], a.C, a.act, scores + (size_t)t * C_max, lane);
  }
}

// Contexts with slot chains: one CTA per row, the row held in registers while the apps of its chain
// are applied one after the other (probe / steering / projection; an SAE app at the end of a chain
// is left to the SAE kernels, which start after this one).  A write rounds the row to bf16 in
// registers, exactly as a store and reload would; the row goes back to memory once, at the end,
// if any app changed it.  The j-th probe of a chain writes its scores after those of the earlier
// ones.  Control flow is uniform across the CTA.
constexpr int kChainWarps = 8;

__global__ void __launch_bounds__(kChainWarps * 32)
probe_steer_chain_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
                         const AppEntry* __restrict__ apps, const GateEntry* __restrict__ gates,
                         const int* __restrict__ chain_next, int n_slots, __nv_bfloat16* __restrict__ hidden, int d,
                         float* __restrict__ scores, int C_max, unsigned* __restrict__ status) {
  __shared__ float s_part[kChainWarps][kMaxClasses];
  constexpr int NT = kChainWarps * 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x;                      // < T_max: the slot map has an entry for every row
  // programmatic dependent launch, as in probe_steer_team_kernel: the live count and the slot id (library-owned,
  // written only by copies) may be read while the predecessor still runs; everything else comes after the wait,
  // and every thread waits before it leaves
  pdl_launch_dependents();
  const int n_live = __ldg(n_live_p);
  int slot = __ldg(token_slot + t);
  pdl_wait();
  if (t >= min(T, n_live) || slot == -1) return;
  const int nvec = d >> 3;
  uint4* hrow = reinterpret_cast<uint4*>(hidden + (size_t)t * d);
  uint4 hq[kTeamVec];
#pragma unroll
  for (int u = 0; u < kTeamVec; ++u) {
    const int v = threadIdx.x + u * NT;
    hq[u] = make_uint4(0u, 0u, 0u, 0u);
    if (v < nvec && slot >= 0 && slot < n_slots) hq[u] = __ldcs(hrow + v);
  }
  bool dirty = false;
  int col = 0;
  for (int depth = 0; depth < kMaxChain; ++depth) {
    const RowApp a = lookup(slot, t, apps, gates, n_slots, status, threadIdx.x == 0);
    if ((a.kind == MIX_STEER || a.kind == MIX_PROJECT) && a.alpha != 0.f) {   // alpha = 0: identity, bit-exact
      uint4 vq[kTeamVec];
#pragma unroll
      for (int u = 0; u < kTeamVec; ++u) {
        const int v = threadIdx.x + u * NT;
        vq[u] = make_uint4(0u, 0u, 0u, 0u);
        if (v < nvec) vq[u] = __ldg(a.W + v);
      }
      float coef = a.alpha;
      if (a.kind == MIX_PROJECT) {               // h - beta (h . r) r
        float dot = 0.f;
#pragma unroll
        for (int u = 0; u < kTeamVec; ++u) {
          float x[8], y[8];
          unpack8(hq[u], x);
          unpack8(vq[u], y);
#pragma unroll
          for (int e = 0; e < 8; ++e) dot = fmaf(x[e], y[e], dot);
        }
        dot = warp_sum(dot);
        if (lane == 0) s_part[warp][0] = dot;
        __syncthreads();
        float total = 0.f;
#pragma unroll
        for (int w = 0; w < kChainWarps; ++w) total += s_part[w][0];
        coef = -a.alpha * total;
      }
#pragma unroll
      for (int u = 0; u < kTeamVec; ++u) {
        float x[8], y[8];
        unpack8(hq[u], x);
        unpack8(vq[u], y);
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = fmaf(coef, y[e], x[e]);
        hq[u] = pack8(x);
      }
      dirty = true;
    } else if (a.kind == MIX_PROBE && scores != nullptr) {
      for (int c0 = 0; c0 < a.C; c0 += 4) {
        const int nc = min(4, a.C - c0);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int u = 0; u < kTeamVec; ++u) {
          const int v = threadIdx.x + u * NT;
          if (v < nvec) {
            float x[8];
            unpack8(hq[u], x);
#pragma unroll
            for (int c = 0; c < 4; ++c)
              if (c < nc) {
                float y[8];
                unpack8(__ldg(a.W + (size_t)(c0 + c) * nvec + v), y);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[c] = fmaf(x[e], y[e], acc[c]);
              }
          }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float z = warp_sum(acc[c]);
          if (lane == 0 && c < nc) s_part[warp][c0 + c] = z;
        }
      }
      __syncthreads();
      if (warp == 0) {
        for (int c = lane; c < a.C; c += 32) {
          float z = a.b ? __ldg(a.b + c) : 0.f;
#pragma unroll
          for (int w = 0; w < kChainWarps; ++w) z += s_part[w][c];
          s_part[0][c] = z;            // only this lane reads or writes column c from here on
        }
        __syncwarp();
        finish_probe(s_part[0], a.C, a.act, scores + (size_t)t * C_max + col, lane);
      }
    }
    if (!a.chained) break;
    if (a.raw_kind == MIX_PROBE) col += a.C;
    slot = __ldg(chain_next + slot);             // slot was in range: lookup() found a valid entry
    if (slot < 0) break;
    __syncthreads();                             // s_part is reused by the next app
  }
  if (dirty) {
#pragma unroll
    for (int u = 0; u < kTeamVec; ++u) {
      const int v = threadIdx.x + u * NT;
      if (v < nvec) __stcs(hrow + v, hq[u]);
    }
  }
}

// Router-logit steering: one thread per (row, expert).
__global__ void __launch_bounds__(256)
router_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
              const AppEntry* __restrict__ apps, const GateEntry* __restrict__ gates, int n_slots,
              float* __restrict__ logits, int n_experts) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int t = (int)(i / n_experts), e = (int)(i - (long long)t * n_experts);
  if (t >= min(T, __ldg(n_live_p))) return;
  const RowApp a = lookup(__ldg(token_slot + t), t, apps, gates, n_slots, nullptr, false);
  if (a.kind != MIX_ROUTER || a.C != n_experts) return;
  logits[i] += __ldg(reinterpret_cast<const float*>(a.W) + e);
}

__global__ void compose_map_kernel(const int* __restrict__ token_req, const int* __restrict__ req_slot, int T_live,
                                   int n_req, int* __restrict__ token_slot) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T_live) return;
  const int r = token_req[t];
  token_slot[t] = (r >= 0 && r < n_req) ? req_slot[r] : -1;
}

// b_eff[j] = b_enc[j] - sum_i W_enc[j,i] * b_dec[i]   (one warp per feature; registration time)
__global__ void fold_bias_kernel(const __nv_bfloat16* __restrict__ W_enc, const float* __restrict__ b_enc,
                                 const float* __restrict__ b_dec, float* __restrict__ b_eff, long long d_sae, int d) {
  const long long j = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (j >= d_sae) return;
  float acc = 0.f;
  for (int i = lane; i < d; i += 32) acc = fmaf(__bfloat162float(W_enc[j * d + i]), b_dec[i], acc);
  acc = warp_sum(acc);
  if (lane == 0) b_eff[j] = b_enc[j] - acc;
}

// Census of the batch's multi-class probe rows (2..32 classes; gates are not looked at): a CTA takes 8 tiles of
// 128 rows, one per warp (four rows per lane, their loads in flight together), counts each tile's such rows and
// appends the tiles that have any to a list -- one reservation per CTA, so the shared counters see two additions
// per 1024 rows; the last CTA to finish publishes the totals and the choice between the two probe kernels, and
// puts the working counters back to zero for the next call.
// The tensor-core kernel streams whole tiles, the 16-row kernel reaches 38 % of the HBM rate against its 80 %:
// it takes the call when the listed tiles are, on average, at least half full of such rows.
constexpr int kCensusWarps = 8;
__global__ void __launch_bounds__(kCensusWarps * 32)
mc_census_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
                 const AppEntry* __restrict__ apps, int n_slots, McCensus* __restrict__ census, int* __restrict__ tiles) {
  __shared__ int s_cnt[kCensusWarps];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int live = min(T, __ldg(n_live_p));
  const int tile = blockIdx.x * kCensusWarps + warp;
  int slot[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int t = tile * kTileM + i * 32 + lane;
    slot[i] = t < live ? __ldg(token_slot + t) : -1;
  }
  int4 q[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    q[i] = make_int4(0, 0, 0, 0);
    if (slot[i] >= 0 && slot[i] < n_slots) q[i] = __ldg(reinterpret_cast<const int4*>(apps + slot[i]));    // valid, kind, n_classes, act
  }
  int cnt = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const bool hit = q[i].x && (q[i].y & kKindMask) == MIX_PROBE && q[i].z > 1 && q[i].z <= 32;
    cnt += __popc(__ballot_sync(0xffffffffu, hit));
  }
  if (lane == 0) s_cnt[warp] = cnt;
  __syncthreads();
  if (threadIdx.x == 0) {
    int n_local = 0, rows = 0;
#pragma unroll
    for (int w = 0; w < kCensusWarps; ++w) {
      n_local += s_cnt[w] > 0;
      rows += s_cnt[w];
    }
    if (n_local > 0) {
      int pos = atomicAdd(&census->w_tiles, n_local);
#pragma unroll
      for (int w = 0; w < kCensusWarps; ++w)
        if (s_cnt[w] > 0) tiles[pos++] = blockIdx.x * kCensusWarps + w;
      atomicAdd(&census->w_rows, rows);
    }
    __threadfence();
    if (atomicAdd(&census->w_done, 1) == (int)gridDim.x - 1) {
      const int n_tiles = atomicAdd(&census->w_tiles, 0), n_rows = atomicAdd(&census->w_rows, 0);
      census->n_tiles = n_tiles;
      census->n_rows = n_rows;
      census->use_tc = n_tiles > 0 && 2 * n_rows >= n_tiles * kTileM;
      census->w_tiles = 0;
      census->w_rows = 0;
      census->w_done = 0;
    }
  }
}

}  // namespace


bool has_multiclass_stage(const Ctx* c) {
  return c->cfg.T_max > kTeamMaxRows && c->cfg.C_max > 1 && !(c->cfg.flags & MIX_FLAG_SLOT_CHAINS);
}

cudaError_t launch_mc_census(const Ctx* c, int T, cudaStream_t s) {
  const int rows_per_cta = kCensusWarps * kTileM;
  mc_census_kernel<<<(c->cfg.T_max + rows_per_cta - 1) / rows_per_cta, kCensusWarps * 32, 0, s>>>(c->d_token_slot, c->d_n_live, T, c->d_apps,
                                                                           c->cfg.n_slots_max, c->d_mc_census, c->d_mc_tiles);
  return cudaGetLastError();
}

// The tensor-core probe kernel holds a whole SM's shared memory, as the SAE encode does: beside an encode
// it could only wait, so contexts with SAE weight sets leave every batch to the 16-row kernel.
bool has_tc_probe_stage(const Ctx* c) { return has_multiclass_stage(c) && c->cfg.n_groups_max == 0; }

cudaError_t launch_probe_steer(const Ctx* c, __nv_bfloat16* hidden, int T, float* scores, cudaStream_t s, bool allow_pdl) {
  if (c->cfg.flags & MIX_FLAG_SLOT_CHAINS) {
    return launch_pdl(allow_pdl ? kPdlHook : 0, probe_steer_chain_kernel, dim3(c->cfg.T_max), dim3(kChainWarps * 32), 0, s,
                      c->d_token_slot, c->d_n_live, T, c->d_apps, c->d_gates, c->d_chain_next, c->cfg.n_slots_max, hidden,
                      c->cfg.d_model, scores, c->cfg.C_max, c->d_status);
  } else if (c->cfg.T_max <= kTeamMaxRows) {
    const int pdl = (allow_pdl && (pdl_mask() & kPdlHook)) ? 1 : 0;
    return launch_pdl(allow_pdl ? kPdlHook : 0, probe_steer_team_kernel<8>, dim3(c->cfg.T_max), dim3(8 * 32), 0, s,
                      c->d_token_slot, c->d_n_live, T, c->d_apps, c->d_gates, c->cfg.n_slots_max, hidden, c->cfg.d_model,
                      scores, c->cfg.C_max, c->d_status, reinterpret_cast<const uint4*>(c->d_vec_arena), pdl);
  } else {
    const int blocks = (c->cfg.T_max + kWarpsPerBlock - 1) / kWarpsPerBlock;
    probe_steer_kernel<<<blocks, kWarpsPerBlock * 32, 0, s>>>(c->d_token_slot, c->d_n_live, T, c->d_apps, c->d_gates,
                                                              c->cfg.n_slots_max, hidden, c->cfg.d_model, scores,
                                                              c->cfg.C_max, c->d_status, has_multiclass_stage(c) ? 1 : 0);
  }
  return cudaGetLastError();
}

cudaError_t launch_probe_multiclass(const Ctx* c, const __nv_bfloat16* hidden, int T, float* scores, cudaStream_t s) {
  const int blocks = (c->cfg.T_max + kMcRows - 1) / kMcRows;
  probe_multiclass_kernel<<<blocks, kMcWarps * 32, 0, s>>>(c->d_token_slot, c->d_n_live, T, c->d_apps, c->d_gates,
                                                                 c->cfg.n_slots_max, hidden, c->cfg.d_model, scores,
                                                                 c->cfg.C_max, has_tc_probe_stage(c) ? c->d_mc_census : nullptr);
  return cudaGetLastError();
}

cudaError_t launch_router(const Ctx* c, float* logits, int n_experts, int T, cudaStream_t s) {
  const long long n = (long long)c->cfg.T_max * n_experts;
  router_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(c->d_token_slot, c->d_n_live, T, c->d_apps, c->d_gates,
                                                            c->cfg.n_slots_max, logits, n_experts);
  return cudaGetLastError();
}

cudaError_t launch_compose_map(const Ctx* c, int T_live, int n_req, cudaStream_t s) {
  if (T_live == 0) return cudaSuccess;
  compose_map_kernel<<<(T_live + 255) / 256, 256, 0, s>>>(c->d_tmp_req, c->d_tmp_req_slot, T_live, n_req,
                                                          c->d_token_slot);
  return cudaGetLastError();
}

cudaError_t launch_fold_bias(const __nv_bfloat16* W_enc, const float* b_enc, const float* b_dec, float* b_eff,
                             long long d_sae, int d, cudaStream_t s) {
  const unsigned blocks = (unsigned)((d_sae + 7) / 8);
  fold_bias_kernel<<<blocks, 256, 0, s>>>(W_enc, b_enc, b_dec, b_eff, d_sae, d);
  return cudaGetLastError();
}

}  // namespace mix
