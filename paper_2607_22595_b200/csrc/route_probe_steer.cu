// Slot routing, the read (probe) and write (steering) primitives, and the SAE row pack.
//
// probe_steer_kernel is the bandwidth kernel of the hook: one warp per token row, 16-byte
// loads, fp32 FMA, shuffle reductions.  A row whose slot is -1 costs one 4-byte load.
#include "mix_internal.h"

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

// h + alpha v for one row; nvec = d / 8 16-byte vectors.
__device__ __forceinline__ void steer_row(uint4* __restrict__ h, const uint4* __restrict__ v, float alpha,
                                          int nvec, int lane) {
  constexpr int U = 4;
  int i = lane;
  for (; i + (U - 1) * 32 < nvec; i += U * 32) {
    uint4 hq[U], vq[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      hq[u] = __ldcs(h + i + u * 32);
      vq[u] = __ldg(v + i + u * 32);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float a[8], b[8];
      unpack8(hq[u], a);
      unpack8(vq[u], b);
#pragma unroll
      for (int e = 0; e < 8; ++e) a[e] = fmaf(alpha, b[e], a[e]);
      __stcs(h + i + u * 32, pack8(a));
    }
  }
  for (; i < nvec; i += 32) {
    float a[8], b[8];
    unpack8(__ldcs(h + i), a);
    unpack8(__ldg(v + i), b);
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = fmaf(alpha, b[e], a[e]);
    __stcs(h + i, pack8(a));
  }
}

// NC logits of one row against NC consecutive probe rows; every lane returns the full sums.
template <int NC>
__device__ __forceinline__ void probe_dots(const uint4* __restrict__ h, const uint4* __restrict__ W, int nvec,
                                           int nc, int lane, float* out) {
  float acc[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) acc[c] = 0.f;
  constexpr int U = (NC == 1) ? 4 : 1;
  int i = lane;
  for (; i + (U - 1) * 32 < nvec; i += U * 32) {
    uint4 hq[U];
#pragma unroll
    for (int u = 0; u < U; ++u) hq[u] = __ldg(h + i + u * 32);
    uint4 wq[U][NC];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int c = 0; c < NC; ++c)
        if (c < nc) wq[u][c] = __ldg(W + (size_t)c * nvec + i + u * 32);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float a[8];
      unpack8(hq[u], a);
#pragma unroll
      for (int c = 0; c < NC; ++c)
        if (c < nc) {
          float b[8];
          unpack8(wq[u][c], b);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[c] = fmaf(a[e], b[e], acc[c]);
        }
    }
  }
  if (U > 1) {
    for (; i < nvec; i += 32) {
      float a[8], b[8];
      unpack8(__ldg(h + i), a);
      unpack8(__ldg(W + i), b);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[0] = fmaf(a[e], b[e], acc[0]);
    }
  }
#pragma unroll
  for (int c = 0; c < NC; ++c) out[c] = warp_sum(acc[c]);
}

constexpr int kWarpsPerBlock = 8;

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
probe_steer_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
                   const AppEntry* __restrict__ apps, int n_slots, __nv_bfloat16* __restrict__ hidden, int d,
                   float* __restrict__ scores, int C_max, unsigned* __restrict__ status) {
  __shared__ float s_logit[kWarpsPerBlock][kMaxClasses];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  const int n_live = min(T, __ldg(n_live_p));
  if (t >= n_live) return;
  const int s = __ldg(token_slot + t);
  if (s == -1) return;
  if (s < -1 || s >= n_slots) {
    if (lane == 0) atomicOr(status, MIX_STATUS_BAD_SLOT);
    return;
  }
  const AppEntry* e = apps + s;
  const int4 head = __ldg(reinterpret_cast<const int4*>(e));   // valid, kind, n_classes, act
  if (!head.x) {
    if (lane == 0) atomicOr(status, MIX_STATUS_BAD_SLOT);
    return;
  }
  const int nvec = d >> 3;
  uint4* hrow = reinterpret_cast<uint4*>(hidden + (size_t)t * d);
  if (head.y == MIX_STEER) {
    const float alpha = __ldg(&e->alpha);
    if (alpha == 0.f) return;                 // identity, and keeps the row bit-exact (-0.0 stays -0.0)
    steer_row(hrow, reinterpret_cast<const uint4*>(__ldg(reinterpret_cast<const unsigned long long*>(&e->W))),
              alpha, nvec, lane);
    return;
  }
  if (head.y != MIX_PROBE || scores == nullptr) return;
  const int C = head.z, act = head.w;
  const uint4* W = reinterpret_cast<const uint4*>(__ldg(reinterpret_cast<const unsigned long long*>(&e->W)));
  const float* b = reinterpret_cast<const float*>(__ldg(reinterpret_cast<const unsigned long long*>(&e->b)));
  float* out = scores + (size_t)t * C_max;
  if (C == 1) {
    float z;
    probe_dots<1>(hrow, W, nvec, 1, lane, &z);
    if (lane == 0) {
      if (b) z += __ldg(b);
      out[0] = (act == MIX_ACT_NONE) ? z : 1.f / (1.f + expf(-z));
    }
    return;
  }
  for (int c0 = 0; c0 < C; c0 += 8) {
    float z[8];
    const int nc = min(8, C - c0);
    probe_dots<8>(hrow, W + (size_t)c0 * nvec, nvec, nc, lane, z);
    if (lane == 0) {
#pragma unroll
      for (int c = 0; c < 8; ++c)
        if (c < nc) s_logit[warp][c0 + c] = z[c] + (b ? __ldg(b + c0 + c) : 0.f);
    }
  }
  __syncwarp();
  // C <= 64: lane handles classes lane and lane + 32
  float z0 = lane < C ? s_logit[warp][lane] : -INFINITY;
  float z1 = lane + 32 < C ? s_logit[warp][lane + 32] : -INFINITY;
  if (act == MIX_ACT_SOFTMAX) {
    float m = fmaxf(z0, z1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float e0 = lane < C ? expf(z0 - m) : 0.f;
    float e1 = lane + 32 < C ? expf(z1 - m) : 0.f;
    float sum = warp_sum(e0 + e1);
    z0 = e0 / sum;
    z1 = e1 / sum;
  } else if (act == MIX_ACT_SIGMOID) {
    z0 = 1.f / (1.f + expf(-z0));
    z1 = 1.f / (1.f + expf(-z1));
  }
  if (lane < C) out[lane] = z0;
  if (lane + 32 < C) out[lane + 32] = z1;
}

// ---------------------------------------------------------------------------------------
// SAE routing: one CTA builds, in ascending row order, the packed-panel position of every
// SAE row, the per-group counts and the encode tile schedule.  Integer work only.
// ---------------------------------------------------------------------------------------
constexpr int kRouteThreads = 1024;
constexpr int kRouteWarps = kRouteThreads / 32;

__global__ void __launch_bounds__(kRouteThreads)
route_kernel(const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
             const AppEntry* __restrict__ apps, int n_slots, const GroupEntry* __restrict__ groups, int n_groups,
             int* __restrict__ panel_row, int panel_cap, int* __restrict__ mtile_group, RouteState* __restrict__ rs,
             unsigned* __restrict__ status) {
  extern __shared__ int s_cnt[];                      // [n_chunks * kRouteWarps][n_groups]
  __shared__ int s_total[kMaxGroups], s_base[kMaxGroups + 1];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_live = min(T, __ldg(n_live_p));
  const int n_chunks = (n_live + kRouteThreads - 1) / kRouteThreads;

  for (int p = tid; p < panel_cap; p += kRouteThreads) panel_row[p] = -1;
  for (int m = tid; m < panel_cap / kTileM; m += kRouteThreads) mtile_group[m] = -1;

  auto group_of = [&](int t) -> int {
    if (t >= n_live) return -1;
    const int s = token_slot[t];
    if (s < 0 || s >= n_slots) return -1;
    const AppEntry* e = apps + s;
    if (!e->valid || e->kind != MIX_SAE) return -1;
    const int g = e->group;
    if (g < 0 || g >= n_groups || !groups[g].valid) {
      atomicOr(status, MIX_STATUS_BAD_GROUP);
      return -1;
    }
    return g;
  };

  // phase A: per (chunk, warp) counts per group
  for (int c = 0; c < n_chunks; ++c) {
    const int g = group_of(c * kRouteThreads + tid);
    for (int q = 0; q < n_groups; ++q) {
      const unsigned m = __ballot_sync(0xffffffffu, g == q);
      if (lane == 0) s_cnt[(c * kRouteWarps + warp) * n_groups + q] = __popc(m);
    }
  }
  __syncthreads();
  // phase B: exclusive scan over (chunk, warp) for each group; warp q owns group q
  const int n_seg = n_chunks * kRouteWarps;
  for (int q = warp; q < n_groups; q += kRouteWarps) {
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
    int mt = 0, tiles = 0, rows = 0;
    for (int q = 0; q < n_groups; ++q) {
      s_base[q] = mt * kTileM;
      rs->group_count[q] = s_total[q];
      rs->group_mtile0[q] = mt;
      rs->group_tile0[q] = tiles;
      const int m_tiles = (s_total[q] + kTileM - 1) / kTileM;
      for (int m = 0; m < m_tiles; ++m) mtile_group[mt + m] = q;
      mt += m_tiles;
      rows += s_total[q];
      tiles += s_total[q] > 0 ? m_tiles * (int)(groups[q].d_sae / kTileN) : 0;
    }
    s_base[n_groups] = mt * kTileM;
    for (int q = n_groups; q <= kMaxGroups; ++q) {
      rs->group_mtile0[q] = mt;
      rs->group_tile0[q] = tiles;
      if (q < kMaxGroups) rs->group_count[q] = 0;
    }
    rs->n_panel_rows = mt * kTileM;
    rs->n_mtiles = mt;
    rs->n_sae_rows = rows;
    rs->total_tiles = tiles;
  }
  __syncthreads();
  // phase C: stable scatter
  for (int c = 0; c < n_chunks; ++c) {
    const int t = c * kRouteThreads + tid;
    const int g = group_of(t);
    for (int q = 0; q < n_groups; ++q) {
      const unsigned m = __ballot_sync(0xffffffffu, g == q);
      if (g == q) {
        const int pos = s_base[q] + s_cnt[(c * kRouteWarps + warp) * n_groups + q] + __popc(m & ((1u << lane) - 1u));
        panel_row[pos] = t;
      }
    }
  }
}

// Copy every routed row into the packed K-major panel (one warp per panel row).
__global__ void __launch_bounds__(256)
pack_kernel(const __nv_bfloat16* __restrict__ hidden, const int* __restrict__ panel_row,
            const RouteState* __restrict__ rs, __nv_bfloat16* __restrict__ panel, int d) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int p = blockIdx.x * 8 + warp;
  if (p >= rs->n_panel_rows) return;
  const int t = panel_row[p];
  uint4* dst = reinterpret_cast<uint4*>(panel + (size_t)p * d);
  const int nvec = d >> 3;
  if (t < 0) {   // padding rows of a tile: keep them finite
    for (int i = lane; i < nvec; i += 32) dst[i] = make_uint4(0, 0, 0, 0);
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)t * d);
  for (int i = lane; i < nvec; i += 32) dst[i] = __ldg(src + i);
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

}  // namespace

cudaError_t launch_probe_steer(const Ctx* c, __nv_bfloat16* hidden, int T, float* scores, cudaStream_t s) {
  const int blocks = (c->cfg.T_max + kWarpsPerBlock - 1) / kWarpsPerBlock;
  probe_steer_kernel<<<blocks, kWarpsPerBlock * 32, 0, s>>>(c->d_token_slot, c->d_n_live, T, c->d_apps,
                                                            c->cfg.n_slots_max, hidden, c->cfg.d_model, scores,
                                                            c->cfg.C_max, c->d_status);
  return cudaGetLastError();
}

cudaError_t launch_route(const Ctx* c, int T, cudaStream_t s) {
  const int n_chunks = (c->cfg.T_max + kRouteThreads - 1) / kRouteThreads;
  const size_t smem = (size_t)n_chunks * kRouteWarps * c->cfg.n_groups_max * sizeof(int);
  route_kernel<<<1, kRouteThreads, smem, s>>>(c->d_token_slot, c->d_n_live, T, c->d_apps, c->cfg.n_slots_max,
                                              c->d_groups, c->cfg.n_groups_max, c->d_panel_row, c->panel_rows_cap,
                                              c->d_mtile_group, c->d_route, c->d_status);
  return cudaGetLastError();
}

cudaError_t launch_pack(const Ctx* c, const __nv_bfloat16* hidden, cudaStream_t s) {
  const int blocks = (c->panel_rows_cap + 7) / 8;
  pack_kernel<<<blocks, 256, 0, s>>>(hidden, c->d_panel_row, c->d_route, c->d_panel, c->cfg.d_model);
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
