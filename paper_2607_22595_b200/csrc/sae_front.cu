// Front of the SAE chain: slot routing and the row pack in ONE launch.
//
// Routing is integer work on the slot map: which rows carry an SAE app, of which weight set, and where each of
// them goes in the packed panel (weight set by weight set, ascending token order inside a set, every set
// starting on a 128-row tile).  The kernel does it as a chunked scan inside one grid -- every CTA classifies 256
// token rows and publishes their counts, every CTA then reads the small count table -- and packs the rows right
// after, each CTA the eight panel rows it owns, found through the published per-row records.  The only waiting
// between CTAs is a bounded wait for the published chunks; see front_kernel.
//
// Pack forms: the bf16 row as it is; with an 8-bit encoder the row as E4M3 codes with a power-of-two row
// scale -- quantised (MIX_FLAG_FP8_ACT), or split exactly into two E4M3 operands hi + lo.
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "mix_internal.h"
#include "row_lookup.cuh"

namespace mix {

namespace {

constexpr int kFrontThreads = 256;        // = token rows a CTA classifies
constexpr int kFrontWarps = kFrontThreads / 32;   // = panel rows a CTA packs

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
  for (int i = lane; i < nvec; i += 256) {               // eight loads in flight per lane, the ragged end included
    uint4 q[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (i + 32 * u < nvec) q[u] = __ldg(src + i + 32 * u);
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (i + 32 * u < nvec) dst[i + 32 * u] = q[u];
  }
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
  // exchange between the CTAs of one launch
  int2* row_meta;          // [T_max] per token row: (weight set + 1) | edit count << 8 | error-term flag << 16 (0: not an SAE row), slot
  int* counts;             // [chunks][n_groups + 1] SAE rows per weight set in each chunk of 256 token rows; last column: delta-role rows
  int* sync;               // [0] chunks published so far in this call, [1] CTAs of this call that are done (both back to 0 when the call ends)
  // routing results (written)
  int* panel_row;
  RowRec* row_rec;
  int panel_cap;
  int* mtile_group;
  RouteState* rs;
  unsigned* status;
  int* row_flag;
  int* mtile_flag;
  int* n_flagged;
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
  int pair_mode;             // 0: the encode runs on single CTAs, 1: on CTA pairs, 2: decided here from the routing result
};

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

constexpr long long kFrontWaitCycles = 2000000000ll;   // ~1 s: cap of the wait for the other CTAs' chunks

// One launch, three steps, no CTA doing another's work:
//   1. CTA c < chunks classifies token rows [256 c, 256 c + 256) -- slot -> app entry -> SAE row of which weight set --
//      and PUBLISHES the chunk: per-row records, per-set counts, then one more on the call's counter of published chunks.
//   2. Every CTA waits (one thread polls, bounded) until the counter says all chunks are there, reads the small count table and scans it: totals
//      per weight set, the sets' first panel rows, and for every chunk the rank of its first row within each set.
//      The publishing CTAs never wait before they publish, and CTAs are dispatched in index order, so whoever waits,
//      waits for work that is already running.
//   3. CTA b packs panel rows [8 b, 8 b + 8), one per warp: the row's set and rank follow from its position, the
//      chunk that holds that rank from the scan, the token from that chunk's published records.
// CTA 0 alone writes what exists once (the routing result the encode reads, the tile -> weight-set map, the
// conditional handle).  The last CTA of the launch to leave puts the two counters back to zero for the next call.
// kPack: 0 the bf16 row, 1 E4M3 hi + lo (exact split), 2 E4M3 quantised.
template <int kPack>
__global__ void __launch_bounds__(kFrontThreads)
front_kernel(const FrontArgs a) {
  extern __shared__ int s_tab[];                      // [chunks][n_groups + 1]: counts, then exclusive prefixes over the chunks
  __shared__ int s_total[kMaxGroups + 1], s_base[kMaxGroups + 1];
  __shared__ int s_gact[kMaxGroups], s_gtiles[kMaxGroups];   // per weight set: activation, feature tiles (0: not registered)
  __shared__ const __nv_bfloat16* s_gwdec[kMaxGroups];
  __shared__ const float* s_gtheta[kMaxGroups];
  __shared__ int s_wcnt[kFrontWarps][kMaxGroups + 1];
  __shared__ int s_n_panel_rows;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x;
  const bool first_cta = cta == 0;
  const int n_groups = a.n_groups, n_slots = a.n_slots, ncol = n_groups + 1;
  const int n_chunks = (a.T + kFrontThreads - 1) / kFrontThreads;     // the same in every CTA: who publishes is fixed by the launch
  phase_stamp(a.clk, 0, first_cta && tid == 0);
  if (tid < n_groups) {                                // requested now, needed after the first barrier
    const bool valid = __ldg(&a.groups[tid].valid) != 0;
    s_gact[tid] = __ldg(&a.groups[tid].act);
    s_gtiles[tid] = valid ? (int)(__ldg(&a.groups[tid].d_sae) / kTileN) : 0;
    s_gwdec[tid] = a.groups[tid].W_dec;
    s_gtheta[tid] = a.groups[tid].theta;
  }
  // ---- step 1: classify and publish one chunk
  if (cta < n_chunks) {
    const int t = cta * kFrontThreads + tid;
    const int n_live = min(a.T, __ldg(a.n_live_p));   // both loads issue together
    int slot = t < a.T ? __ldg(a.token_slot + t) : -1;
    if (t >= n_live || slot >= n_slots) slot = -1;
    int2 q0 = make_int2(0, 0);                         // valid, kind
    int g = -1, n_edit = 0, add_error = 0;
    if (slot >= 0) {
      const AppEntry* e = a.apps + slot;
      q0 = __ldg(reinterpret_cast<const int2*>(e));
      g = __ldg(&e->group);
      const int2 ne = __ldg(reinterpret_cast<const int2*>(&e->n_edit));
      n_edit = ne.x;
      add_error = ne.y != 0;
    }
    // a row whose slot starts a chain is an SAE row if the chain ends in an SAE app: follow the links
    if (q0.x && (q0.y & kKindChained) && (q0.y & kKindMask) != MIX_SAE) {
      int s2 = slot;
      int2 h2 = q0;
      for (int depth = 1; depth < kMaxChain && s2 >= 0; ++depth) {
        s2 = (h2.y & kKindChained) ? __ldg(a.chain_next + s2) : -1;
        if (s2 < 0 || s2 >= n_slots) { s2 = -1; break; }
        h2 = __ldg(reinterpret_cast<const int2*>(a.apps + s2));
        if (!h2.x) { s2 = -1; break; }
        if ((h2.y & kKindMask) == MIX_SAE) break;
      }
      if (s2 >= 0 && (h2.y & kKindMask) != MIX_SAE) s2 = -1;
      slot = s2;
      q0 = s2 >= 0 ? h2 : make_int2(0, 0);
      if (s2 >= 0) {
        g = __ldg(&a.apps[s2].group);
        n_edit = __ldg(&a.apps[s2].n_edit);
        add_error = __ldg(&a.apps[s2].add_error) != 0;
      }
    }
    __syncthreads();                                   // the weight-set table is in shared memory
    int meta = 0, is_delta = 0;
    if (q0.x && (q0.y & kKindMask) == MIX_SAE) {
      if (g < 0 || g >= n_groups || s_gtiles[g] == 0) {
        atomicOr(a.status, MIX_STATUS_BAD_GROUP);
      } else if (a.edit_only && add_error && s_gact[g] != MIX_SAE_TOPK) {
        // handled by sae_edit_only_kernel: with the error term on, a ReLU / JumpReLU row needs
        // only the pre-activations of its edited features, not the whole encode
      } else if (!(q0.y & kKindGated) || gate_open(a.gates, slot, t)) {
        meta = (g + 1) | (n_edit << 8) | (add_error << 16);
        is_delta = add_error && n_edit > 0 && s_gact[g] != MIX_SAE_TOPK;
      }
    }
    if (t < a.T) a.row_meta[t] = make_int2(meta, slot);
    const int grp = (meta & 0xff) - 1;
    for (int q = 0; q < n_groups; ++q) {
      const unsigned m = __ballot_sync(0xffffffffu, grp == q);
      if (lane == 0) s_wcnt[warp][q] = __popc(m);
    }
    {
      const unsigned m = __ballot_sync(0xffffffffu, is_delta != 0);
      if (lane == 0) s_wcnt[warp][n_groups] = __popc(m);
    }
    __syncthreads();
    if (tid < ncol) {
      int sum = 0;
#pragma unroll
      for (int w = 0; w < kFrontWarps; ++w) sum += s_wcnt[w][tid];
      a.counts[cta * ncol + tid] = sum;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) atomicAdd(a.sync, 1);                // (fence above + this: the chunk is published)
  } else {
    __syncthreads();                                   // (the weight-set table)
  }
  phase_stamp(a.clk, 1, first_cta && tid == 0);
  // ---- step 2: wait for every chunk, scan the counts
  bool ok = true;
  if (tid == 0 && ld_acquire(a.sync) < n_chunks) {     // one polling thread per CTA, backing off: a thousand CTAs ask about one word
    const long long t0 = clock64();
    unsigned ns = 32;
    while (ld_acquire(a.sync) < n_chunks) {
      if (clock64() - t0 > kFrontWaitCycles) { ok = false; break; }
      __nanosleep(ns);
      if (ns < 256) ns *= 2;
    }
  }
  ok = __syncthreads_and(ok) != 0;
  if (ok) {
    for (int i = tid; i < n_chunks * ncol; i += kFrontThreads) s_tab[i] = __ldcg(a.counts + i);   // (never through L1: written by other SMs)
    __syncthreads();
    for (int q = warp; q < ncol; q += kFrontWarps) {   // exclusive scan over the chunks, one column per warp
      int carry = 0;
      for (int c0 = 0; c0 < n_chunks; c0 += 32) {
        const int c = c0 + lane;
        const int v = c < n_chunks ? s_tab[c * ncol + q] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += y;
        }
        if (c < n_chunks) s_tab[c * ncol + q] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) s_total[q] = carry;
    }
    __syncthreads();
    phase_stamp(a.clk, 2, first_cta && tid == 0);
    if (tid == 0) {
      int mt = 0, tiles = 0, rows = 0, topk_rows = 0;
      long long cost_single = 0, cost_pair = 0, cost_split = 0;
      int live_mask = 0, split_mask = 0, n_even = 0, n_odd3 = 0;
      for (int q = 0; q < n_groups; ++q) {
        s_base[q] = mt * kTileM;
        const int m_tiles = (s_total[q] + kTileM - 1) / kTileM;
        if (first_cta) {
          a.rs->group_count[q] = s_total[q];
          a.rs->group_mtile0[q] = mt;
          a.rs->group_tile0[q] = tiles;
          for (int m = 0; m < m_tiles; ++m) a.mtile_group[mt + m] = q;
        }
        mt += m_tiles;
        rows += s_total[q];
        if (s_total[q] > 0 && s_gact[q] == MIX_SAE_TOPK) topk_rows += s_total[q];
        tiles += s_total[q] > 0 ? m_tiles * s_gtiles[q] : 0;
        if (s_total[q] > 0) {
          // per feature tile, in units of 1/40 of the time the W_enc tile takes to stream from HBM (measured on one
          // weight set with 64 ... 1024 rows): single CTAs stream at the full rate for one row tile, and from two row
          // tiles on every further tile costs 25 -- each of them fetches the W_enc tile again, from L2; a pair costs 46
          // per 256-row tile whether its second half has rows or not, streaming at a slightly lower rate
          const long long cs = (long long)(m_tiles == 1 ? 40 : 25 * m_tiles) * s_gtiles[q];
          const long long cp = (long long)(46 * ((m_tiles + 1) / 2)) * s_gtiles[q];
          cost_single += cs;
          cost_pair += cp;
          cost_split += min(cs, cp);
          live_mask |= 1 << q;
          if (cp < cs) {
            split_mask |= 1 << q;
            ++n_even;
          } else if (m_tiles >= 3) {
            ++n_odd3;
          }
        }
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
        a.rs->n_delta_rows = s_total[n_groups];
        // Pairs win where a weight set has an even number of row tiles (two tiles share one fetch of W_enc, and the
        // pair's instruction fills less shared memory per flop) and lose where half of a pair would repeat the other
        // half's work: one row tile, or three.  Each weight set may go to the form that is cheaper for it -- the two
        // encode kernels then both work, one after the other, which costs a second ramp-up and drain (about 25 us:
        // in the units above 25 x 40 / (time to stream one tile of 512 d bytes at 6.3 TB/s) = 1.23e7 / d).
        // Measured on config 4's replays, the split pays when two or more sets go to the pairs, or when a set of
        // three or more row tiles stays with the single CTAs; ONE two-tile set among one-tile sets does not: inside
        // the single-CTA kernel its second fetch of each W_enc tile and its tensor time hide behind the other sets'
        // streams (1.67 ms all single against 1.71-1.74 ms split for sets of 1, 1, 1, 1, 2 tiles), so such a call
        // stays with one form.
        int mask = a.pair_mode == 1 ? live_mask : 0;
        if (a.pair_mode == 2) {
          const bool both = split_mask != 0 && split_mask != live_mask;
          const long long split_total = cost_split + (both ? 12300000ll / max(a.d, 1) : 0ll);
          const bool split_pays = !both || n_even >= 2 || n_odd3 >= 1;
          if (split_pays && split_total <= min(cost_single, cost_pair)) mask = split_mask;
          else mask = cost_pair < cost_single ? live_mask : 0;
        }
        a.rs->pair_mask = mask;
        a.rs->use_pair = mask != 0;
        if (a.n_flagged) *a.n_flagged = 0;       // fallback-selection flags of the fused TopK path start clear every call
        // graph-conditional form: the rest of the SAE chain sits in the body of an IF node that runs only when a row needs it
        if (a.use_cond) cudaGraphSetConditional(a.cond, rows > 0 ? 1u : 0u);
      }
    }
    if (first_cta && a.mtile_flag)
      for (int m = tid; m < a.panel_cap / kTileM; m += kFrontThreads) a.mtile_flag[m] = 0;
    __syncthreads();
    phase_stamp(a.clk, 3, first_cta && tid == 0);
    // ---- step 3: this CTA's panel rows, one per warp
    const int p = cta * kFrontWarps + warp;
    if (p < a.panel_cap) {
      int t = -1, meta = 0, slot = -1;
      if (p < s_n_panel_rows) {
        int g = 0;
        while (g + 1 < n_groups && p >= s_base[g + 1]) ++g;
        const int r = p - s_base[g];                   // rank of the row within its weight set
        if (r < s_total[g]) {
          // the chunk that holds rank r: the last one whose first rank is <= r
          int c_hit = 0;
          for (int c0 = 0; c0 < n_chunks; c0 += 32) {
            const int c = c0 + lane;
            const unsigned m = __ballot_sync(0xffffffffu, c < n_chunks && s_tab[c * ncol + g] <= r);
            if (m) c_hit = c0 + 31 - __clz(m);
          }
          int left = r - s_tab[c_hit * ncol + g];      // rank inside the chunk
          int2 mm[kFrontThreads / 32];
#pragma unroll
          for (int i = 0; i < kFrontThreads / 32; ++i) {
            const int tt = c_hit * kFrontThreads + i * 32 + lane;
            mm[i] = tt < a.T ? __ldcg(a.row_meta + tt) : make_int2(0, -1);
          }
          bool found = false;
#pragma unroll
          for (int i = 0; i < kFrontThreads / 32; ++i) {
            const unsigned m = __ballot_sync(0xffffffffu, (mm[i].x & 0xff) - 1 == g);
            const int cnt = __popc(m);
            if (!found) {
              if (left < cnt) {
                const int src = __fns(m, 0, left + 1);
                t = c_hit * kFrontThreads + i * 32 + src;
                meta = __shfl_sync(0xffffffffu, mm[i].x, src);
                slot = __shfl_sync(0xffffffffu, mm[i].y, src);
                found = true;
              } else {
                left -= cnt;
              }
            }
          }
        }
        if (a.tau_slots) {                               // the encode's TopK bound starts empty
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
        const int g = (meta & 0xff) - 1;
        rec.t = t;
        rec.slot = t >= 0 ? slot : -1;
        rec.n_edit = (meta >> 8) & 0xff;
        rec.group_flags = t >= 0 ? (g | ((meta >> 16) & 1 ? kRecAddError : 0) | (s_gact[g] << kRecActShift)) : 0;
        rec.W_dec = t >= 0 ? s_gwdec[g] : nullptr;
        rec.theta = t >= 0 ? s_gtheta[g] : nullptr;
        a.row_rec[p] = rec;
        a.panel_row[p] = t;
        if (a.row_flag) a.row_flag[p] = 0;
      }
    }
  } else if (tid == 0) {
    atomicOr(a.status, MIX_STATUS_WAIT_TIMEOUT);
  }
  phase_stamp(a.clk, 4, first_cta && tid == 0);
  // Only now may the encode's CTAs be scheduled (where it is launched programmatically): they take most of an SM's
  // registers and shared memory, and resident any earlier they would crowd out the CTAs that still have rows to pack.
  pdl_launch_dependents();
  // the last CTA to leave closes the call: both counters are zero again when the next launch starts
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    if (atomicAdd(a.sync + 1, 1) == (int)gridDim.x - 1) {
      a.sync[0] = 0;
      a.sync[1] = 0;
    }
  }
}

}  // namespace

int front_chunks(int T_max) { return (T_max + kFrontThreads - 1) / kFrontThreads; }

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
  a.row_meta = c->d_row_meta;
  a.counts = c->d_front_counts;
  a.sync = c->d_front_sync;
  a.panel_row = c->d_panel_row;
  a.row_rec = c->d_row_rec;
  a.panel_cap = c->panel_rows_cap;
  a.mtile_group = c->d_mtile_group;
  a.rs = c->d_route;
  a.status = c->d_status;
  a.row_flag = c->d_row_flag;
  a.mtile_flag = c->d_mtile_flag;
  a.n_flagged = c->d_n_flagged;
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
  a.pair_mode = ((c->cfg.flags & MIX_FLAG_ENCODE_SIMT) || !encode_pair_possible(c)) ? 0 : encode_pair_mode(-1);
  const int chunks = front_chunks(T);
  const size_t smem = (size_t)front_chunks(c->cfg.T_max) * (c->cfg.n_groups_max + 1) * sizeof(int);
  const int pack_ctas = (c->panel_rows_cap + kFrontWarps - 1) / kFrontWarps;
  const dim3 grid(chunks > pack_ctas ? chunks : pack_ctas);
  if (c->cfg.flags & MIX_FLAG_FP8_ACT)
    front_kernel<2><<<grid, kFrontThreads, smem, s>>>(a);
  else if (c->cfg.flags & MIX_FLAG_FP8_W_ENC)      // hi codes in rows [0, P), lo codes in rows [P, 2P) of the same buffer
    front_kernel<1><<<grid, kFrontThreads, smem, s>>>(a);
  else
    front_kernel<0><<<grid, kFrontThreads, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace mix
