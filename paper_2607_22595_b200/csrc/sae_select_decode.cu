// SAE activation / selection and sparse decode, plus the plain CUDA-core encode that serves
// as the in-library cross-check of the tensor-core encode.
//
//   select_kernel : per packed row, exact TopK of the fp32 pre-activations (radix refinement
//                   on order-preserving keys, then an in-shared-memory bitonic sort; ties go
//                   to the lower feature id), or the active count for ReLU / JumpReLU.
//   decode_kernel : per packed row, h' = base + sum_j coef_j * W_dec[j,:], where
//                   (base, coef) = (h, f'_j - f_j over edited j)        with the error term,
//                                  (b_dec, f'_j over active/edited j)   without it.
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

// ---------------------------------------------------------------------------------------
// selection
// ---------------------------------------------------------------------------------------
constexpr int kSelThreads = 512;
constexpr int kCand = 1024;        // composites sorted in shared memory (>= k_max)
constexpr int kBins = 2048;
static_assert(kCand >= kMaxK, "the sort buffer must hold a full TopK list");

// In-place bitonic sort of the first n entries of `a` (shared memory), descending.  Entries up
// to the next power of two are overwritten with 0 (the smallest composite key).
__device__ void bitonic_sort_desc(unsigned long long* a, int n) {
  const int tid = threadIdx.x;
  int n2 = 1;
  while (n2 < n) n2 <<= 1;
  for (int i = n + tid; i < n2; i += kSelThreads) a[i] = 0ull;
  __syncthreads();
  for (int size = 2; size <= n2; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = tid; i < n2 / 2; i += kSelThreads) {
        const int lo = 2 * i - (i & (stride - 1));
        const int hi = lo + stride;
        const bool desc = ((lo & size) == 0);
        const unsigned long long x = a[lo], y = a[hi];
        if ((x < y) == desc) {
          a[lo] = y;
          a[hi] = x;
        }
      }
      __syncthreads();
    }
  }
}

// Write the first k sorted composites (key << 32 | ~id) as the row's TopK lists.
__device__ void emit_topk(const unsigned long long* a, int k, int k_max, int p, int t, int* __restrict__ ws_idx,
                          float* __restrict__ ws_val, int* __restrict__ out_idx, float* __restrict__ out_val,
                          int* __restrict__ out_n_active, int* s_count) {
  const int tid = threadIdx.x;
  int pos_cnt = 0;
  for (int i = tid; i < k; i += kSelThreads) {
    const unsigned long long c = a[i];
    const int j = (int)(0xffffffffu - (unsigned)(c & 0xffffffffull));
    const float v = key2f((unsigned)(c >> 32));
    ws_idx[(size_t)p * k_max + i] = j;
    ws_val[(size_t)p * k_max + i] = v;
    if (out_idx) out_idx[(size_t)t * k_max + i] = j;
    if (out_val) out_val[(size_t)t * k_max + i] = v;
    pos_cnt += v > 0.f;
  }
  if (out_n_active) {
    if (tid == 0) *s_count = 0;
    __syncthreads();
    pos_cnt = __reduce_add_sync(0xffffffffu, pos_cnt);
    if ((tid & 31) == 0) atomicAdd(s_count, pos_cnt);
    __syncthreads();
    if (tid == 0) out_n_active[t] = *s_count;
  }
}

// Largest digit D with count(digit >= D) >= need, and the count of digits > D.  One warp, two
// levels: each lane sums a run of n_bins / 32 bins (largest digits in lane 0) and a warp scan
// finds the run where the running count reaches `need`; then the 32 lanes split that run.
__device__ void find_digit(const int* hist, int n_bins, int need, int* s_out) {
  const int lane = threadIdx.x & 31;
  const int per = n_bins / 32;                  // 64 or 32: a multiple of 4
  const int hi = n_bins - lane * per;           // this lane's run is [hi - per, hi)
  int sum = 0;
  const int4* h4 = reinterpret_cast<const int4*>(hist + hi - per);
  for (int i = 0; i < per / 4; ++i) {
    const int4 v = h4[i];
    sum += v.x + v.y + v.z + v.w;
  }
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  const int excl = incl - sum;                  // elements in bins above this lane's run
  const unsigned hit = __ballot_sync(0xffffffffu, excl < need && incl >= need);
  const int L = __ffs(hit) - 1;                 // exactly one lane (need <= total count)
  const int run_hi = n_bins - L * per;
  const int above_run = __shfl_sync(0xffffffffu, excl, L);
  // level 2: lane l takes bins run_hi - 1 - l*w .. run_hi - (l+1)*w, w = per / 32 (2 or 1), descending
  const int w = per / 32;
  int c0 = hist[run_hi - 1 - lane * w], c1 = w == 2 ? hist[run_hi - 2 - lane * w] : 0;
  int inc2 = c0 + c1;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, inc2, o);
    if (lane >= o) inc2 += y;
  }
  const int before = above_run + inc2 - (c0 + c1);     // elements in bins above this lane's bins
  if (before < need && before + c0 + c1 >= need) {
    if (before + c0 >= need) {
      s_out[0] = run_hi - 1 - lane * w;
      s_out[1] = before;
    } else {
      s_out[0] = run_hi - 2 - lane * w;
      s_out[1] = before + c0;
    }
  }
}

// The two places a row's values can come from.
struct ZRow {            // all pre-activations of the row; position = feature id
  const float* z;
  int n;
  __device__ __forceinline__ unsigned key(int i) const { return f2key(z[i]); }
  __device__ __forceinline__ unsigned id(int i) const { return (unsigned)i; }
};
struct CandRow {         // per-tile candidates of the fused encode epilogue
  const float* v;
  const int* j;
  int n;
  __device__ __forceinline__ unsigned key(int i) const { return f2key(v[i]); }
  __device__ __forceinline__ unsigned id(int i) const { return (unsigned)j[i]; }
};

struct SelShared {
  int hist[kBins];
  unsigned long long cand[kCand];
  int n, res[2], count;
};

// Append `c` to sh.cand for every thread whose `take` is set: one shared-memory atomic per warp
// (the lanes of a warp are ranked by ballot), not one per element on a single hot counter.
// Every thread of the warp must call this.
__device__ __forceinline__ void push_cand(SelShared& sh, bool take, unsigned long long c) {
  const unsigned m = __ballot_sync(0xffffffffu, take);
  if (m == 0u) return;
  const int lane = threadIdx.x & 31, leader = __ffs(m) - 1;
  int base = 0;
  if (lane == leader) base = atomicAdd(&sh.n, __popc(m));
  base = __shfl_sync(0xffffffffu, base, leader);
  if (take) {
    const int pos = base + __popc(m & ((1u << lane) - 1u));
    if (pos < kCand) sh.cand[pos] = c;
  }
}

// Collect into sh.cand (unsorted composites key << 32 | ~id) a set that contains the k largest
// entries of `src` under the order (value descending, id ascending): radix refinement on the
// order-preserving keys, up to 11 bits at a time, until what is still undecided fits the buffer.
// The first digit starts at the highest bit in which the keys differ at all (the candidates of a
// row are its largest values: they share sign, exponent and often leading mantissa bits, and a
// digit taken from those bits would put them all into a handful of bins -- thousands of atomic
// increments on the same few counters).  If more than the buffer's worth of entries tie EXACTLY
// with the k-th value:
//   ORDERED sources (position order = id order) finish with an index-ordered pass and return 2;
//   other sources return 0 (the caller falls back).
// Returns 1 in the ordinary case.  Every thread of the CTA must call this.
template <bool ORDERED, class Src>
__device__ int radix_collect(const Src& src, int k, SelShared& sh) {
  const int tid = threadIdx.x, n = src.n;
  // range of the keys
  unsigned kmin = 0xffffffffu, kmax = 0u;
  for (int i = tid; i < n; i += kSelThreads) {
    const unsigned key = src.key(i);
    kmin = min(kmin, key);
    kmax = max(kmax, key);
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if ((tid & 31) == 0) {
    sh.hist[tid >> 5] = (int)kmin;
    sh.hist[32 + (tid >> 5)] = (int)kmax;
  }
  __syncthreads();
  for (int w = 0; w < kSelThreads / 32; ++w) {
    kmin = min(kmin, (unsigned)sh.hist[w]);
    kmax = max(kmax, (unsigned)sh.hist[32 + w]);
  }
  __syncthreads();
  int hi_bit = (kmax ^ kmin) ? 32 - __clz(kmax ^ kmin) : 0;     // bits [0, hi_bit) vary; the rest is common
  unsigned prefix = hi_bit >= 32 ? 0u : (kmax >> hi_bit);       // digits fixed so far (= key >> hi_bit of the k-th)
  int need = k;                 // winners still to be found inside the prefix set
  // Refinement goes on while the undecided set is much larger than k, even if it would already fit
  // the buffer: one more histogram pass costs far less than sorting a thousand composites.
  const int enough = max(2 * k, 128);
  bool done = false;
  while (hi_bit > 0) {
    const int width = min(11, hi_bit), shift = hi_bit - width, nb = 1 << width;
    for (int b = tid; b < kBins; b += kSelThreads) sh.hist[b] = 0;     // digits >= nb do not occur: their bins stay 0
    __syncthreads();
    for (int i = tid; i < n; i += kSelThreads) {
      const unsigned key = src.key(i);
      if (hi_bit >= 32 || (key >> hi_bit) == prefix) atomicAdd(&sh.hist[(key >> shift) & (nb - 1)], 1);
    }
    __syncthreads();
    if (tid < 32) find_digit(sh.hist, kBins, need, sh.res);
    __syncthreads();
    const int D = sh.res[0], above = sh.res[1];
    const int in_bin = sh.hist[D];
    need -= above;
    prefix = (prefix << width) | (unsigned)D;
    hi_bit = shift;
    done = (k - need) + in_bin <= kCand;
    __syncthreads();
    if (done && (k - need) + in_bin <= enough) break;
  }
  if (tid == 0) sh.n = 0;
  __syncthreads();
  const int n_up = (n + kSelThreads - 1) / kSelThreads * kSelThreads;    // whole warps take part in every ballot
  if (done) {
    for (int i = tid; i < n_up; i += kSelThreads) {
      const unsigned key = i < n ? src.key(i) : 0u;
      const bool take = i < n && (key >> hi_bit) >= prefix;
      push_cand(sh, take, take ? (((unsigned long long)key << 32) | (0xffffffffu - src.id(i))) : 0ull);
    }
    __syncthreads();
    return 1;
  }
  if constexpr (!ORDERED) {
    return 0;
  } else {
  // every larger key, then the `need` lowest ids among the exact ties, in index order
  for (int i = tid; i < n_up; i += kSelThreads) {
    const unsigned key = i < n ? src.key(i) : 0u;
    const bool take = i < n && key > prefix;
    push_cand(sh, take, take ? (((unsigned long long)key << 32) | (0xffffffffu - src.id(i))) : 0ull);
  }
  __syncthreads();
  int taken = 0;               // uniform across the block
  for (int i0 = 0; i0 < n && taken < need; i0 += kSelThreads) {
    const int i = i0 + tid;
    const bool eq = i < n && src.key(i) == prefix;
    const unsigned m = __ballot_sync(0xffffffffu, eq);
    if ((tid & 31) == 0) sh.hist[tid >> 5] = __popc(m);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < kSelThreads / 32; ++w) {
      const int c = sh.hist[w];
      if (w < (tid >> 5)) before += c;
      total += c;
    }
    const int rank = taken + before + __popc(m & ((1u << (tid & 31)) - 1u));
    if (eq && rank < need) {
      const int pos = atomicAdd(&sh.n, 1);
      sh.cand[pos] = ((unsigned long long)prefix << 32) | (0xffffffffu - src.id(i));
    }
    taken += total;
    __syncthreads();
  }
  __syncthreads();
  return 2;
  }
}

// select_kernel: exact TopK of a row from the Z scratch (all rows, or only rows the merge step
// flagged), and the active count of ReLU / JumpReLU rows.
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ Z, long long ldz, const int* __restrict__ panel_row,
              const int* __restrict__ mtile_group, const RouteState* __restrict__ rs,
              const GroupEntry* __restrict__ groups, int k_max, int* __restrict__ ws_idx, float* __restrict__ ws_val,
              int* __restrict__ out_idx, float* __restrict__ out_val, int* __restrict__ out_n_active,
              unsigned* __restrict__ status, const int* __restrict__ row_flag, const int* __restrict__ n_flagged) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ SelShared sh;
  // nothing to do: no flagged TopK row, and nobody asked for the other sets' active counts
  if (row_flag != nullptr && *n_flagged == 0 && (out_n_active == nullptr || rs->n_topk_rows == rs->n_sae_rows)) return;
  const int n_rows = rs->n_panel_rows;
  for (int p = blockIdx.x; p < n_rows; p += gridDim.x) {
    const int t = panel_row[p];
    if (t < 0) continue;
    const GroupEntry ge = groups[mtile_group[p / kTileM]];
    const int S = (int)ge.d_sae;
    const float* z = Z + (size_t)p * ldz;
    const int tid = threadIdx.x;
    if (ge.act != MIX_SAE_TOPK) {
      if (out_n_active == nullptr) continue;
      int cnt = 0;
      for (int j = tid; j < S; j += kSelThreads) {
        const float v = z[j];
        const bool on = ge.act == MIX_SAE_RELU ? v > 0.f : (v > ge.theta[j] && v > 0.f);
        cnt += on;
      }
      if (tid == 0) sh.count = 0;
      __syncthreads();
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if ((tid & 31) == 0) atomicAdd(&sh.count, cnt);
      __syncthreads();
      if (tid == 0) out_n_active[t] = sh.count;
      __syncthreads();
      continue;
    }
    if (row_flag != nullptr && !row_flag[p]) continue;   // the merge step already settled this row
    ZRow src{z, S};
    const int how = radix_collect<true>(src, ge.k, sh);
    if (how == 2 && tid == 0) atomicOr(status, MIX_STATUS_TOPK_GENERAL);
    bitonic_sort_desc(sh.cand, sh.n);
    emit_topk(sh.cand, ge.k, k_max, p, t, ws_idx, ws_val, out_idx, out_val, out_n_active, &sh.count);
    __syncthreads();
  }
}

// merge_kernel: exact TopK from the per-tile candidates of the fused encode epilogue.
// Every (row, feature tile) contributed its 8 largest pre-activations and its 9th.  The k
// largest candidates are the row's TopK unless some tile's 9th value reaches the k-th
// candidate, i.e. that tile may hide a winner (or an exact tie whose order matters).  Such rows
// are flagged; their row tiles are re-encoded to Z and selected exactly by select_kernel.
__global__ void __launch_bounds__(kSelThreads)
merge_kernel(const float* __restrict__ cand_val, const int* __restrict__ cand_idx, const float* __restrict__ cand_ninth,
             int cand_tiles, const int* __restrict__ panel_row, const int* __restrict__ mtile_group,
             const RouteState* __restrict__ rs, const GroupEntry* __restrict__ groups, int k_max,
             int* __restrict__ ws_idx, float* __restrict__ ws_val, int* __restrict__ out_idx, float* __restrict__ out_val,
             int* __restrict__ out_n_active, int* __restrict__ row_flag, int* __restrict__ mtile_flag,
             int* __restrict__ n_flagged) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ SelShared sh;
  if (rs->n_topk_rows == 0) return;                  // no TopK row routed this call
  const int n_rows = rs->n_panel_rows;
  for (int p = blockIdx.x; p < n_rows; p += gridDim.x) {
    const int t = panel_row[p];
    if (t < 0) continue;
    const GroupEntry ge = groups[mtile_group[p / kTileM]];
    if (ge.act != MIX_SAE_TOPK) continue;
    const int tid = threadIdx.x;
    const int n_tiles = (int)(ge.d_sae / kTileN);
    const int n = n_tiles * kCandPerTile, k = ge.k;
    bool flag = n < k;                               // uniform
    if (!flag) {
      CandRow src{cand_val + (size_t)p * cand_tiles * kCandPerTile, cand_idx + (size_t)p * cand_tiles * kCandPerTile, n};
      flag = radix_collect<false>(src, k, sh) == 0;
    }
    if (!flag) {
      bitonic_sort_desc(sh.cand, sh.n);
      const unsigned kth = (unsigned)(sh.cand[k - 1] >> 32);
      const float* ninth = cand_ninth + (size_t)p * cand_tiles;
      int over = 0;
      for (int i = tid; i < n_tiles; i += kSelThreads) over |= f2key(ninth[i]) >= kth;
      flag = __syncthreads_or(over) != 0;
    }
    if (flag) {
      if (tid == 0) {
        row_flag[p] = 1;
        mtile_flag[p / kTileM] = 1;
        atomicAdd(n_flagged, 1);
      }
    } else {
      emit_topk(sh.cand, k, k_max, p, t, ws_idx, ws_val, out_idx, out_val, out_n_active, &sh.count);
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------
// decode
// ---------------------------------------------------------------------------------------
constexpr int kDecThreads = 256;
constexpr int kDecList = 1024 + kMaxEdits;     // >= k_max + r_max
constexpr int kDecU = 4;                       // 16-byte column vectors per thread

__device__ __forceinline__ void axpy8(float* acc, float c, const uint4& q) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    acc[2 * i] = fmaf(c, t.x, acc[2 * i]);
    acc[2 * i + 1] = fmaf(c, t.y, acc[2 * i + 1]);
  }
}

__device__ __forceinline__ void accumulate_list(float (*acc)[8], const float* coef, const int* feat, int n,
                                                const __nv_bfloat16* __restrict__ W_dec, int d, int nvec) {
  const int tid = threadIdx.x;
  for (int e = 0; e < n; ++e) {
    const float c = coef[e];
    if (c == 0.f) continue;
    const uint4* row = reinterpret_cast<const uint4*>(W_dec + (size_t)feat[e] * d);
#pragma unroll
    for (int u = 0; u < kDecU; ++u) {
      const int v = tid + u * kDecThreads;
      if (v < nvec) axpy8(acc[u], c, __ldg(row + v));
    }
  }
}

constexpr int kDecRows = kDecThreads / 32;     // packed rows per CTA of decode_kernel: one per warp

// A row that keeps the error term: one warp works out f'_j - f_j for each of its edit entries and leaves
// them, with the row's slot (-1 when no edit changes anything: the row then stays bit-exact) and the
// decoder pointer, for decode_delta_kernel.
__device__ __forceinline__ void warp_edit_coefs(int p, int slot, const AppEntry& app, const GroupEntry& ge,
                                                const float* __restrict__ z, const int* __restrict__ K,
                                                const float* __restrict__ Kv, const int* __restrict__ edit_idx,
                                                const float* __restrict__ edit_val,
                                                const unsigned char* __restrict__ edit_mode, int r_max,
                                                RowDelta* __restrict__ row_delta, float* __restrict__ edit_coef,
                                                int* s_e, float* s_f, int lane) {
  const int n_edit = app.n_edit;
  for (int e = lane; e < n_edit; e += 32) {
    s_e[e] = edit_idx[slot * r_max + e];
    s_f[e] = 0.f;
  }
  __syncwarp();
  if (ge.act == MIX_SAE_TOPK) {
    // the value of a selected feature comes from the row's TopK list (the Z scratch is not written for
    // TopK sets unless the row took the fallback selection); an unselected one is 0
    for (int i = lane; i < ge.k; i += 32) {
      const int id = K[i];
      for (int e = 0; e < n_edit; ++e)
        if (s_e[e] == id) s_f[e] = fmaxf(Kv[i], 0.f);
    }
    __syncwarp();
  }
  bool any = false;
  for (int e = lane; e < n_edit; e += 32) {
    const int j = s_e[e];
    bool alive = true;                                   // a later entry for the same feature wins
    for (int e2 = e + 1; e2 < n_edit; ++e2) alive = alive && (s_e[e2] != j);
    float f;
    if (ge.act == MIX_SAE_RELU) {
      f = fmaxf(z[j], 0.f);
    } else if (ge.act == MIX_SAE_JUMPRELU) {
      const float zj = z[j];
      f = zj > ge.theta[j] ? zj : 0.f;
    } else {
      f = s_f[e];
    }
    const float fnew = edit_mode[slot * r_max + e] == MIX_EDIT_CLAMP ? edit_val[slot * r_max + e] : 0.f;
    const float delta = alive ? fnew - f : 0.f;
    edit_coef[(size_t)p * r_max + e] = delta;
    any = any || delta != 0.f;
  }
  any = __any_sync(0xffffffffu, any);
  if (lane == 0) {
    RowDelta rd;
    rd.slot = any ? slot : -1;
    rd.n_edit = n_edit;
    rd.W_dec = ge.W_dec;
    row_delta[p] = rd;
  }
}

// decode_kernel: a CTA owns `rows_per_cta` (kDecRows or 1) consecutive packed rows.  Rows that keep the error
// term only get their edit coefficients (one warp per row, all at once); rows whose app replaces the
// residual are then rebuilt one after the other by the whole CTA:  h' = b_dec + sum_j f'_j W_dec[j].
// Eight rows per CTA is the form for contexts whose apps all keep the error term (an eighth of the CTAs);
// where a replacing app is registered the launch gives every row its own CTA, so that those rows -- a
// CTA-wide gather each -- run side by side.  Either form handles every kind of row.
__global__ void __launch_bounds__(kDecThreads)
decode_kernel(__nv_bfloat16* __restrict__ hidden, int d, const float* __restrict__ Z, long long ldz,
              const int* __restrict__ panel_row, const int* __restrict__ row_slot,
              const RouteState* __restrict__ rs, const AppEntry* __restrict__ apps,
              const GroupEntry* __restrict__ groups, const int* __restrict__ edit_idx,
              const float* __restrict__ edit_val, const unsigned char* __restrict__ edit_mode, int r_max, int k_max,
              const int* __restrict__ ws_idx, const float* __restrict__ ws_val,
              RowDelta* __restrict__ row_delta, float* __restrict__ edit_coef, int rows_per_cta) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ float s_coef[kDecList];
  __shared__ int s_feat[kDecList];
  __shared__ int s_we[kDecRows][kMaxEdits];
  __shared__ float s_wf[kDecRows][kMaxEdits];
  __shared__ int s_replace[kDecRows];                  // token row of a replace-mode row, else -1
  __shared__ int s_n;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p0 = blockIdx.x * rows_per_cta;
  const int n_rows = rs->n_panel_rows;
  if (p0 >= n_rows) return;
  if (warp < rows_per_cta) {
    const int p = p0 + warp;
    const int t = p < n_rows ? panel_row[p] : -1;
    int replace_t = -1;
    if (t < 0) {
      if (p < n_rows && lane == 0) row_delta[p].slot = -1;           // padding row of a tile
    } else {
      const int slot = row_slot[t];                    // the SAE app's slot (the row's own, or the last of its chain)
      const AppEntry app = apps[slot];
      if (!app.add_error) {
        replace_t = t;
        if (lane == 0) row_delta[p].slot = -1;
      } else {
        const GroupEntry ge = groups[app.group];
        warp_edit_coefs(p, slot, app, ge, Z + (size_t)p * ldz, ws_idx + (size_t)p * k_max, ws_val + (size_t)p * k_max,
                        edit_idx, edit_val, edit_mode, r_max, row_delta, edit_coef, s_we[warp], s_wf[warp], lane);
      }
    }
    if (lane == 0) s_replace[warp] = replace_t;
  }
  __syncthreads();
  const int nvec = d >> 3;
  for (int r = 0; r < rows_per_cta; ++r) {             // CTA-uniform
    const int t = s_replace[r];
    if (t < 0) continue;
    const int p = p0 + r;
    const int slot = row_slot[t];
    const AppEntry app = apps[slot];
    const GroupEntry ge = groups[app.group];
    const int n_edit = app.n_edit;
    const int S = (int)ge.d_sae;
    const float* z = Z + (size_t)p * ldz;
    const int* K = ws_idx + (size_t)p * k_max;
    const float* Kv = ws_val + (size_t)p * k_max;
    int* s_eidx = s_we[0];                             // the per-warp scratch is free again
    if (tid == 0) s_n = 0;
    if (tid < n_edit) s_eidx[tid] = edit_idx[slot * r_max + tid];
    __syncthreads();
    // edited features contribute f' (live entries only: a later entry for the same feature wins)
    if (tid < n_edit) {
      const int j = s_eidx[tid];
      bool alive = true;
      for (int e2 = tid + 1; e2 < n_edit; ++e2) alive = alive && (s_eidx[e2] != j);
      const float fnew = edit_mode[slot * r_max + tid] == MIX_EDIT_CLAMP ? edit_val[slot * r_max + tid] : 0.f;
      s_coef[tid] = alive ? fnew : 0.f;
      s_feat[tid] = j;
    }
    float acc[kDecU][8];
    uint4* hrow = reinterpret_cast<uint4*>(hidden + (size_t)t * d);
#pragma unroll
    for (int u = 0; u < kDecU; ++u) {
      const int v = tid + u * kDecThreads;
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[u][i] = (ge.b_dec && v < nvec) ? ge.b_dec[v * 8 + i] : 0.f;
    }
    __syncthreads();
    accumulate_list(acc, s_coef, s_feat, n_edit, ge.W_dec, d, nvec);
    __syncthreads();
    if (ge.act == MIX_SAE_TOPK) {
      for (int i = tid; i < ge.k; i += kDecThreads) {
        const int j = K[i];
        bool edited = false;
        for (int e = 0; e < n_edit; ++e) edited = edited || (s_eidx[e] == j);
        // an id outside the SAE can only come from a call whose encode timed out: never address with it
        const bool in_range = (unsigned)j < (unsigned)S;
        s_coef[i] = (edited || !in_range) ? 0.f : fmaxf(Kv[i], 0.f);
        s_feat[i] = in_range ? j : 0;
      }
      __syncthreads();
      accumulate_list(acc, s_coef, s_feat, ge.k, ge.W_dec, d, nvec);
    } else {
      // dense scan of the activations in chunks; active, unedited features are compacted
      // into shared memory and applied chunk by chunk
      for (int c0 = 0; c0 < S; c0 += 1024) {
        for (int j = c0 + tid; j < min(S, c0 + 1024); j += kDecThreads) {
          const float zj = z[j];
          const float f = ge.act == MIX_SAE_RELU ? fmaxf(zj, 0.f) : (zj > ge.theta[j] ? zj : 0.f);
          if (f != 0.f) {
            bool edited = false;
            for (int e = 0; e < n_edit; ++e) edited = edited || (s_eidx[e] == j);
            if (!edited) {
              const int pos = atomicAdd(&s_n, 1);
              s_coef[pos] = f;
              s_feat[pos] = j;
            }
          }
        }
        __syncthreads();
        accumulate_list(acc, s_coef, s_feat, s_n, ge.W_dec, d, nvec);
        __syncthreads();
        if (tid == 0) s_n = 0;
        __syncthreads();
      }
    }
#pragma unroll
    for (int u = 0; u < kDecU; ++u) {
      const int v = tid + u * kDecThreads;
      if (v < nvec) {
        uint4 q;
        __nv_bfloat162* pp = reinterpret_cast<__nv_bfloat162*>(&q);
#pragma unroll
        for (int i = 0; i < 4; ++i) pp[i] = __floats2bfloat162_rn(acc[u][2 * i], acc[u][2 * i + 1]);
        hrow[v] = q;
      }
    }
    __syncthreads();                                   // the shared lists are reused by the next row
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

// decode_kernel has already left, per packed row, the slot (or -1 when there is nothing to add), the
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

// one CTA per packed row, but never more than a few waves: rows are walked grid-stride
static int row_grid(const Ctx* c) {
  const int cap = (c->n_sms > 0 ? c->n_sms : 148) * 8;
  return c->panel_rows_cap < cap ? c->panel_rows_cap : cap;
}

cudaError_t launch_encode_simt(const Ctx* c, cudaStream_t s) {
  dim3 grid((unsigned)(c->cfg.d_sae_max / 64), (unsigned)(c->panel_rows_cap / 64));
  return launch_pdl(kPdlEncode, encode_simt_kernel, dim3(grid), dim3(256), 0, s, c->d_panel, c->d_mtile_group, c->d_route, c->d_groups, c->d_z,
                                          c->cfg.d_sae_max, c->cfg.d_model);
}

cudaError_t launch_merge(const Ctx* c, cudaStream_t s) {
  return launch_pdl(kPdlTail, merge_kernel, dim3(row_grid(c)), dim3(kSelThreads), 0, s, c->d_cand_val, c->d_cand_idx, c->d_cand_ninth, c->cand_tiles,
                                                         c->d_panel_row, c->d_mtile_group, c->d_route, c->d_groups,
                                                         c->cfg.k_max, c->d_topk_idx, c->d_topk_val, c->out_topk_idx,
                                                         c->out_topk_val, c->out_n_active, c->d_row_flag,
                                                         c->d_mtile_flag, c->d_n_flagged);
}

cudaError_t launch_select(const Ctx* c, bool flagged_only, cudaStream_t s) {
  return launch_pdl(kPdlTail, select_kernel, dim3(row_grid(c)), dim3(kSelThreads), 0, s, c->d_z, c->cfg.d_sae_max, c->d_panel_row,
                                                          c->d_mtile_group, c->d_route, c->d_groups, c->cfg.k_max,
                                                          c->d_topk_idx, c->d_topk_val, c->out_topk_idx,
                                                          c->out_topk_val, c->out_n_active, c->d_status,
                                                          flagged_only ? c->d_row_flag : nullptr, c->d_n_flagged);
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

// Two kernels: decode_kernel rebuilds the rows whose app replaces the residual and, for the rows that keep
// the error term, only works out the coefficients of their edits; decode_delta_kernel then adds those
// rows' deltas, eight rows per CTA.  decode_kernel's rows per CTA follow from the apps registered when the
// call is enqueued (or captured): eight where every SAE app keeps the error term, one as soon as a
// replacing app exists (the sae_static path, whose context keeps no host copy of the app table, takes one).
cudaError_t launch_decode(const Ctx* c, __nv_bfloat16* hidden, cudaStream_t s) {
  bool replacing = c->h_apps == nullptr;
  for (int i = 0; c->h_apps != nullptr && i < c->cfg.n_slots_max; ++i)
    replacing = replacing || (c->h_apps[i].valid && (c->h_apps[i].kind & kKindMask) == MIX_SAE && !c->h_apps[i].add_error);
  const int rows_per_cta = replacing ? 1 : kDecRows;
  return launch_pdl(kPdlTail, decode_kernel, dim3((c->panel_rows_cap + rows_per_cta - 1) / rows_per_cta), dim3(kDecThreads), 0, s,
                    hidden, c->cfg.d_model, c->d_z, c->cfg.d_sae_max, c->d_panel_row, c->d_row_slot, c->d_route, c->d_apps,
                    c->d_groups, c->d_edit_idx, c->d_edit_val, c->d_edit_mode, c->cfg.r_max, c->cfg.k_max, c->d_topk_idx,
                    c->d_topk_val, c->d_row_delta, c->d_edit_coef, rows_per_cta);
}

cudaError_t launch_decode_delta(const Ctx* c, __nv_bfloat16* hidden, cudaStream_t s) {
  dim3 grid((unsigned)((c->panel_rows_cap + kDdRows - 1) / kDdRows),
            (unsigned)((c->cfg.d_model / 8 + kDdThreads - 1) / kDdThreads));
  return launch_pdl(kPdlTail, decode_delta_kernel, dim3(grid), dim3(kDdThreads), 0, s, hidden, c->cfg.d_model, c->d_panel_row, c->d_route, c->d_row_delta,
                                                  c->d_edit_coef, c->d_edit_idx, c->cfg.r_max, 0);
}

}  // namespace mix
