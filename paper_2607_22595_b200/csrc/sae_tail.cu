// Everything behind the SAE encode, in one launch: activation / selection, per-feature edits, sparse decode,
// error term and write-back (with a second launch of the same kernel for rows that need the exact fallback).
//
//   tail_kernel, row role (one CTA per packed row, grid-stride):
//     TopK row   : exact TopK -- from the per-tile candidates of the fused encode epilogue (radix refinement on
//                  order-preserving keys, then a sort of the few composites left; ties go to the lower feature
//                  id), or from the fp32 pre-activations Z when the encode wrote those -- then, with the list
//                  still in shared memory, the edits and the decode of the row:
//                    error term on : h' = h + sum over edited j of (f'_j - f_j) W_dec[j]
//                    error term off: h' = b_dec + sum_j f'_j W_dec[j]
//                  A row whose candidates cannot prove the TopK is flagged and left to the fallback launch.
//     other rows : the active count if asked for; rows whose app replaces the residual are rebuilt from Z.
//   tail_kernel, delta role (a CTA owns 4 consecutive packed rows x 2048 columns):
//     ReLU / JumpReLU rows that keep the error term: f_j of the edited features from Z, then the deltas.
//     Neighbouring packed rows mostly share a request, hence an edit list, so each edited W_dec row is
//     fetched once per CTA and applied to its rows with per-row coefficients.
// The two roles own disjoint rows, so they run side by side in one grid.
#include "mix_internal.h"

namespace mix {

namespace {

// ---------------------------------------------------------------------------------------
// selection
// ---------------------------------------------------------------------------------------
constexpr int kTailThreads = 256;
constexpr int kCand = 1024;        // composites sorted in shared memory (>= k_max)
constexpr int kBins = 2048;
static_assert(kCand >= kMaxK, "the sort buffer must hold a full TopK list");

// In-place bitonic sort of the first n entries of `a` (shared memory), descending.  Entries up
// to the next power of two are overwritten with 0 (the smallest composite key).
__device__ void bitonic_sort_desc(unsigned long long* a, int n) {
  const int tid = threadIdx.x;
  int n2 = 1;
  while (n2 < n) n2 <<= 1;
  for (int i = n + tid; i < n2; i += kTailThreads) a[i] = 0ull;
  __syncthreads();
  for (int size = 2; size <= n2; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = tid; i < n2 / 2; i += kTailThreads) {
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

// Largest digit D with count(digit >= D) >= need, and the count of digits > D.  One warp, two
// levels: each lane sums a run of n_bins / 32 bins (largest digits in lane 0) and a warp scan
// finds the run where the running count reaches `need`; then the 32 lanes split that run.
__device__ void find_digit(const int* hist, int n_bins, int need, int* s_out) {
  const int lane = threadIdx.x & 31;
  const int per = n_bins / 32;                  // 64 (2048 bins) or 8 (256 bins): a multiple of 4
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
  // level 2: the run's bins, descending, w = max(per / 32, 1) per lane (lanes beyond the run hold nothing)
  const int w = per >= 64 ? 2 : 1;
  const bool in_run = lane * w < per;
  const int c0 = in_run ? hist[run_hi - 1 - lane * w] : 0, c1 = (in_run && w == 2) ? hist[run_hi - 2 - lane * w] : 0;
  int inc2 = c0 + c1;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, inc2, o);
    if (lane >= o) inc2 += y;
  }
  const int before = above_run + inc2 - (c0 + c1);     // elements in bins above this lane's bins
  if (in_run && before < need && before + c0 + c1 >= need) {
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
struct CandRow {         // per-tile candidates of the fused encode epilogue, their keys staged in shared memory.
  // The id of a candidate is its POSITION in the row's candidate array: positions run tile by tile, and inside a
  // tile by decreasing value with the lower column first among equal values, so among equal keys position order
  // is feature-id order -- the tie rule -- and the feature ids are fetched for the k winners only.
  const unsigned* key_s;
  int n;
  __device__ __forceinline__ unsigned key(int i) const { return key_s[i]; }
  __device__ __forceinline__ unsigned id(int i) const { return (unsigned)i; }
};

// f(i, key, valid) for i = tid, tid + 256, ... < n_up (n_up: n rounded up to whole CTAs, so that whole warps take
// part), the keys of four steps requested before the first is used: a source in global memory is then read
// with four loads in flight per thread instead of one (a loop that mixes loads with shared-memory atomics is
// not reordered by the compiler).
template <class Src, class F>
__device__ __forceinline__ void scan_keys(const Src& src, int n, int n_up, F&& f) {
  constexpr int U = 4;
  for (int i0 = threadIdx.x; i0 < n_up; i0 += U * kTailThreads) {
    unsigned key[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * kTailThreads;
      key[u] = i < n ? src.key(i) : 0u;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * kTailThreads;
      if (i < n_up) f(i, key[u], i < n);
    }
  }
}

struct SelShared {
  __align__(16) int hist[kBins];            // radix histogram; afterwards the output of the counting sort (kBins / 2 composites)
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
// kDigitBits: bits per refinement pass.  11 for a long source (the pre-activations of a whole row: fewer passes over
// global memory); 8 for a row's candidates (a few thousand keys in shared memory: one pass nearly always settles
// them, and a 256-bin histogram is cheap to clear and to search).
// have_range: the caller already holds this thread's share of the keys' minimum and maximum in kmin / kmax.
template <bool ORDERED, int kDigitBits, class Src>
__device__ int radix_collect(const Src& src, int k, SelShared& sh, bool have_range = false, unsigned kmin = 0xffffffffu,
                             unsigned kmax = 0u, unsigned long long* clk = nullptr, bool stamp = false) {
  const int tid = threadIdx.x, n = src.n;
  const int n_up = (n + kTailThreads - 1) / kTailThreads * kTailThreads;    // whole warps take part in every ballot
  constexpr int kNb = 1 << kDigitBits;
  static_assert(kNb <= kBins && kNb % 128 == 0, "digit width");
  // range of the keys
  if (!have_range)
    scan_keys(src, n, n_up, [&](int, unsigned key, bool valid) {
      if (valid) {
        kmin = min(kmin, key);
        kmax = max(kmax, key);
      }
    });
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if ((tid & 31) == 0) {
    sh.hist[tid >> 5] = (int)kmin;
    sh.hist[32 + (tid >> 5)] = (int)kmax;
  }
  __syncthreads();
  for (int w = 0; w < kTailThreads / 32; ++w) {
    kmin = min(kmin, (unsigned)sh.hist[w]);
    kmax = max(kmax, (unsigned)sh.hist[32 + w]);
  }
  __syncthreads();
  phase_stamp(clk, 16, stamp);
  int n_pass = 0;
  int hi_bit = (kmax ^ kmin) ? 32 - __clz(kmax ^ kmin) : 0;     // bits [0, hi_bit) vary; the rest is common
  unsigned prefix = hi_bit >= 32 ? 0u : (kmax >> hi_bit);       // digits fixed so far (= key >> hi_bit of the k-th)
  int need = k;                 // winners still to be found inside the prefix set
  // Refinement goes on while the undecided set is much larger than k, even if it would already fit
  // the buffer: one more histogram pass costs far less than sorting a thousand composites.
  const int enough = max(2 * k, 128);
  bool done = false;
  while (hi_bit > 0) {
    const int width = min(kDigitBits, hi_bit), shift = hi_bit - width, nb = 1 << width;
    for (int b = tid; b < kNb; b += kTailThreads) sh.hist[b] = 0;       // digits >= nb do not occur: their bins stay 0
    __syncthreads();
    scan_keys(src, n, n_up, [&](int, unsigned key, bool valid) {
      if (valid && (hi_bit >= 32 || (key >> hi_bit) == prefix)) atomicAdd(&sh.hist[(key >> shift) & (nb - 1)], 1);
    });
    __syncthreads();
    if (tid < 32) find_digit(sh.hist, kNb, need, sh.res);
    __syncthreads();
    const int D = sh.res[0], above = sh.res[1];
    const int in_bin = sh.hist[D];
    need -= above;
    prefix = (prefix << width) | (unsigned)D;
    hi_bit = shift;
    done = (k - need) + in_bin <= kCand;
    __syncthreads();
    phase_stamp(clk, 17 + min(n_pass, 3), stamp);
    ++n_pass;
    if (done && (k - need) + in_bin <= enough) break;
  }
  if (tid == 0) sh.n = 0;
  __syncthreads();
  if (done) {
    // every thread counts its survivors, a warp reserves room for all of its lanes with one atomic, then they write
    int cnt = 0;
    scan_keys(src, n, n_up, [&](int, unsigned key, bool valid) { cnt += valid && (key >> hi_bit) >= prefix; });
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if ((tid & 31) >= o) incl += y;
    }
    int base = 0;
    if ((tid & 31) == 31 && incl > 0) base = atomicAdd(&sh.n, incl);
    int pos = __shfl_sync(0xffffffffu, base, 31) + incl - cnt;
    scan_keys(src, n, n_up, [&](int i, unsigned key, bool valid) {
      if (valid && (key >> hi_bit) >= prefix) {
        if (pos < kCand) sh.cand[pos] = ((unsigned long long)key << 32) | (0xffffffffu - src.id(i));
        ++pos;
      }
    });
    __syncthreads();
    return 1;
  }
  if constexpr (!ORDERED) {
    return 0;
  } else {
  // every larger key, then the `need` lowest ids among the exact ties, in index order
  scan_keys(src, n, n_up, [&](int i, unsigned key, bool valid) {
    const bool take = valid && key > prefix;
    push_cand(sh, take, take ? (((unsigned long long)key << 32) | (0xffffffffu - src.id(i))) : 0ull);
  });
  __syncthreads();
  int taken = 0;               // uniform across the block
  for (int i0 = 0; i0 < n && taken < need; i0 += kTailThreads) {
    const int i = i0 + tid;
    const bool eq = i < n && src.key(i) == prefix;
    const unsigned m = __ballot_sync(0xffffffffu, eq);
    if ((tid & 31) == 0) sh.hist[tid >> 5] = __popc(m);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < kTailThreads / 32; ++w) {
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


// The sh.n composites of sh.cand in descending order.  Up to one composite per thread they are sorted by
// counting (composites are distinct: the rank of one is the number of larger ones; one pass over shared memory
// and one barrier, where the bitonic network needs dozens of barriers); longer lists take the network.
// Returns where the sorted list is.  Every thread of the CTA must call this.
__device__ const unsigned long long* sort_desc(SelShared& sh) {
  const int tid = threadIdx.x, n = sh.n;
  if (n <= kTailThreads) {
    unsigned long long* out = reinterpret_cast<unsigned long long*>(sh.hist);
    if (tid < n) {
      const unsigned long long c = sh.cand[tid];
      int rank = 0;
      for (int j = 0; j < n; ++j) rank += sh.cand[j] > c;
      out[rank] = c;
    }
    __syncthreads();
    return out;
  }
  bitonic_sort_desc(sh.cand, n);
  return sh.cand;
}

__device__ __forceinline__ int comp_id(unsigned long long c) { return (int)(0xffffffffu - (unsigned)(c & 0xffffffffull)); }
__device__ __forceinline__ float comp_val(unsigned long long c) { return key2f((unsigned)(c >> 32)); }

// Read-out of a row's TopK: ids in order of decreasing pre-activation, the pre-activations, the active count.
__device__ void emit_topk(const int* ids, const float* vals, int k, int k_max, int t, int* __restrict__ out_idx,
                          float* __restrict__ out_val, int* __restrict__ out_n_active, int* s_count) {
  const int tid = threadIdx.x;
  if (out_idx == nullptr && out_val == nullptr && out_n_active == nullptr) return;
  int pos_cnt = 0;
  for (int i = tid; i < k; i += kTailThreads) {
    const float v = vals[i];
    if (out_idx) out_idx[(size_t)t * k_max + i] = ids[i];
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

// ---------------------------------------------------------------------------------------
// decode
// ---------------------------------------------------------------------------------------
constexpr int kDecList = 1024 + kMaxEdits;     // >= k_max + r_max
constexpr int kGatherBatch = 8;                // decoder rows in flight per thread

__device__ __forceinline__ void axpy8(float* acc, float c, const uint4& q) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    acc[2 * i] = fmaf(c, t.x, acc[2 * i]);
    acc[2 * i + 1] = fmaf(c, t.y, acc[2 * i + 1]);
  }
}

// The gather of the decode.  A row is rebuilt in passes of 2048 columns: thread `tid` owns the 16-byte column
// vector v = pass * 256 + tid, so one decoder row is read as 4 KiB of contiguous 16-byte loads per pass, and
// acc (8 columns) += sum_e coef[e] * W_dec[feat[e], 8v .. 8v+7] with kGatherBatch decoder rows in flight per
// thread -- the loop is bound by load latency, not arithmetic.  Entries with a zero coefficient are not fetched.
__device__ __forceinline__ void gather_list(float (&acc)[8], const float* coef, const int* feat, int n,
                                            const __nv_bfloat16* __restrict__ W_dec, int d, int v, bool in_cols) {
#pragma unroll 1
  for (int e0 = 0; e0 < n; e0 += kGatherBatch) {
    uint4 q[kGatherBatch];
    float c[kGatherBatch];
#pragma unroll
    for (int u = 0; u < kGatherBatch; ++u) {
      const int e = e0 + u;
      c[u] = e < n ? coef[e] : 0.f;
      q[u] = make_uint4(0u, 0u, 0u, 0u);
      if (c[u] != 0.f && in_cols) q[u] = __ldg(reinterpret_cast<const uint4*>(W_dec + (size_t)feat[e] * d) + v);
    }
#pragma unroll
    for (int u = 0; u < kGatherBatch; ++u) axpy8(acc, c[u], q[u]);
  }
}

__device__ __forceinline__ void load8(float (&acc)[8], const uint4& q) {
  const __nv_bfloat162* pp = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f2 = __bfloat1622float2(pp[i]);
    acc[2 * i] = f2.x;
    acc[2 * i + 1] = f2.y;
  }
}

__device__ __forceinline__ uint4 pack8(const float (&acc)[8]) {
  uint4 q;
  __nv_bfloat162* pp = reinterpret_cast<__nv_bfloat162*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) pp[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
  return q;
}

enum { kTailCand = 0, kTailZ = 1, kTailFallback = 2 };

struct TailArgs {
  __nv_bfloat16* hidden;
  int d;
  const float* Z;
  long long ldz;
  const RowRec* row_rec;
  const RouteState* rs;
  const GroupEntry* groups;
  const int* edit_idx;
  const float* edit_val;
  const unsigned char* edit_mode;
  int r_max, k_max;
  const float* cand_val;
  const int* cand_idx;
  const float* cand_ninth;
  int cand_tiles;
  int* out_idx;
  float* out_val;
  int* out_n_active;
  int* row_flag;
  int* mtile_flag;
  int* n_flagged;
  unsigned* status;
  int mode;                 // kTailCand: TopK from the encode's candidates; kTailZ: TopK from Z; kTailFallback: flagged rows only, from Z
  int n_col_slices;         // delta role: ceil(d / 2048)
  unsigned long long* clk;  // profiling aid or null
  int n_groups;
};

struct RowShared {
  SelShared sel;
  __align__(16) unsigned keys[kCandMax];  // a TopK row's candidate keys (the radix passes run on shared memory)
  GroupEntry grp[kMaxGroups];             // the weight-set table, fetched once per CTA
  float coef[kDecList];
  int feat[kDecList];
  int eidx[kMaxEdits];
  float ef[kMaxEdits];      // f_j of each edited feature before the edit
  float enew[kMaxEdits];    // f'_j
  int n_list;
  int cum[kMaxGroups + 1];  // SAE rows in the weight sets before each one: work index -> packed row, padding rows skipped
  int row0[kMaxGroups];     // first packed row of each weight set
};


// Row role.  Per row, the dependent round trips are: the row's record; then -- requested together -- the edit
// list, the candidate keys (into shared memory: the selection passes never go back to global memory) and the
// tiles' 9th values; then the winners' feature ids; then the gather.  (Prefetching the edited decoder rows into
// L2 while the selection runs was tried twice: line by line, one 128-byte line per lane, the 1024 prefetches of a
// row cost more issue time -- 3 us -- than the latency they hid; one bulk prefetch per decoder row made the
// staging step 1.5 us slower and the gather no faster.)
__device__ void tail_rows(const TailArgs& a, RowShared& sh, int n_groups) {
  const int tid = threadIdx.x;
  const int d = a.d, nvec = d >> 3;
  // the call's SAE rows, numbered through the weight sets without the padding rows of their last tiles
  constexpr int kGrpVecs = (int)(sizeof(GroupEntry) / sizeof(uint4));
  if (tid >= 32 && tid < 32 + n_groups * kGrpVecs)
    reinterpret_cast<uint4*>(sh.grp)[tid - 32] = reinterpret_cast<const uint4*>(a.groups)[tid - 32];
  if (tid == 0) {
    int cum = 0;
    for (int g = 0; g < n_groups; ++g) {
      sh.cum[g] = cum;
      sh.row0[g] = a.rs->group_mtile0[g] * kTileM;
      cum += a.rs->group_count[g];
    }
    sh.cum[n_groups] = cum;
  }
  __syncthreads();
  const int n_work = sh.cum[n_groups];
  // A call with few rows leaves most of the grid without work while each row's gather runs with one CTA's worth
  // of loads in flight (32 KiB, i.e. about 30 GB/s at DRAM latency).  Where the grid has room, 2 or 4 CTAs take a
  // TopK row together: each repeats the selection for itself -- a few KB of candidates out of L2 -- and gathers
  // every 2nd or 4th pass of 2048 columns; the first of them writes what exists once per row (read-out, flags).
  int n_split = 1;
  if (n_work > 0 && a.mode != kTailFallback) {
    const int room = (int)gridDim.x / n_work, passes = (nvec + kTailThreads - 1) / kTailThreads;
    while (n_split < 4 && 2 * n_split <= room && 2 * n_split <= passes) n_split *= 2;
  }
  for (int item = blockIdx.x; item < n_work * n_split; item += gridDim.x) {
    const int w = item / n_split, part = item - w * n_split;
    int g_w = 0;
    while (g_w + 1 < n_groups && w >= sh.cum[g_w + 1]) ++g_w;
    const int p = sh.row0[g_w] + (w - sh.cum[g_w]);
    const bool stamp = item == 0 && tid == 0 && a.mode != kTailFallback;
    phase_stamp(a.clk, 9, stamp);
    const RowRec rec = a.row_rec[p];
    const int t = rec.t;
    if (t < 0) continue;                               // padding row of a tile (uniform across the CTA, like every branch below)
    // (the weight-set entry field by field, not as a struct held in registers across the whole row)
    const GroupEntry* gp = sh.grp + (rec.group_flags & kRecGroupMask);
    const int act = (rec.group_flags >> kRecActShift) & 3;
    const bool add_error = (rec.group_flags & kRecAddError) != 0;
    const bool topk = act == MIX_SAE_TOPK;
    if (part > 0 && !topk) continue;                   // rows of the other activations are one CTA's
    if (a.mode == kTailFallback && !(topk && a.row_flag[p])) continue;
    if (!topk && add_error && a.out_n_active == nullptr) continue;     // the delta role's row, and nobody wants its active count
    const int slot = rec.slot, n_edit = rec.n_edit;
    const bool from_cand = topk && a.mode == kTailCand;
    const __nv_bfloat16* W_dec = rec.W_dec;
    uint4* hrow = reinterpret_cast<uint4*>(a.hidden + (size_t)t * d);
    // ---- everything the record alone gives the address of, requested together
    if (tid < n_edit) {
      const int j = a.edit_idx[slot * a.r_max + tid];
      sh.eidx[tid] = j;
      sh.enew[tid] = a.edit_mode[slot * a.r_max + tid] == MIX_EDIT_CLAMP ? a.edit_val[slot * a.r_max + tid] : 0.f;
      sh.ef[tid] = 0.f;
    }
    const int S = (int)gp->d_sae, k = gp->k;
    const float* z = a.Z + (size_t)p * a.ldz;
    const int n_tiles = S / kTileN, n_cand = n_tiles * kCandPerTile;
    unsigned ninth_max = 0u;                           // largest key among this thread's share of the tiles' 9th values
    unsigned kmin = 0xffffffffu, kmax = 0u;            // range of this thread's share of the candidate keys
    if (from_cand && n_cand >= k) {
      // (16-byte pieces, four in flight per thread: 4096 candidates are one round trip)
      const float4* cv = reinterpret_cast<const float4*>(a.cand_val + (size_t)p * a.cand_tiles * kCandPerTile);
      const int n_vec = n_cand >> 2;
      for (int i0 = tid; i0 < n_vec; i0 += 4 * kTailThreads) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kTailThreads;
          v[u] = i < n_vec ? cv[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kTailThreads;
          if (i < n_vec) {
            const uint4 key = make_uint4(f2key(v[u].x), f2key(v[u].y), f2key(v[u].z), f2key(v[u].w));
            reinterpret_cast<uint4*>(sh.keys)[i] = key;
            kmin = min(min(kmin, key.x), min(min(key.y, key.z), key.w));
            kmax = max(max(kmax, key.x), max(max(key.y, key.z), key.w));
          }
        }
      }
      const float* ninth = a.cand_ninth + (size_t)p * a.cand_tiles;
      for (int i = tid; i < n_tiles; i += kTailThreads) ninth_max = max(ninth_max, f2key(ninth[i]));
    }
    __syncthreads();
    phase_stamp(a.clk, 21, stamp);
    int* win_id = sh.feat + n_edit;                    // the winners follow the edit entries in the gather lists
    float* win_val = sh.coef + n_edit;
    if (topk) {
      const unsigned long long* sorted;
      if (from_cand) {
        // Every (row, feature tile) contributed its 8 largest pre-activations and its 9th.  The k largest
        // candidates are the row's TopK unless some tile's 9th value reaches the k-th candidate, i.e. that tile
        // may hide a winner (or an exact tie whose order matters): such rows are flagged, their row tiles are
        // re-encoded to Z and the fallback launch selects exactly.
        bool flag = n_cand < k;                        // uniform
        if (!flag) {
          CandRow src{sh.keys, n_cand};
          flag = radix_collect<false, 8>(src, k, sh.sel, true, kmin, kmax, a.clk, stamp) == 0;
        }
        phase_stamp(a.clk, 10, stamp);
        if (!flag) {
          sorted = sort_desc(sh.sel);
          phase_stamp(a.clk, 11, stamp);
          const unsigned kth = (unsigned)(sorted[k - 1] >> 32);
          flag = __syncthreads_or(ninth_max >= kth) != 0;
        }
        if (flag) {
          if (tid == 0 && part == 0) {
            a.row_flag[p] = 1;
            a.mtile_flag[p / kTileM] = 1;
            atomicAdd(a.n_flagged, 1);
          }
          __syncthreads();
          continue;
        }
        const int* ci = a.cand_idx + (size_t)p * a.cand_tiles * kCandPerTile;
        for (int i = tid; i < k; i += kTailThreads) {
          win_id[i] = ci[comp_id(sorted[i])];          // position -> feature id, for the winners only
          win_val[i] = comp_val(sorted[i]);
        }
      } else {
        ZRow src{z, S};
        const int how = radix_collect<true, 11>(src, k, sh.sel);
        if (how == 2 && tid == 0 && part == 0) atomicOr(a.status, MIX_STATUS_TOPK_GENERAL);
        sorted = sort_desc(sh.sel);
        for (int i = tid; i < k; i += kTailThreads) {
          win_id[i] = comp_id(sorted[i]);
          win_val[i] = comp_val(sorted[i]);
        }
      }
      __syncthreads();
      phase_stamp(a.clk, 12, stamp);
      if (part == 0) emit_topk(win_id, win_val, k, a.k_max, t, a.out_idx, a.out_val, a.out_n_active, &sh.sel.count);
    } else {
      if (a.out_n_active != nullptr) {
        int cnt = 0;
        const float* theta = gp->theta;
        for (int j = tid; j < S; j += kTailThreads) {
          const float v = z[j];
          cnt += act == MIX_SAE_RELU ? v > 0.f : (v > theta[j] && v > 0.f);
        }
        if (tid == 0) sh.sel.count = 0;
        __syncthreads();
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if ((tid & 31) == 0) atomicAdd(&sh.sel.count, cnt);
        __syncthreads();
        if (tid == 0) a.out_n_active[t] = sh.sel.count;
      }
      if (add_error) {                                 // the delta role's row
        __syncthreads();
        continue;
      }
    }
    // ---- edits and decode of this row
    bool alive = true;                                 // a later entry for the same feature wins
    if (tid < n_edit)
      for (int e2 = tid + 1; e2 < n_edit; ++e2) alive = alive && (sh.eidx[e2] != sh.eidx[tid]);
    if (add_error) {
      // (TopK rows only.)  f_j of an edited feature comes from the row's TopK list, 0 if it was not selected
      for (int i = tid; i < k; i += kTailThreads) {
        const int id = win_id[i];
        for (int e = 0; e < n_edit; ++e)
          if (sh.eidx[e] == id) sh.ef[e] = fmaxf(win_val[i], 0.f);
      }
      __syncthreads();
      float delta = 0.f;
      if (tid < n_edit) {
        delta = alive ? sh.enew[tid] - sh.ef[tid] : 0.f;
        sh.coef[tid] = delta;
        sh.feat[tid] = sh.eidx[tid];
      }
      phase_stamp(a.clk, 13, stamp);
      if (__syncthreads_or(delta != 0.f)) {            // no effective edit: the row stays as it is, bit for bit
        for (int v = part * kTailThreads + tid; v < nvec; v += n_split * kTailThreads) {
          float acc[8];
          load8(acc, hrow[v]);
          gather_list(acc, sh.coef, sh.feat, n_edit, W_dec, d, v, true);
          hrow[v] = pack8(acc);
        }
      }
      __syncthreads();
      phase_stamp(a.clk, 14, stamp);
      continue;
    }
    // the app replaces the residual: h' = b_dec + sum_j f'_j W_dec[j]
    if (tid < n_edit) {       // edited features contribute f' (live entries only)
      sh.coef[tid] = alive ? sh.enew[tid] : 0.f;
      sh.feat[tid] = sh.eidx[tid];
    }
    const float* b_dec = gp->b_dec;
    if (topk) {
      for (int i = tid; i < k; i += kTailThreads) {
        const int j = win_id[i];
        bool edited = false;
        for (int e = 0; e < n_edit; ++e) edited = edited || (sh.eidx[e] == j);
        // an id outside the SAE can only come from a call whose encode timed out: never address with it
        const bool in_range = (unsigned)j < (unsigned)S;
        win_val[i] = (edited || !in_range) ? 0.f : fmaxf(win_val[i], 0.f);
        win_id[i] = in_range ? j : 0;
      }
      __syncthreads();
      for (int v = part * kTailThreads + tid; v < nvec; v += n_split * kTailThreads) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = b_dec ? b_dec[v * 8 + i] : 0.f;
        gather_list(acc, sh.coef, sh.feat, n_edit + k, W_dec, d, v, true);
        hrow[v] = pack8(acc);
      }
    } else {
      // ReLU / JumpReLU: per pass of 2048 columns, the edited features first, then a dense scan of the
      // activations in chunks of 1024 -- active, unedited features are compacted into shared memory and
      // applied chunk by chunk.  (Every thread walks every pass: the scan needs the whole CTA.)
      const float* theta = gp->theta;
      for (int v0 = 0; v0 < nvec; v0 += kTailThreads) {
        const int v = v0 + tid;
        const bool in_cols = v < nvec;
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = (b_dec && in_cols) ? b_dec[v * 8 + i] : 0.f;
        __syncthreads();
        gather_list(acc, sh.coef, sh.feat, n_edit, W_dec, d, v, in_cols);
        for (int c0 = 0; c0 < S; c0 += 1024) {
          if (tid == 0) sh.n_list = 0;
          __syncthreads();
          for (int j = c0 + tid; j < min(S, c0 + 1024); j += kTailThreads) {
            const float zj = z[j];
            const float f = act == MIX_SAE_RELU ? fmaxf(zj, 0.f) : (zj > theta[j] ? zj : 0.f);
            if (f != 0.f) {
              bool edited = false;
              for (int e = 0; e < n_edit; ++e) edited = edited || (sh.eidx[e] == j);
              if (!edited) {
                const int pos = atomicAdd(&sh.n_list, 1);
                sh.coef[kMaxEdits + pos] = f;
                sh.feat[kMaxEdits + pos] = j;
              }
            }
          }
          __syncthreads();
          gather_list(acc, sh.coef + kMaxEdits, sh.feat + kMaxEdits, sh.n_list, W_dec, d, v, in_cols);
          __syncthreads();
        }
        if (in_cols) hrow[v] = pack8(acc);
      }
    }
    __syncthreads();                                   // the shared lists are reused by the next row
  }
}

// ---------------------------------------------------------------------------------------
// delta role: ReLU / JumpReLU rows with the error term
// ---------------------------------------------------------------------------------------
constexpr int kDlRows = 4;
constexpr int kDlBatch = 8;
constexpr int kDlEntries = kDlRows * kMaxEdits;

struct DeltaShared {
  __align__(16) float coef[kDlEntries + kDlBatch][kDlRows];
  const uint4* wrow[kDlEntries + kDlBatch];
  int eidx[kDlEntries];               // feature of each entry
  float enew[kDlEntries];             // f'_j of each entry
  short efirst[kDlEntries], elen[kDlEntries];   // where the entry's own edit list starts among the entries, and its length
  short eslot_row[kDlEntries];        // first row of the item that carries the entry's slot
  int t[kDlRows], slot[kDlRows], n_edit[kDlRows], act[kDlRows], changed[kDlRows];
  const __nv_bfloat16* wdec[kDlRows];
  const float* theta[kDlRows];
};

// One work item of the delta role: row group `item / n_cg`, column slices `item % n_cg`, `+ n_cg`, ... (n_cg: into how
// many items a row group's columns are split this call -- as many as still fit the grid in one wave, because the
// steps in front of the gather are repeated by every item of a row group).
// Dependent round trips: the rows' records (which carry the decoder and threshold pointers); the edit lists of
// their slots; the pre-activations and thresholds of the edited features; then, per slice, the decoder rows and
// the rows themselves.
__device__ void tail_delta(const TailArgs& a, DeltaShared& sh, int item, int n_rows, int n_cg) {
  const int tid = threadIdx.x;
  const int rg = item / n_cg, cg = item - rg * n_cg;
  const int p0 = rg * kDlRows;
  __syncthreads();                                       // the shared lists of the previous item are free
  const bool stamp = item == 0 && tid == 0;
  phase_stamp(a.clk, 22, stamp);
  if (tid < kDlRows) {
    const int p = p0 + tid;                              // in bounds: the panel capacity is a multiple of 128
    const RowRec rec = a.row_rec[p];
    const int act = (rec.group_flags >> kRecActShift) & 3;
    const bool on = p < n_rows && rec.t >= 0 && (rec.group_flags & kRecAddError) && rec.n_edit > 0 && act != MIX_SAE_TOPK;
    sh.t[tid] = on ? rec.t : -1;
    sh.slot[tid] = on ? rec.slot : -1;
    sh.n_edit[tid] = rec.n_edit;
    sh.act[tid] = act;
    sh.wdec[tid] = rec.W_dec;
    sh.theta[tid] = rec.theta;
    sh.changed[tid] = 0;
  }
  __syncthreads();
  bool any = false;
#pragma unroll
  for (int r = 0; r < kDlRows; ++r) any = any || sh.slot[r] >= 0;
  phase_stamp(a.clk, 23, stamp);
  if (!any) return;
  const int d = a.d;
  // entries: the edit lists of the distinct slots, one after the other (the coefficient of a row of another slot is zero)
  int n_entries = 0;                                    // CTA-uniform
  for (int r = 0; r < kDlRows; ++r) {
    const int slot = sh.slot[r];
    bool first = slot >= 0;
    for (int r2 = 0; r2 < r; ++r2) first = first && sh.slot[r2] != slot;
    if (!first) continue;
    const int n_edit = sh.n_edit[r];
    if (tid < n_edit) {
      const int e = n_entries + tid;
      const int j = a.edit_idx[slot * a.r_max + tid];
      sh.eidx[e] = j;
      sh.enew[e] = a.edit_mode[slot * a.r_max + tid] == MIX_EDIT_CLAMP ? a.edit_val[slot * a.r_max + tid] : 0.f;
      sh.efirst[e] = (short)n_entries;
      sh.elen[e] = (short)n_edit;
      sh.eslot_row[e] = (short)r;
      sh.wrow[e] = reinterpret_cast<const uint4*>(sh.wdec[r] + (size_t)j * d);
    }
    n_entries += n_edit;
  }
  __syncthreads();
  if (tid < kDlBatch) sh.wrow[n_entries + tid] = sh.wrow[n_entries - 1];     // pad to a whole batch: repeats of the last decoder row
  __syncthreads();
  // thread e works out entry e's coefficient for every row of its slot.  (Requesting the first decoder rows before
  // this step, so that they are in flight meanwhile, was tried: the registers they hold push the kernel over its
  // 64-register budget and the spills cost more than the overlap gains.)
  for (int e = tid; e < n_entries + kDlBatch; e += kTailThreads) {
    float c[kDlRows] = {0.f, 0.f, 0.f, 0.f};
    if (e < n_entries) {
      const int j = sh.eidx[e], r = sh.eslot_row[e], slot = sh.slot[r], act = sh.act[r];
      bool alive = true;                                 // a later entry for the same feature wins
      for (int e2 = e + 1; e2 < sh.efirst[e] + sh.elen[e]; ++e2) alive = alive && (sh.eidx[e2] != j);
      const float theta = act == MIX_SAE_JUMPRELU ? sh.theta[r][j] : 0.f;
      const float fnew = sh.enew[e];
#pragma unroll
      for (int r2 = 0; r2 < kDlRows; ++r2) {
        if (sh.slot[r2] == slot && alive) {
          const float zj = a.Z[(size_t)(p0 + r2) * a.ldz + j];
          const float f = act == MIX_SAE_RELU ? fmaxf(zj, 0.f) : (zj > theta ? zj : 0.f);
          c[r2] = fnew - f;
          if (c[r2] != 0.f) sh.changed[r2] = 1;
        }
      }
    }
#pragma unroll
    for (int r2 = 0; r2 < kDlRows; ++r2) sh.coef[e][r2] = c[r2];
  }
  __syncthreads();
  phase_stamp(a.clk, 24, stamp);
  for (int cs = cg; cs < a.n_col_slices; cs += n_cg) {
  const int v = cs * kTailThreads + tid;                 // this thread's 16-byte column vector
  if (v >= (d >> 3)) break;
  float acc[kDlRows][8];
#pragma unroll
  for (int r = 0; r < kDlRows; ++r)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[r][i] = 0.f;
  // kDlBatch decoder rows in flight per thread: the loop is bound by load latency, not arithmetic
  for (int e0 = 0; e0 < n_entries; e0 += kDlBatch) {
    uint4 q[kDlBatch];
#pragma unroll
    for (int u = 0; u < kDlBatch; ++u) q[u] = __ldg(sh.wrow[e0 + u] + v);
#pragma unroll
    for (int u = 0; u < kDlBatch; ++u) {
      const float4 c4 = *reinterpret_cast<const float4*>(&sh.coef[e0 + u][0]);
      axpy8(acc[0], c4.x, q[u]);
      axpy8(acc[1], c4.y, q[u]);
      axpy8(acc[2], c4.z, q[u]);
      axpy8(acc[3], c4.w, q[u]);
    }
  }
  phase_stamp(a.clk, 25, stamp);
  uint4 hraw[kDlRows];
#pragma unroll
  for (int r = 0; r < kDlRows; ++r)
    hraw[r] = sh.t[r] >= 0 ? reinterpret_cast<const uint4*>(a.hidden + (size_t)sh.t[r] * d)[v] : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
  for (int r = 0; r < kDlRows; ++r) {
    if (sh.slot[r] < 0 || !sh.changed[r]) continue;     // no effective edit: the row stays bit-exact
    const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hraw[r]);
    uint4 o;
    __nv_bfloat162* pp = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 h2 = __bfloat1622float2(hp[i]);
      pp[i] = __floats2bfloat162_rn(h2.x + acc[r][2 * i], h2.y + acc[r][2 * i + 1]);
    }
    reinterpret_cast<uint4*>(a.hidden + (size_t)sh.t[r] * d)[v] = o;
  }
  }
}

// Profiling aid: the time the LAST CTA of a launch ended (slot 30: main launch, 31: fallback launch), as the
// largest nanosecond-timer value any CTA saw at its end.
__device__ __forceinline__ void stamp_launch_end(unsigned long long* clk, int mode) {
  if (clk != nullptr && threadIdx.x == 0) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    atomicMax(clk + (mode == kTailFallback ? 31 : 30), t);
  }
}

// A fixed grid of CTAs (a few per SM, all resident at once or nearly) walks the work of the call: first the
// packed rows that need the row role, then the row groups x column slices of the delta role.  Both lists are as
// long as THIS call's routing made them, not as long as the context's capacity, and a role with no rows this
// call (no TopK / replacing row; no ReLU / JumpReLU row with edits) is skipped without looking at a single row.
__global__ void __launch_bounds__(kTailThreads, 4)
tail_kernel(const TailArgs a) {
  phase_stamp(a.clk, 7, blockIdx.x == 0 && threadIdx.x == 0 && a.mode != kTailFallback);
  pdl_wait();
  pdl_launch_dependents();
  phase_stamp(a.clk, 8, blockIdx.x == 0 && threadIdx.x == 0 && a.mode != kTailFallback);
  __shared__ union TailShared {     // a CTA finishes its rows before it turns to the delta role: the two share the space
    RowShared row;
    DeltaShared delta;
  } s_u;
  RowShared& s_row = s_u.row;
  DeltaShared& s_delta = s_u.delta;
  if (a.mode == kTailFallback && *a.n_flagged == 0) {   // nothing was flagged: the usual case
    stamp_launch_end(a.clk, a.mode);
    return;
  }
  const int n_rows = a.rs->n_panel_rows, n_delta = a.rs->n_delta_rows, n_sae = a.rs->n_sae_rows;
  if (a.mode == kTailFallback || n_sae > n_delta || (a.out_n_active != nullptr && n_sae > 0)) tail_rows(a, s_row, a.n_groups);
  if (a.mode != kTailFallback && n_delta > 0) {
    const int n_rg = n_rows / kDlRows;
    const int n_cg = min(a.n_col_slices, max(1, (int)gridDim.x / n_rg));
    const int n_items = n_rg * n_cg;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) tail_delta(a, s_delta, item, n_rows, n_cg);
  }
  phase_stamp(a.clk, 15, blockIdx.x == 0 && threadIdx.x == 0 && a.mode != kTailFallback);
  stamp_launch_end(a.clk, a.mode);
}

}  // namespace

// mode: 0 the main launch behind the tensor-core encode, 1 the main launch behind the CUDA-core encode (TopK
// straight from Z), 2 the fallback launch (flagged rows only; returns at once when there are none).
cudaError_t launch_tail(const Ctx* c, __nv_bfloat16* hidden, int mode, cudaStream_t s) {
  TailArgs a;
  a.hidden = hidden;
  a.d = c->cfg.d_model;
  a.Z = c->d_z;
  a.ldz = c->cfg.d_sae_max;
  a.row_rec = c->d_row_rec;
  a.rs = c->d_route;
  a.groups = c->d_groups;
  a.edit_idx = c->d_edit_idx;
  a.edit_val = c->d_edit_val;
  a.edit_mode = c->d_edit_mode;
  a.r_max = c->cfg.r_max;
  a.k_max = c->cfg.k_max;
  a.cand_val = c->d_cand_val;
  a.cand_idx = c->d_cand_idx;
  a.cand_ninth = c->d_cand_ninth;
  a.cand_tiles = c->cand_tiles;
  a.out_idx = c->out_topk_idx;
  a.out_val = c->out_topk_val;
  a.out_n_active = c->out_n_active;
  a.row_flag = c->d_row_flag;
  a.mtile_flag = c->d_mtile_flag;
  a.n_flagged = c->d_n_flagged;
  a.status = c->d_status;
  a.mode = mode;
  a.clk = c->d_phase_clk;
  a.n_groups = c->cfg.n_groups_max;
  const int n_sms = c->n_sms > 0 ? c->n_sms : 148;
  a.n_col_slices = (c->cfg.d_model / 8 + kTailThreads - 1) / kTailThreads;
  const int work_cap = c->panel_rows_cap > (c->panel_rows_cap / kDlRows) * a.n_col_slices ? c->panel_rows_cap
                                                                                          : (c->panel_rows_cap / kDlRows) * a.n_col_slices;
  const int grid = work_cap < n_sms * 4 ? work_cap : n_sms * 4;      // four CTAs per SM: all of them resident at once
  return launch_pdl(kPdlTail, tail_kernel, dim3(grid), dim3(kTailThreads), 0, s, a);
}

}  // namespace mix
