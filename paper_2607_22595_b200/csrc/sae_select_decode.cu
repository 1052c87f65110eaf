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
constexpr int kCand = 4096;
constexpr int kBins = 2048;

__device__ __forceinline__ unsigned f2key(float f) {
  const unsigned b = __float_as_uint(f + 0.f);          // -0.0 -> +0.0: equal values, equal keys
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key2f(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Largest digit D with count(digit >= D) >= need, and the count of digits > D.  One warp.
__device__ void find_digit(const int* hist, int n_bins, int need, int* s_out) {
  const int lane = threadIdx.x & 31;
  const int per = n_bins / 32;
  // lane L owns bins [n_bins - (L+1)*per, n_bins - L*per): lane 0 holds the largest digits
  const int hi = n_bins - lane * per;
  int sum = 0;
  for (int b = hi - per; b < hi; ++b) sum += hist[b];
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  const int excl = incl - sum;                 // elements in bins above this lane's range
  if (excl < need && incl >= need) {
    int above = excl;
    for (int b = hi - 1; b >= hi - per; --b) {
      if (above + hist[b] >= need) {
        s_out[0] = b;
        s_out[1] = above;
        break;
      }
      above += hist[b];
    }
  }
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ Z, long long ldz, const int* __restrict__ panel_row,
              const int* __restrict__ mtile_group, const RouteState* __restrict__ rs,
              const GroupEntry* __restrict__ groups, int k_max, int* __restrict__ ws_idx, float* __restrict__ ws_val,
              int* __restrict__ out_idx, float* __restrict__ out_val, int* __restrict__ out_n_active,
              unsigned* __restrict__ status) {
  __shared__ int s_hist[kBins];
  __shared__ unsigned long long s_cand[kCand];
  __shared__ int s_n, s_res[2], s_count;
  const int p = blockIdx.x;
  if (p >= rs->n_panel_rows) return;
  const int t = panel_row[p];
  if (t < 0) return;
  const GroupEntry ge = groups[mtile_group[p / kTileM]];
  const int S = (int)ge.d_sae;
  const float* z = Z + (size_t)p * ldz;
  const int tid = threadIdx.x;

  if (ge.act != MIX_SAE_TOPK) {
    if (out_n_active == nullptr) return;
    int cnt = 0;
    for (int j = tid; j < S; j += kSelThreads) {
      const float v = z[j];
      const bool on = ge.act == MIX_SAE_RELU ? v > 0.f : (v > ge.theta[j] && v > 0.f);
      cnt += on;
    }
    if (tid == 0) s_count = 0;
    __syncthreads();
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if ((tid & 31) == 0) atomicAdd(&s_count, cnt);
    __syncthreads();
    if (tid == 0) out_n_active[t] = s_count;
    return;
  }

  const int k = ge.k;
  // radix refinement: 11 + 11 + 10 bits from the top
  const int shifts[3] = {21, 10, 0};
  const int widths[3] = {11, 11, 10};
  unsigned prefix = 0;          // digits fixed so far (value of key >> (shift + width))
  int need = k;                 // winners still to be found inside the prefix set
  bool done = false;
  int pass = 0;
  unsigned thr_hi = 0;          // elements with (key >> thr_shift) >= thr_hi are candidates
  int thr_shift = 0;
  for (; pass < 3 && !done; ++pass) {
    const int shift = shifts[pass], nb = 1 << widths[pass];
    for (int b = tid; b < nb; b += kSelThreads) s_hist[b] = 0;
    __syncthreads();
    for (int j = tid; j < S; j += kSelThreads) {
      const unsigned key = f2key(z[j]);
      if (pass == 0 || (key >> (shift + widths[pass])) == prefix) atomicAdd(&s_hist[(key >> shift) & (nb - 1)], 1);
    }
    __syncthreads();
    if (tid < 32) find_digit(s_hist, nb, need, s_res);
    __syncthreads();
    const int D = s_res[0], above = s_res[1];
    const int in_bin = s_hist[D];
    need -= above;
    prefix = (prefix << widths[pass]) | (unsigned)D;
    thr_hi = prefix;
    thr_shift = shift;
    if ((k - need) + in_bin <= kCand) done = true;
    __syncthreads();
  }

  if (tid == 0) s_n = 0;
  __syncthreads();
  if (done) {
    for (int j = tid; j < S; j += kSelThreads) {
      const unsigned key = f2key(z[j]);
      if ((key >> thr_shift) >= thr_hi) {
        const int pos = atomicAdd(&s_n, 1);
        s_cand[pos] = ((unsigned long long)key << 32) | (unsigned)(0xffffffffu - (unsigned)j);
      }
    }
  } else {
    // more than kCand exact ties at the k-th value: take every larger key, then the `need`
    // lowest feature ids among the tied ones, in index order.
    if (tid == 0) atomicOr(status, MIX_STATUS_TOPK_GENERAL);
    for (int j = tid; j < S; j += kSelThreads) {
      const unsigned key = f2key(z[j]);
      if (key > prefix) {
        const int pos = atomicAdd(&s_n, 1);
        s_cand[pos] = ((unsigned long long)key << 32) | (unsigned)(0xffffffffu - (unsigned)j);
      }
    }
    __syncthreads();
    int taken = 0;               // uniform across the block
    for (int j0 = 0; j0 < S && taken < need; j0 += kSelThreads) {
      const int j = j0 + tid;
      const bool eq = j < S && f2key(z[j]) == prefix;
      const unsigned m = __ballot_sync(0xffffffffu, eq);
      if ((tid & 31) == 0) s_hist[tid >> 5] = __popc(m);
      __syncthreads();
      int before = 0, total = 0;
      for (int w = 0; w < kSelThreads / 32; ++w) {
        const int c = s_hist[w];
        if (w < (tid >> 5)) before += c;
        total += c;
      }
      const int rank = taken + before + __popc(m & ((1u << (tid & 31)) - 1u));
      if (eq && rank < need) {
        const int pos = atomicAdd(&s_n, 1);
        s_cand[pos] = ((unsigned long long)prefix << 32) | (unsigned)(0xffffffffu - (unsigned)j);
      }
      taken += total;
      __syncthreads();
    }
  }
  __syncthreads();
  const int n = s_n;
  int n2 = 1;
  while (n2 < n) n2 <<= 1;
  for (int i = n + tid; i < n2; i += kSelThreads) s_cand[i] = 0ull;
  __syncthreads();
  // bitonic sort, descending
  for (int size = 2; size <= n2; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = tid; i < n2 / 2; i += kSelThreads) {
        const int lo = 2 * i - (i & (stride - 1));
        const int hi = lo + stride;
        const bool desc = ((lo & size) == 0);
        const unsigned long long a = s_cand[lo], b = s_cand[hi];
        if ((a < b) == desc) {
          s_cand[lo] = b;
          s_cand[hi] = a;
        }
      }
      __syncthreads();
    }
  }
  int pos_cnt = 0;
  for (int i = tid; i < k; i += kSelThreads) {
    const unsigned long long c = s_cand[i];
    const int j = (int)(0xffffffffu - (unsigned)(c & 0xffffffffull));
    const float v = key2f((unsigned)(c >> 32));
    ws_idx[(size_t)p * k_max + i] = j;
    ws_val[(size_t)p * k_max + i] = v;
    if (out_idx) out_idx[(size_t)t * k_max + i] = j;
    if (out_val) out_val[(size_t)t * k_max + i] = v;
    pos_cnt += v > 0.f;
  }
  if (out_n_active) {
    if (tid == 0) s_count = 0;
    __syncthreads();
    pos_cnt = __reduce_add_sync(0xffffffffu, pos_cnt);
    if ((tid & 31) == 0) atomicAdd(&s_count, pos_cnt);
    __syncthreads();
    if (tid == 0) out_n_active[t] = s_count;
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

__global__ void __launch_bounds__(kDecThreads)
decode_kernel(__nv_bfloat16* __restrict__ hidden, int d, const float* __restrict__ Z, long long ldz,
              const int* __restrict__ panel_row, const int* __restrict__ token_slot,
              const RouteState* __restrict__ rs, const AppEntry* __restrict__ apps,
              const GroupEntry* __restrict__ groups, const int* __restrict__ edit_idx,
              const float* __restrict__ edit_val, const unsigned char* __restrict__ edit_mode, int r_max, int k_max,
              const int* __restrict__ ws_idx, const float* __restrict__ ws_val) {
  __shared__ float s_coef[kDecList];
  __shared__ int s_feat[kDecList];
  __shared__ float s_fnew[kMaxEdits];
  __shared__ int s_eidx[kMaxEdits];
  __shared__ int s_alive[kMaxEdits];
  __shared__ int s_any, s_n;
  const int p = blockIdx.x;
  if (p >= rs->n_panel_rows) return;
  const int t = panel_row[p];
  if (t < 0) return;
  const int slot = token_slot[t];
  const AppEntry app = apps[slot];
  const GroupEntry ge = groups[app.group];
  const int tid = threadIdx.x;
  const int n_edit = app.n_edit;
  const int S = (int)ge.d_sae;
  const float* z = Z + (size_t)p * ldz;
  const int* K = ws_idx + (size_t)p * k_max;
  const float* Kv = ws_val + (size_t)p * k_max;
  const int nvec = d >> 3;

  if (tid == 0) { s_any = 0; s_n = 0; }
  if (tid < n_edit) s_eidx[tid] = edit_idx[slot * r_max + tid];
  __syncthreads();
  // edits: f_j before and after; a later entry for the same feature overrides an earlier one
  if (tid < n_edit) {
    const int j = s_eidx[tid];
    bool alive = true;
    for (int e2 = tid + 1; e2 < n_edit; ++e2) alive = alive && (s_eidx[e2] != j);
    const float zj = z[j];
    float f;
    if (ge.act == MIX_SAE_RELU) {
      f = fmaxf(zj, 0.f);
    } else if (ge.act == MIX_SAE_JUMPRELU) {
      f = zj > ge.theta[j] ? zj : 0.f;
    } else {
      bool in = false;
      for (int i = 0; i < ge.k; ++i) in = in || (K[i] == j);
      f = in ? fmaxf(zj, 0.f) : 0.f;
    }
    const float fnew = edit_mode[slot * r_max + tid] == MIX_EDIT_CLAMP ? edit_val[slot * r_max + tid] : 0.f;
    s_alive[tid] = alive;
    s_fnew[tid] = fnew;
    if (app.add_error) {
      const float delta = alive ? fnew - f : 0.f;
      s_coef[tid] = delta;
      s_feat[tid] = j;
      if (delta != 0.f) s_any = 1;
    }
  }
  __syncthreads();

  float acc[kDecU][8];
  uint4* hrow = reinterpret_cast<uint4*>(hidden + (size_t)t * d);
  if (app.add_error) {
    if (!s_any) return;                       // no effective edit: the row stays bit-exact
#pragma unroll
    for (int u = 0; u < kDecU; ++u) {
      const int v = tid + u * kDecThreads;
      if (v < nvec) {
        const uint4 q = hrow[v];
        const __nv_bfloat162* pp = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f2 = __bfloat1622float2(pp[i]);
          acc[u][2 * i] = f2.x;
          acc[u][2 * i + 1] = f2.y;
        }
      }
    }
    accumulate_list(acc, s_coef, s_feat, n_edit, ge.W_dec, d, nvec);
  } else {
#pragma unroll
    for (int u = 0; u < kDecU; ++u) {
      const int v = tid + u * kDecThreads;
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[u][i] = (ge.b_dec && v < nvec) ? ge.b_dec[v * 8 + i] : 0.f;
    }
    // edited features contribute f' (live entries only)
    if (tid < n_edit) {
      s_coef[tid] = s_alive[tid] ? s_fnew[tid] : 0.f;
      s_feat[tid] = s_eidx[tid];
    }
    __syncthreads();
    accumulate_list(acc, s_coef, s_feat, n_edit, ge.W_dec, d, nvec);
    __syncthreads();
    if (ge.act == MIX_SAE_TOPK) {
      for (int i = tid; i < ge.k; i += kDecThreads) {
        const int j = K[i];
        bool edited = false;
        for (int e = 0; e < n_edit; ++e) edited = edited || (s_eidx[e] == j);
        s_coef[i] = edited ? 0.f : fmaxf(Kv[i], 0.f);
        s_feat[i] = j;
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
}

}  // namespace

cudaError_t launch_encode_simt(const Ctx* c, cudaStream_t s) {
  dim3 grid((unsigned)(c->cfg.d_sae_max / 64), (unsigned)(c->panel_rows_cap / 64));
  encode_simt_kernel<<<grid, 256, 0, s>>>(c->d_panel, c->d_mtile_group, c->d_route, c->d_groups, c->d_z,
                                          c->cfg.d_sae_max, c->cfg.d_model);
  return cudaGetLastError();
}

cudaError_t launch_select(const Ctx* c, cudaStream_t s) {
  select_kernel<<<c->panel_rows_cap, kSelThreads, 0, s>>>(c->d_z, c->cfg.d_sae_max, c->d_panel_row,
                                                          c->d_mtile_group, c->d_route, c->d_groups, c->cfg.k_max,
                                                          c->d_topk_idx, c->d_topk_val, c->out_topk_idx,
                                                          c->out_topk_val, c->out_n_active, c->d_status);
  return cudaGetLastError();
}

cudaError_t launch_decode(const Ctx* c, __nv_bfloat16* hidden, cudaStream_t s) {
  decode_kernel<<<c->panel_rows_cap, kDecThreads, 0, s>>>(hidden, c->cfg.d_model, c->d_z, c->cfg.d_sae_max,
                                                          c->d_panel_row, c->d_token_slot, c->d_route, c->d_apps,
                                                          c->d_groups, c->d_edit_idx, c->d_edit_val, c->d_edit_mode,
                                                          c->cfg.r_max, c->cfg.k_max, c->d_topk_idx, c->d_topk_val);
  return cudaGetLastError();
}

}  // namespace mix
