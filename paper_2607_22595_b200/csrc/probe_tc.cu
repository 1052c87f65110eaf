// Multi-class probes of large batches on the 5th-generation tensor cores (sm_100a only).
//
//   logits[t, c] = sum_i hidden[t, i] * W_s[c, i] + b_s[c],   s = slot of row t,   2 <= C_s <= 32
//
// 128 consecutive rows x up to 32 classes x d is a very skinny contraction: the arithmetic is
// nothing, the job is to stream `hidden` from HBM once, at HBM speed.  That is what the TMA ->
// tcgen05 pipeline of the SAE encode is good at, so the same machinery is used: one persistent CTA
// per SM; warp 0 = TMA producer (a 128 x 64 tile of `hidden`, straight from the caller's tensor, and
// a 32 x 64 tile of each probe matrix that occurs in the tile, per k-block, into a 5-stage ring:
// ~80 KiB of `hidden` in flight per SM without holding a single register), warp 1 = MMA issuer
// (M = 128, N = 32 per distinct probe of the tile, up to 4 probes side by side, fp32 accumulators
// in tensor memory, double buffered), warps 2..5 = epilogue (one lane per row: its probe's 32
// columns, + bias, softmax / sigmoid / identity, scores out), warp 6 = scout (reads the tile's slot
// ids and app entries, evaluates gates, groups the rows by probe and hands the other roles one
// descriptor per pass through a small ring).  Rows of other kinds inside a tile are streamed but
// ignored.  The CTAs share out the tiles that a census kernel listed as holding such rows (mc_census_kernel), and the
// kernel takes the call when those tiles are at least half full of such rows; thinly scattered rows go to the 16-row mma.sync kernel.  No TMA multicast, no clusters; every wait is
// bounded (on expiry: MIX_STATUS_WAIT_TIMEOUT, copies are given time to land, tensor memory freed).
#include "mix_internal.h"
#include "row_lookup.cuh"
#include "tc_common.cuh"

namespace mix {

namespace {

using namespace tc;

constexpr int kPStages = 9;
constexpr int kPABytes = kTileM * kTileK * 2;          // 16 KiB: 128 rows x 64 columns of hidden
constexpr int kPBlockCols = 32;                        // accumulator columns per probe (= most classes taken)
constexpr int kPBlocks = 2;                            // probes side by side in one pass
constexpr int kPBlockBytes = kPBlockCols * kTileK * 2; // 4 KiB: 32 classes x 64 columns
constexpr int kPBBytes = kPBlocks * kPBlockBytes;      // 8 KiB
constexpr int kPStageBytes = kPABytes + kPBBytes;
constexpr int kPThreads = 7 * 32;
constexpr int kPTmemCols = 2 * kPBlocks * kPBlockCols; // 128: two accumulators of 64 columns
constexpr long long kPWaitCycles = 4000000000ll;       // ~2 s at 2 GHz
constexpr long long kPWaitCyclesTest = 2000000ll;      // ~1 ms: the cap under MIX_FLAG_TEST_STALL_ENCODE

struct PDesc {
  int t0;                       // first row of the tile
  int n_blocks;                 // probes in this pass (1..4); 0 = no more work for this CTA
  int slot[kPBlocks];
  signed char row_block[kTileM];   // block of each row in this pass, or -1
};

struct __align__(8) PShared {
  unsigned long long full[kPStages];
  unsigned long long empty[kPStages];
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
  unsigned long long desc_full[2];
  unsigned long long desc_empty[2];
  unsigned tmem_base;
  volatile int abort_flag;
  long long wait_cycles;        // cap of every bounded wait in this launch
  PDesc desc[2];
};
constexpr int kPSmemBytes = kPStages * kPStageBytes + 1024 /* alignment slack */ + 1024 /* PShared */;
static_assert(kPSmemBytes <= 227 * 1024, "shared memory per CTA");
static_assert(sizeof(PShared) <= 1024, "PShared must fit the space reserved for it");

__device__ __forceinline__ bool pwait(unsigned bar, unsigned parity, PShared* sh, unsigned* status) {
  return mbar_wait_bounded(bar, parity, &sh->abort_flag, &sh->wait_cycles, status);
}

__global__ void __launch_bounds__(kPThreads, 1)
probe_tc_kernel(const __grid_constant__ CUtensorMap tmap_hidden, const CUtensorMap* __restrict__ tmap_probe,
                const int* __restrict__ token_slot, const int* __restrict__ n_live_p, int T,
                const AppEntry* __restrict__ apps, const GateEntry* __restrict__ gates, int n_slots, int d,
                float* __restrict__ scores, int C_max, unsigned* __restrict__ status, const McCensus* __restrict__ census,
                const int* __restrict__ census_tiles, int test_stall) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* tiles = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  PShared* sh = reinterpret_cast<PShared*>(tiles + kPStages * kPStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_live = min(T, __ldg(n_live_p));
  // the tiles of this call that hold multi-class probe rows, as the census listed them (in no particular order):
  // CTAs share THEM out, so a batch whose hooked requests are clustered still spreads evenly over the SMs
  if (!census->use_tc) return;                         // rows scattered thinly: probe_multiclass_kernel's call
  const int n_tiles = census->n_tiles;
  if ((int)blockIdx.x >= n_tiles) return;              // CTA-uniform: this CTA owns no tile
  if (threadIdx.x == 0) {
    for (int s = 0; s < kPStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sh->tmem_full[a]), 1);
      mbar_init(smem_u32(&sh->tmem_empty[a]), 4);
      mbar_init(smem_u32(&sh->desc_full[a]), 1);
      mbar_init(smem_u32(&sh->desc_empty[a]), 6);      // producer, MMA issuer, four epilogue warps
    }
    sh->abort_flag = 0;
    sh->wait_cycles = test_stall ? kPWaitCyclesTest : kPWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (warp == 1) tmem_alloc(smem_u32(&sh->tmem_base), kPTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = sh->tmem_base;
  const int num_kb = d / kTileK;

  if (warp == 6) {
    // ---- scout: one descriptor per (tile, pass of up to 4 probes), then a terminator
    int di = 0;
    unsigned dphase = 0;
    bool ok = true;
    for (int ti = blockIdx.x; ti < n_tiles && ok; ti += gridDim.x) {
      const int tile = __ldg(census_tiles + ti);
      int s[4], blk[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        s[i] = -1;
        blk[i] = -1;
        const int t = tile * kTileM + i * 32 + lane;
        if (t < n_live) {
          const int sl = __ldg(token_slot + t);
          const RowApp a = lookup(sl, t, apps, gates, n_slots, nullptr, false);   // bad slots: flagged by probe_steer_kernel
          if (a.kind == MIX_PROBE && a.C > 1 && a.C <= kPBlockCols) s[i] = sl;
        }
      }
      int nd = 0;                                       // distinct probes of the tile, in order of first row
      for (;;) {
        int src_i = -1, src_lane = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const unsigned m = __ballot_sync(0xffffffffu, s[i] >= 0 && blk[i] < 0);
          if (src_i < 0 && m != 0u) {
            src_i = i;
            src_lane = __ffs(m) - 1;
          }
        }
        if (src_i < 0) break;
        int S = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int v = __shfl_sync(0xffffffffu, s[i], src_lane);
          if (i == src_i) S = v;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (s[i] == S) blk[i] = nd;
        ++nd;
      }
      const int n_pass = (nd + kPBlocks - 1) / kPBlocks;                 // a tile without such rows emits nothing
      for (int p = 0; p < n_pass && ok; ++p) {
        if (!__all_sync(0xffffffffu, pwait(smem_u32(&sh->desc_empty[di]), dphase ^ 1u, sh, status))) { ok = false; break; }
        PDesc* ds = &sh->desc[di];
        if (lane == 0) {
          ds->t0 = tile * kTileM;
          ds->n_blocks = min(kPBlocks, nd - p * kPBlocks);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int b = blk[i] - p * kPBlocks;
          const bool in = blk[i] >= 0 && b >= 0 && b < kPBlocks;
          ds->row_block[i * 32 + lane] = (signed char)(in ? b : -1);
          if (in) ds->slot[b] = s[i];                  // every row of the block writes the same value
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh->desc_full[di]));
        di ^= 1;
        if (di == 0) dphase ^= 1u;
      }
    }
    if (ok && __all_sync(0xffffffffu, pwait(smem_u32(&sh->desc_empty[di]), dphase ^ 1u, sh, status))) {
      if (lane == 0) {
        sh->desc[di].n_blocks = 0;                     // terminator: the other roles leave their loops
        mbar_arrive(smem_u32(&sh->desc_full[di]));
      }
    }
  } else if (warp == 0) {
    // ---- producer
    if (lane == 0) {
      int di = 0, stage = 0;
      unsigned dphase = 0, phase = 0;
      for (;;) {
        if (!pwait(smem_u32(&sh->desc_full[di]), dphase, sh, status)) break;
        const PDesc* ds = &sh->desc[di];
        const int nb = ds->n_blocks, t0 = ds->t0;
        int slot[kPBlocks];
#pragma unroll
        for (int b = 0; b < kPBlocks; ++b) slot[b] = ds->slot[b];
        mbar_arrive(smem_u32(&sh->desc_empty[di]));    // everything this role needs has been copied out
        di ^= 1;
        if (di == 0) dphase ^= 1u;
        if (nb == 0) break;
        bool ok = true;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!pwait(smem_u32(&sh->empty[stage]), phase ^ 1u, sh, status)) { ok = false; break; }
          // Test hook (MIX_FLAG_TEST_STALL_ENCODE): the producer never fills a stage, so the consumers' bounded
          // waits run out and the whole CTA leaves through the time-out path.
          if (test_stall) { ok = false; break; }
          const unsigned bar = smem_u32(&sh->full[stage]);
          mbar_expect_tx(bar, kPABytes + nb * kPBlockBytes);
          const unsigned sa = smem_u32(tiles + stage * kPStageBytes);
          tma_load_2d(sa, &tmap_hidden, kb * kTileK, t0, bar);
          for (int b = 0; b < nb; ++b)
            tma_load_2d(sa + kPABytes + b * kPBlockBytes, tmap_probe + slot[b], kb * kTileK, 0, bar);
          if (++stage == kPStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer
    if (lane == 0) {
      int di = 0, stage = 0;
      unsigned dphase = 0, phase = 0, acc = 0, acc_phase = 0;
      for (;;) {
        if (!pwait(smem_u32(&sh->desc_full[di]), dphase, sh, status)) break;
        const int nb = sh->desc[di].n_blocks;
        mbar_arrive(smem_u32(&sh->desc_empty[di]));
        di ^= 1;
        if (di == 0) dphase ^= 1u;
        if (nb == 0) break;
        if (!pwait(smem_u32(&sh->tmem_empty[acc]), acc_phase ^ 1u, sh, status)) break;
        tc_fence_after();
        const unsigned d_tmem = tmem_base + acc * (kPBlocks * kPBlockCols);
        const unsigned idesc = idesc_f16(kTileM, nb * kPBlockCols);
        bool ok = true;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!pwait(smem_u32(&sh->full[stage]), phase, sh, status)) { ok = false; break; }
          tc_fence_after();
          const unsigned sa = smem_u32(tiles + stage * kPStageBytes);
          const unsigned long long da = umma_desc(sa), db = umma_desc(sa + kPABytes);
#pragma unroll
          for (int k = 0; k < kTileK / 16; ++k) umma_f16(d_tmem, da + 2ull * k, db + 2ull * k, idesc, (unsigned)((kb | k) != 0));
          umma_commit(smem_u32(&sh->empty[stage]));
          if (++stage == kPStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&sh->tmem_full[acc]));
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ---- epilogue: lane = row
    const int q = warp & 3;                            // tensor-memory lane quarter this warp may read
    int di = 0;
    unsigned dphase = 0, acc = 0, acc_phase = 0;
    for (;;) {
      if (!__all_sync(0xffffffffu, pwait(smem_u32(&sh->desc_full[di]), dphase, sh, status))) break;
      const PDesc* ds = &sh->desc[di];
      const int nb = ds->n_blocks;
      if (nb == 0) {
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh->desc_empty[di]));
        break;
      }
      const int row = q * 32 + lane;
      const int t = ds->t0 + row;
      const int my_block = ds->row_block[row];
      if (!__all_sync(0xffffffffu, pwait(smem_u32(&sh->tmem_full[acc]), acc_phase, sh, status))) break;
      tc_fence_after();
      const unsigned taddr = tmem_base + ((unsigned)(q * 32) << 16) + acc * (kPBlocks * kPBlockCols);
      for (int b = 0; b < nb; ++b) {
        float v[32];
        tmem_ld32(taddr + b * kPBlockCols, v);
        if (my_block != b) continue;                   // the load above is warp-wide; the rest is per row
        const AppEntry* e = apps + ds->slot[b];
        const int C = __ldg(&e->n_classes), act = __ldg(&e->act);
        const float* bias = reinterpret_cast<const float*>(__ldg(reinterpret_cast<const unsigned long long*>(&e->b)));
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          if (c < C) {
            v[c] += bias ? __ldg(bias + c) : 0.f;
            mx = fmaxf(mx, v[c]);
          }
        }
        float* out = scores + (size_t)t * C_max;
        if (act == MIX_ACT_SOFTMAX) {
          float sum = 0.f;
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            if (c < C) {
              v[c] = expf(v[c] - mx);
              sum += v[c];
            }
          }
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c < C) out[c] = v[c] / sum;
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c < C) out[c] = act == MIX_ACT_SIGMOID ? 1.f / (1.f + expf(-v[c])) : v[c];
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&sh->tmem_empty[acc]));
        mbar_arrive(smem_u32(&sh->desc_empty[di]));
      }
      acc ^= 1u;
      if (acc == 0) acc_phase ^= 1u;
      di ^= 1;
      if (di == 0) dphase ^= 1u;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (sh->abort_flag) {
    // give copies that are still in flight time to land before shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kPTmemCols);
  }
}

}  // namespace

cudaError_t probe_tc_prepare() {
  return cudaFuncSetAttribute(probe_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemBytes);
}

cudaError_t launch_probe_tc(const Ctx* c, const CUtensorMap& tmap_hidden, int T, float* scores, cudaStream_t s) {
  if (scores == nullptr) return cudaSuccess;
  probe_tc_kernel<<<c->n_sms, kPThreads, kPSmemBytes, s>>>(tmap_hidden, c->d_tmap_probe, c->d_token_slot, c->d_n_live, T,
                                                           c->d_apps, c->d_gates, c->cfg.n_slots_max, c->cfg.d_model, scores,
                                                           c->cfg.C_max, c->d_status, c->d_mc_census, c->d_mc_tiles,
                                                           (c->cfg.flags & MIX_FLAG_TEST_STALL_ENCODE) ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace mix
