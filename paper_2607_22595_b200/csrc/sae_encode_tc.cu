// SAE encode on the 5th-generation tensor cores (sm_100a only).
//
//   Z[p, j] = sum_i panel[p, i] * W_enc[j, i] + b_eff[j]        bf16 x bf16 -> fp32
//
// One persistent CTA per SM walks a device-built tile schedule (group, feature tile, row tile).
// Warp roles:  warp 0 = TMA producer (panel tile 128x64 and W_enc tile 256x64 per k-block into
// a 4-stage ring of 128-byte-swizzled shared memory), warp 1 = MMA issuer (tcgen05.mma
// 128x256x16, fp32 accumulators in tensor memory, double buffered so the epilogue of one tile
// overlaps the main loop of the next), warps 2..9 = epilogue, two per tensor-memory lane quarter
// with 128 columns of the tile each (tcgen05.ld, + bias -- the warp's columns of it copied to shared
// memory before the accumulator is waited for -- then either
// the fp32 pre-activations to the Z scratch, or -- for TopK weight sets -- only the tile's 8
// largest values per row plus its 9th, which the tail kernel turns into the exact TopK; the two
// warps of a quarter merge their lists through shared memory).
// A second form (kPair) runs on clusters of two CTAs that share a 256-row tile through
// tcgen05.mma.cta_group::2; which form works on a call is decided on the device (see TcCfg).
// No TMA multicast in either form.  Every wait is bounded: on expiry the CTA raises
// MIX_STATUS_WAIT_TIMEOUT, lets its copies land, frees its tensor memory and returns.
//
// 8-bit encoder (kEnc != 0): W_enc is E4M3 codes with one fp32 scale per feature, and the contraction is
// tcgen05.mma kind::f8f6f4 (both operands E4M3), 128 x 256 x 32 per instruction.  A k-block is 128 elements
// (the same 128-byte swizzled rows: 16 KiB of panel, 32 KiB of W_enc, four instructions), so the kernel is the
// bf16 kernel with half as many k-blocks; the epilogue multiplies the accumulator by row scale x feature scale.
//   kEnc == 2 (8-bit input): the panel holds the row quantised to E4M3 with a power-of-two scale.
//   kEnc == 1 (the hidden state stays bf16): the pack step split each row EXACTLY (down to 2^-10 of the scale)
//     into two E4M3 operands hi + lo with one common power-of-two scale; a stage carries both panel tiles
//     (16 + 16 + 32 KiB, three stages) and the eight instructions of a k-block accumulate hi W and lo W into
//     the same accumulator.  Per element of K that is the tensor time of the bf16 kernel with half the W_enc
//     bytes: as fast as kEnc == 2 where the stream of W_enc is the bound, as fast as bf16 where the tensor
//     pipe is.
#include <stdlib.h>

#include "mix_internal.h"
#include "tc_common.cuh"

namespace mix {

namespace {

constexpr int kMaxStages = 6;
constexpr int kABytes = kTileM * kTileK * 2;   // 16 KiB: 128 rows of 128 bytes
constexpr int kBBytes = kTileN * kTileK * 2;   // 32 KiB: 256 rows of 128 bytes
constexpr int kXchgEntries = kCandPerTile + 2;  // a top-9 list and the bound it was collected under
// kEnc: 0 = bf16 encoder and input; 1 = 8-bit encoder, bf16 input as two E4M3 operands; 2 = 8-bit encoder and 8-bit input
// kPair: two CTAs (a cluster) share one 256-row x 256-feature tile: each loads its own 128 panel rows and HALF of the
//        W_enc tile, and one tcgen05.mma.cta_group::2 instruction feeds both SMs' tensor cores -- a third less
//        shared-memory fill per SM and flop than a CTA working alone (32 instead of 48 KiB per k-block).
template <int kEnc, int kEpi, bool kPair> struct TcCfg {
  static_assert(kEpi == 4 || kEpi == 8, "epilogue warps");
  static constexpr bool kSplit = kEnc == 1;            // two panel tiles (hi, lo) per stage
  static constexpr int kBBytesCta = kPair ? kBBytes / 2 : kBBytes;
  static constexpr int kStageBytes = (kSplit ? 2 : 1) * kABytes + kBBytesCta;
  static constexpr int kStages = kPair ? (kSplit ? 4 : 6) : (kSplit ? 3 : 4);
  static constexpr int kRingBytes = kStages * kStageBytes;
  // epilogue warps: 4 (one per tensor-memory lane quarter, all 256 columns) or 8 (two per quarter, 128 columns
  // each; the two top-9 lists of a row meet in shared memory).  One warp per scheduler runs the epilogue's
  // dependent compare/select chains at a fraction of the issue rate; two interleave.
  static constexpr int kEpiWarps = kEpi;
  static constexpr int kXchgBytes = kEpiWarps == 8 ? 2 * 4 * kXchgEntries * 32 * 8 : 0;   // [acc][quarter][entry][lane] x (value, column)
  static constexpr int kThreads = 64 + kEpiWarps * 32;
  // each epilogue warp keeps the bias (and, for codes, the feature scale) of its columns of the current tile in
  // shared memory, fetched while the tile's main loop still runs
  static constexpr int kEpiVecBytes = 2 * 4 * kTileN * 4;   // [bias, scale][warp][its columns] floats: 8 KiB with 4 or 8 warps
  static constexpr int kSmemBytes = kRingBytes + 1024 /* alignment slack */ + 1024 /* TcShared */ + kXchgBytes + kEpiVecBytes;
  static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");
};
constexpr int kTmemCols = 512;                 // two 128 x 256 fp32 accumulators
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s at 2 GHz
constexpr long long kWaitCyclesTest = 2000000ll;  // ~1 ms: the cap under MIX_FLAG_TEST_STALL_ENCODE

struct __align__(8) TcShared {
  unsigned long long full[kMaxStages];      // (a pair's leader: filled by both CTAs' copies)
  unsigned long long empty[kMaxStages];
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
  unsigned long long xchg_full[2][4];     // 8 epilogue warps: the upper-half warp's list of (accumulator, quarter) is in shared memory
  unsigned tmem_base;
  volatile int abort_flag;
  long long wait_cycles;      // cap of every bounded wait in this launch
  RouteState rs;
  // The weight sets of this call that are THIS kernel's (single CTAs or pairs, as the front kernel dealt them; all
  // of them in the pass over flagged row tiles), numbered through: first unit -- a 128-row tile, or a pair of
  // them -- and first tile of each set, totals in entry [n_groups]; sets of the other kernel have no units here
  short unit0[kMaxGroups + 1];
  int utile0[kMaxGroups + 1];
};
static_assert(sizeof(TcShared) <= 1024, "TcShared must fit the space reserved for it");

using namespace tc;

// Bounded wait on this kernel's shared state.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, TcShared* sh, unsigned* status) {
  return mbar_wait_bounded(bar, parity, &sh->abort_flag, &sh->wait_cycles, status);
}

constexpr unsigned kIdesc = idesc_f16(kTileM, kTileN);     // D fp32, A and B bf16, K-major, N = 256, M = 128
constexpr unsigned kIdescE4 = idesc_e4m3(kTileM, kTileN);  // D fp32, A and B E4M3, K-major, N = 256, M = 128
constexpr unsigned kIdescPair = idesc_f16(2 * kTileM, kTileN);     // the pair's instruction: M = 256
constexpr unsigned kIdescE4Pair = idesc_e4m3(2 * kTileM, kTileN);

struct Tile {
  int group, n_tile, m_tile_global, rows_valid;
  int m_tile_peer;      // CTA pairs: the row tile the other CTA of the pair works on (the same one when the weight set has an odd tile left over)
};

// Number of feature tiles per unit if it is the same for every weight set of this kernel that has rows (the
// usual case: one SAE width per context), else 0.
__device__ __forceinline__ int uniform_feature_tiles(const TcShared& sh, int n_groups) {
  int nt = -1;
  for (int g = 0; g < n_groups; ++g) {
    const int units = sh.unit0[g + 1] - sh.unit0[g];
    if (units == 0) continue;
    const int nt_g = (sh.utile0[g + 1] - sh.utile0[g]) / units;
    if (nt >= 0 && nt_g != nt) return 0;
    nt = nt_g;
  }
  return nt > 0 ? nt : 0;
}

// Linear tile id of this kernel -> (weight set, feature tile, unit of the set) and, for the CTA of rank `rank` of a
// pair, its own row tile.  With one SAE width the order is feature tile by feature tile over ALL units, so every
// row sees its first feature tiles finished early in the launch (the TopK epilogue's running bound needs that);
// otherwise weight set by weight set.  A weight set with an odd number of row tiles leaves its last pair half
// empty: the CTA without a tile of its own repeats the other one's loads and keeps nothing (rows_valid = 0).
template <bool kPair>
__device__ __forceinline__ Tile decode_tile(const TcShared& sh, int n_groups, int tile, int uniform_nt, int rank) {
  const RouteState& rs = sh.rs;
  Tile t;
  int g = 0, ul;
  if (uniform_nt > 0) {
    const int n_units = sh.unit0[n_groups];
    t.n_tile = tile / n_units;
    const int u = tile - t.n_tile * n_units;
    while (g + 1 < n_groups && u >= sh.unit0[g + 1]) ++g;
    ul = u - sh.unit0[g];
  } else {
    while (g + 1 < n_groups && tile >= sh.utile0[g + 1]) ++g;
    const int local = tile - sh.utile0[g];
    const int units = sh.unit0[g + 1] - sh.unit0[g];
    t.n_tile = local / units;
    ul = local - t.n_tile * units;
  }
  t.group = g;
  if (kPair) {
    const int mt = rs.group_mtile0[g + 1] - rs.group_mtile0[g];
    const int m_own = 2 * ul + rank, m_peer = 2 * ul + (1 - rank);
    t.m_tile_global = rs.group_mtile0[g] + min(m_own, mt - 1);
    t.m_tile_peer = rs.group_mtile0[g] + min(m_peer, mt - 1);
    t.rows_valid = m_own < mt ? min(kTileM, rs.group_count[g] - m_own * kTileM) : 0;
  } else {
    t.m_tile_global = rs.group_mtile0[g] + ul;
    t.m_tile_peer = t.m_tile_global;
    t.rows_valid = min(kTileM, rs.group_count[g] - ul * kTileM);
  }
  return t;
}

// mode 0: every tile; TopK weight sets emit candidates, the others write Z.
// mode 1: only row tiles flagged by the tail kernel (TopK sets), written to Z for the exact
//         fallback selection; returns at once when nothing is flagged.
__device__ __forceinline__ bool tile_wanted(const Tile& t, const GroupEntry* __restrict__ groups, int mode,
                                            const int* __restrict__ mtile_flag) {
  if (mode == 0) return true;
  return groups[t.group].act == MIX_SAE_TOPK && (mtile_flag[t.m_tile_global] | mtile_flag[t.m_tile_peer]) != 0;   // same answer in both CTAs of a pair
}

// Insert (x, c) into the descending list tv[0..8] if it beats the 9th entry.  Equal values keep
// the earlier (lower) column in front, which is the tie rule of the selection: the new element goes
// in front of the first entry it strictly beats, and everything from there on moves down one place.
__device__ __forceinline__ void top9_insert(float (&tv)[kCandPerTile + 1], int (&ti)[kCandPerTile + 1], float x, int c) {
  if (!(x > tv[kCandPerTile])) return;
  bool moving = false;
#pragma unroll
  for (int s = 0; s <= kCandPerTile; ++s) {
    moving = moving || x > tv[s];
    const float t = tv[s];
    const int u = ti[s];
    tv[s] = moving ? x : t;
    ti[s] = moving ? c : u;
    x = moving ? t : x;
    c = moving ? u : c;
  }
}

template <int kEnc, int kEpi, bool kPair>
__global__ void __launch_bounds__(TcCfg<kEnc, kEpi, kPair>::kThreads, 1)
encode_tc_kernel(const __grid_constant__ CUtensorMap tmap_panel, const CUtensorMap* __restrict__ tmap_w,
                 const RouteState* __restrict__ rs_g, const GroupEntry* __restrict__ groups, int n_groups,
                 float* __restrict__ Z, long long ldz, int d, unsigned* __restrict__ status, int mode,
                 const int* __restrict__ mtile_flag, const int* __restrict__ n_flagged, float* __restrict__ cand_val,
                 int* __restrict__ cand_idx, float* __restrict__ cand_ninth, int cand_tiles, int w_tiled, int test_stall,
                 const float* __restrict__ act_scale, unsigned* __restrict__ tau_slots, unsigned* __restrict__ tau_min,
                 int lo_row0, unsigned long long* __restrict__ clk) {
  constexpr bool kE4 = kEnc != 0;                      // E4M3 x E4M3 contraction
  constexpr bool kSplit = kEnc == 1;                   // the panel row is hi + lo: two operand tiles per k-block
  constexpr int kBlockK = kE4 ? 2 * kTileK : kTileK;   // elements per 128-byte row of either operand
  using Cfg = TcCfg<kEnc, kEpi, kPair>;
  constexpr int kStages = Cfg::kStages;
  constexpr int kStageBytes = Cfg::kStageBytes;
  constexpr int kTcThreads = Cfg::kThreads;
  constexpr int kEpiWarps = Cfg::kEpiWarps;
  constexpr int kEpiCols = kTileN / (kEpiWarps / 4);   // columns of a tile per epilogue warp
  pdl_wait();
  pdl_launch_dependents();
  const bool stamp = clk != nullptr && blockIdx.x == 0 && threadIdx.x == 0 && mode == 0 && !kPair;
  phase_stamp(clk, 26, stamp);
  if (mode == 1 && *n_flagged == 0) return;
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment: required by the 128-byte swizzle atoms
  unsigned char* tiles = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  TcShared* sh = reinterpret_cast<TcShared*>(tiles + Cfg::kRingBytes);
  float* xchg_val = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(sh) + 1024);
  int* xchg_idx = reinterpret_cast<int*>(xchg_val + 2 * 4 * kXchgEntries * 32);
  float* epi_vec = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(sh) + 1024 + Cfg::kXchgBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // CTA pairs: rank 0 leads (it issues the pair's tensor-core instructions and owns the barriers both CTAs' copies
  // complete on); `worker` numbers the units that walk the tile list -- pairs, or single CTAs
  const int rank = kPair ? (int)cluster_ctarank() : 0;
  const bool leader = rank == 0;
  const int worker = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_workers = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  for (int i = threadIdx.x; i < (int)(sizeof(RouteState) / sizeof(int)); i += kTcThreads)
    reinterpret_cast<int*>(&sh->rs)[i] = reinterpret_cast<const int*>(rs_g)[i];
  __syncthreads();
  if (threadIdx.x == 0) {
    {      // this kernel's weight sets: units (row tiles, or pairs of them) and tiles, numbered through
      int nu = 0, ut = 0;
      for (int g = 0; g < n_groups; ++g) {
        const int mt = sh->rs.group_mtile0[g + 1] - sh->rs.group_mtile0[g];
        const int nt = mt > 0 ? (sh->rs.group_tile0[g + 1] - sh->rs.group_tile0[g]) / mt : 0;
        const bool mine = mode != 0 || (((sh->rs.pair_mask >> g) & 1) != 0) == kPair;
        const int units = !mine ? 0 : (kPair ? (mt + 1) / 2 : mt);
        sh->unit0[g] = (short)nu;
        sh->utile0[g] = ut;
        nu += units;
        ut += units * nt;
      }
      for (int g = n_groups; g <= kMaxGroups; ++g) {
        sh->unit0[g] = (short)nu;
        sh->utile0[g] = ut;
      }
    }
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sh->tmem_full[a]), 1);
      mbar_init(smem_u32(&sh->tmem_empty[a]), kPair ? 2 * kEpiWarps : kEpiWarps);   // a pair's leader hears from both CTAs' epilogues
      for (int q = 0; q < 4; ++q) mbar_init(smem_u32(&sh->xchg_full[a][q]), 1);
    }
    sh->abort_flag = 0;
    sh->wait_cycles = test_stall ? kWaitCyclesTest : kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  // the full pass has two kernels, single CTAs and CTA pairs, and the front kernel dealt this call's weight sets
  // between them: nothing routed to any SAE, or no set for this kernel -- no tensor memory is taken (both CTAs
  // of a pair see the same)
  const int total_tiles = sh->utile0[n_groups];
  if (total_tiles == 0) return;

  if (warp == 1) {
    if (kPair) tmem_alloc_pair(smem_u32(&sh->tmem_base), kTmemCols);
    else tmem_alloc(smem_u32(&sh->tmem_base), kTmemCols);
  }
  tc_fence_before();
  if (kPair) cluster_sync_all();           // the peer's barriers are initialised before anything is sent to them
  else __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = sh->tmem_base;
  phase_stamp(clk, 27, stamp);
  // (the interleaved order serves the TopK epilogue's running bound; without TopK rows the plain order is a little faster)
  const int uniform_nt = sh->rs.n_topk_rows > 0 ? uniform_feature_tiles(*sh, n_groups) : 0;
  const int num_kb = d / kBlockK;
  auto tile_of = [&](int tile) { return decode_tile<kPair>(*sh, n_groups, tile, uniform_nt, rank); };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      unsigned phase = 0;
      bool ok = true;
      for (int tile = worker; tile < total_tiles && ok; tile += n_workers) {
        const Tile t = tile_of(tile);
        if (!tile_wanted(t, groups, mode, mtile_flag)) continue;
        const CUtensorMap* tw = tmap_w + t.group;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&sh->empty[stage]), phase ^ 1u, sh, status)) { ok = false; break; }
          // Test hook (MIX_FLAG_TEST_STALL_ENCODE): the producer never fills a stage, so the consumer's
          // bounded wait runs out and the whole CTA leaves through the time-out path.
          if (test_stall) { ok = false; break; }
          const unsigned bar = smem_u32(&sh->full[stage]);
          const unsigned sa = smem_u32(tiles + stage * kStageBytes);
          const unsigned sw = sa + (kSplit ? 2 : 1) * kABytes;
          if (kPair) {
            // both CTAs' copies complete on the LEADER's barrier, which expects the bytes of both; this CTA
            // fetches its own 128 panel rows and its half (128 features) of the W_enc tile
            if (leader) mbar_expect_tx(bar, 2 * kStageBytes);
            const unsigned bar_c = mapa_cluster(bar, 0);
            tma_load_2d_pair(sa, &tmap_panel, kb * kBlockK, t.m_tile_global * kTileM, bar_c);
            if (kSplit) tma_load_2d_pair(sa + kABytes, &tmap_panel, kb * kBlockK, lo_row0 + t.m_tile_global * kTileM, bar_c);
            if (kE4 || w_tiled)
              tma_load_2d_pair(sw, tw, 0, (t.n_tile * num_kb + kb) * kTileN + rank * (kTileN / 2), bar_c);
            else
              tma_load_2d_pair(sw, tw, kb * kTileK, t.n_tile * kTileN + rank * (kTileN / 2), bar_c);
          } else {
            mbar_expect_tx(bar, kStageBytes);
            tma_load_2d(sa, &tmap_panel, kb * kBlockK, t.m_tile_global * kTileM, bar);
            if (kSplit) tma_load_2d(sa + kABytes, &tmap_panel, kb * kBlockK, lo_row0 + t.m_tile_global * kTileM, bar);   // the lo codes
            // W_enc tile: rows n_tile*256.. of the row-major matrix, or -- when the weights were re-laid
            // out at registration (always, for codes) -- block (n_tile, kb) of the tile-contiguous copy
            // [S/256][d/kBlockK][256][kBlockK]
            if (kE4 || w_tiled)
              tma_load_2d(sw, tw, 0, (t.n_tile * num_kb + kb) * kTileN, bar);
            else
              tma_load_2d(sw, tw, kb * kTileK, t.n_tile * kTileN, bar);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      phase_stamp(clk, 28, stamp);          // the last copy of this CTA has been issued
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      int stage = 0;
      unsigned phase = 0, acc = 0, acc_phase = 0;
      bool ok = true;
      for (int tile = worker; tile < total_tiles && ok; tile += n_workers) {
        if (mode != 0 && !tile_wanted(tile_of(tile), groups, mode, mtile_flag)) continue;
        if (!mbar_wait(smem_u32(&sh->tmem_empty[acc]), acc_phase ^ 1u, sh, status)) break;
        tc_fence_after();
        const unsigned d_tmem = tmem_base + acc * kTileN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&sh->full[stage]), phase, sh, status)) { ok = false; break; }
          tc_fence_after();
          const unsigned sa = smem_u32(tiles + stage * kStageBytes);
          const unsigned sb = sa + (kSplit ? 2 : 1) * kABytes;
          const unsigned long long da = umma_desc(sa), db = umma_desc(sb);
#pragma unroll
          for (int k = 0; k < 4; ++k) {   // 16 bf16 or 32 codes = 32 bytes = 2 descriptor units per step
            const unsigned accum = (unsigned)((kb | k) != 0);
            if (kPair) {
              if (kE4) umma_e4m3_pair(d_tmem, da + 2ull * k, db + 2ull * k, kIdescE4Pair, accum);
              else umma_f16_pair(d_tmem, da + 2ull * k, db + 2ull * k, kIdescPair, accum);
            } else {
              if (kE4) umma_e4m3(d_tmem, da + 2ull * k, db + 2ull * k, kIdescE4, accum);
              else umma_f16(d_tmem, da + 2ull * k, db + 2ull * k, kIdesc, accum);
            }
          }
          if (kSplit) {                   // + lo W into the same accumulator
            const unsigned long long dl = umma_desc(sa + kABytes);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              if (kPair) umma_e4m3_pair(d_tmem, dl + 2ull * k, db + 2ull * k, kIdescE4Pair, 1u);
              else umma_e4m3(d_tmem, dl + 2ull * k, db + 2ull * k, kIdescE4, 1u);
            }
          }
          // the stage is free again -- in both CTAs of a pair
          if (kPair) umma_commit_pair(smem_u32(&sh->empty[stage]));
          else umma_commit(smem_u32(&sh->empty[stage]));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (kPair) umma_commit_pair(smem_u32(&sh->tmem_full[acc]));
        else umma_commit(smem_u32(&sh->tmem_full[acc]));
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;                  // tensor-memory lane quarter this warp may read
    const int half = (warp - 2) >> 2;        // 8 epilogue warps: which 128 columns of the tile
    const int c_lo = half * kEpiCols;
    unsigned acc = 0, acc_phase = 0;
    unsigned xchg_phase = 0;                 // bit a: phase of the next hand-over through xchg_full[a][q] (TopK tiles only)
    for (int tile = worker; tile < total_tiles; tile += n_workers) {
      const Tile t = tile_of(tile);
      if (!tile_wanted(t, groups, mode, mtile_flag)) continue;
      const int row_local = q * 32 + lane;
      const bool valid = row_local < t.rows_valid;
      const size_t p = (size_t)t.m_tile_global * kTileM + row_local;
      // TopK tiles: a lower bound on the row's k-th largest pre-activation, from what every CTA has seen of the
      // row so far in this call.  The row's k slots each hold the largest of a disjoint share of the values that
      // tiles already finished published (distinct elements of the row), so once no slot is empty there are k
      // elements >= the smallest slot: nothing below it can be in the TopK, and nearly everything is below it
      // after the first tiles.  Read before the wait for the accumulator; a stale value is merely a lower bound.
      const bool topk_tile = mode == 0 && groups[t.group].act == MIX_SAE_TOPK;
      const int k_row = groups[t.group].k;
      const bool use_tau = topk_tile && valid && tau_slots != nullptr && k_row <= kTauSlots;
      // (tiles of the launch's last wave publish nothing: no tile that starts later is left to read it)
      const bool publish_tau = use_tau && tile + n_workers < total_tiles;
      unsigned tau_key = 0u;                   // 0: no bound yet
      if (use_tau) tau_key = __ldcg(tau_min + p);     // the smallest slot, as of the last time a publisher looked
      // this warp's columns of the bias (and feature scale) go to shared memory now, while the accumulator is
      // still being computed: read from global memory inside the loop below, 32 columns at a time between
      // tensor-memory loads, they were four exposed round trips per tile
      // (Not where both operands are 8-bit and the epilogue selects TopK candidates: there the epilogue, not the
      // main loop, sets the pace -- the accumulator is ready when the warp asks for it -- so a load to wait for in
      // front of every tile costs more than the loads spread over the loop: config 2 with 8-bit operands 240 us
      // against 210 us.  Asking one tile ahead, the vectors held in registers meanwhile, was slower still: 256 us.)
      constexpr bool kScaled = kEnc != 0;      // the accumulator is in units of the codes
      constexpr bool kStageVec = !(kEnc == 2 && kEpi == 8);
      float* wb = epi_vec + (warp - 2) * kEpiCols;
      float* ws = wb + kEpiWarps * kEpiCols;
      const float* bias_t = groups[t.group].b_eff + (size_t)t.n_tile * kTileN + c_lo;
      const float* wsc_t = kScaled ? groups[t.group].w_scale + (size_t)t.n_tile * kTileN + c_lo : nullptr;
      if (kStageVec) {
        const float* bias_g = groups[t.group].b_eff + (size_t)t.n_tile * kTileN + c_lo;
        const float* wsc_g = kScaled ? groups[t.group].w_scale + (size_t)t.n_tile * kTileN + c_lo : nullptr;
        for (int j = lane * 4; j < kEpiCols; j += 128) {
          *reinterpret_cast<float4*>(wb + j) = __ldg(reinterpret_cast<const float4*>(bias_g + j));
          if (kScaled) *reinterpret_cast<float4*>(ws + j) = __ldg(reinterpret_cast<const float4*>(wsc_g + j));
        }
        __syncwarp();
      }
      // warp-uniform decision: tcgen05.ld below needs the whole warp
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&sh->tmem_full[acc]), acc_phase, sh, status))) break;
      tc_fence_after();
      const float ars = kE4 ? (valid ? __ldg(act_scale + p) : 0.f) : 1.f;     // power of two: the products below are exact
      const unsigned taddr = tmem_base + ((unsigned)(q * 32) << 16) + acc * kTileN;
      if (topk_tile) {
        // the list starts out filled with a value just below the bound: whatever is not collected is at most that
        const float tau = tau_key > 1u ? key2f(tau_key) : -INFINITY;
        const float below_tau = tau_key > 1u ? key2f(tau_key - 1u) : -INFINITY;
        float tv[kCandPerTile + 1];
        int ti[kCandPerTile + 1];
#pragma unroll
        for (int s = 0; s <= kCandPerTile; ++s) {
          tv[s] = below_tau;
          ti[s] = 0;
        }
#pragma unroll 1
        for (int c = c_lo; c < c_lo + kEpiCols; c += 32) {
          float v[32];
          tmem_ld32(taddr + c, v);
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 b4 = kStageVec ? *reinterpret_cast<const float4*>(wb + (c - c_lo) + i)
                                        : __ldg(reinterpret_cast<const float4*>(bias_t + (c - c_lo) + i));
            float4 s4 = make_float4(1.f, 1.f, 1.f, 1.f);
            if (kScaled) s4 = kStageVec ? *reinterpret_cast<const float4*>(ws + (c - c_lo) + i)
                                        : __ldg(reinterpret_cast<const float4*>(wsc_t + (c - c_lo) + i));
            if (kE4) { s4.x *= ars; s4.y *= ars; s4.z *= ars; s4.w *= ars; }
            v[i] = kScaled ? fmaf(v[i], s4.x, b4.x) : v[i] + b4.x;
            v[i + 1] = kScaled ? fmaf(v[i + 1], s4.y, b4.y) : v[i + 1] + b4.y;
            v[i + 2] = kScaled ? fmaf(v[i + 2], s4.z, b4.z) : v[i + 2] + b4.z;
            v[i + 3] = kScaled ? fmaf(v[i + 3], s4.w, b4.w) : v[i + 3] + b4.w;
          }
          // (the list's 9th value is at least below_tau, so the test inside top9_insert covers the bound too)
#pragma unroll
          for (int i = 0; i < 32; ++i) top9_insert(tv, ti, v[i], c + i);
        }
        bool writer = true;
        unsigned tau_pub = tau_key;
        if (kEpiWarps == 8) {
          // the upper-half warp hands its list over; the lower-half warp merges it into its own (its columns
          // come first, so equal values keep the lower column in front) and writes the tile's candidates
          float* xv = xchg_val + (size_t)((acc * 4 + q) * kXchgEntries) * 32 + lane;
          int* xi = xchg_idx + (size_t)((acc * 4 + q) * kXchgEntries) * 32 + lane;
          if (half == 1) {
#pragma unroll
            for (int s = 0; s <= kCandPerTile; ++s) {
              xv[s * 32] = tv[s];
              xi[s * 32] = ti[s];
            }
            xi[(kCandPerTile + 1) * 32] = (int)tau_key;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->xchg_full[acc][q]));
            writer = false;
          } else {
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&sh->xchg_full[acc][q]), (xchg_phase >> acc) & 1u, sh, status))) break;
#pragma unroll
            for (int s = 0; s <= kCandPerTile; ++s) top9_insert(tv, ti, xv[s * 32], xi[s * 32]);
            // the two warps may have read the bound at different times: what is at or above the larger one is a
            // real element of the row (each warp's fillers lie below its own bound)
            tau_pub = max(tau_key, (unsigned)xi[(kCandPerTile + 1) * 32]);
          }
        }
        xchg_phase ^= 1u << acc;
        if (valid && writer) {
          const size_t slot = p * (size_t)cand_tiles + (size_t)t.n_tile;
          float4* cv = reinterpret_cast<float4*>(cand_val + slot * kCandPerTile);
          int4* ci = reinterpret_cast<int4*>(cand_idx + slot * kCandPerTile);
          const int j0 = t.n_tile * kTileN;
          cv[0] = make_float4(tv[0], tv[1], tv[2], tv[3]);
          cv[1] = make_float4(tv[4], tv[5], tv[6], tv[7]);
          ci[0] = make_int4(j0 + ti[0], j0 + ti[1], j0 + ti[2], j0 + ti[3]);
          ci[1] = make_int4(j0 + ti[4], j0 + ti[5], j0 + ti[6], j0 + ti[7]);
          cand_ninth[slot] = tv[kCandPerTile];
          if (publish_tau) {
            // this tile's r-th largest goes to slot (n_tile + r k/8) mod k: no two (tile, rank) pairs are the same
            // element, eight consecutive feature tiles fill every slot, and every slot sees all ranks over time
            unsigned* sp = tau_slots + p * kTauSlots;
            bool raised_min = false;
            const int rank_step = max(k_row / kCandPerTile, 1);
            int slot_r = t.n_tile % k_row;
#pragma unroll
            for (int r = 0; r < kCandPerTile; ++r) {
              const unsigned key = f2key(tv[r]);
              if (key >= tau_pub && tv[r] > -INFINITY) {
                const unsigned old = atomicMax(sp + slot_r, key);
                raised_min = raised_min || old < key;      // the smallest slot may have moved up
              }
              slot_r += rank_step;
              if (slot_r >= k_row) slot_r -= k_row;
            }
            if (raised_min) {
              unsigned m = 0xffffffffu;
              for (int j = 0; j < k_row; j += 4) {
                const uint4 w = __ldcg(reinterpret_cast<const uint4*>(sp) + (j >> 2));
                m = min(m, w.x);
                if (j + 1 < k_row) m = min(m, w.y);
                if (j + 2 < k_row) m = min(m, w.z);
                if (j + 3 < k_row) m = min(m, w.w);
              }
              if (m > tau_pub) atomicMax(tau_min + p, m);
            }
          }
        }
      } else {
        float* out = Z + p * (size_t)ldz + (size_t)t.n_tile * kTileN;
#pragma unroll 1
        for (int c = c_lo; c < c_lo + kEpiCols; c += 32) {
          float v[32];
          tmem_ld32(taddr + c, v);
          if (valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const float4 b4 = kStageVec ? *reinterpret_cast<const float4*>(wb + (c - c_lo) + i)
                                          : __ldg(reinterpret_cast<const float4*>(bias_t + (c - c_lo) + i));
              float4 s4 = make_float4(1.f, 1.f, 1.f, 1.f);
              if (kScaled) s4 = kStageVec ? *reinterpret_cast<const float4*>(ws + (c - c_lo) + i)
                                          : __ldg(reinterpret_cast<const float4*>(wsc_t + (c - c_lo) + i));
              if (kE4) { s4.x *= ars; s4.y *= ars; s4.z *= ars; s4.w *= ars; }
              float4 o;
              o.x = kScaled ? fmaf(v[i], s4.x, b4.x) : v[i] + b4.x;
              o.y = kScaled ? fmaf(v[i + 1], s4.y, b4.y) : v[i + 1] + b4.y;
              o.z = kScaled ? fmaf(v[i + 2], s4.z, b4.z) : v[i + 2] + b4.z;
              o.w = kScaled ? fmaf(v[i + 3], s4.w, b4.w) : v[i + 3] + b4.w;
              *reinterpret_cast<float4*>(out + c + i) = o;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {     // the accumulator is free: tell the CTA that issues the instructions
        if (kPair && !leader) mbar_arrive_cluster(mapa_cluster(smem_u32(&sh->tmem_empty[acc]), 0));
        else mbar_arrive(smem_u32(&sh->tmem_empty[acc]));
      }
      acc ^= 1u;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (sh->abort_flag) {
    // give copies that are still in flight time to land before shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) __nanosleep(1000);
  }
  // a pair leaves together: neither CTA's barriers or tensor memory go away while the other may still reach them
  if (kPair) cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    if (kPair) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
  phase_stamp(clk, 29, stamp);
}

// Registration-time copy of W_enc [S, d] into [S/256][d/64][256][64]: one thread per 16 bytes.
__global__ void retile_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, long long d_sae, int d) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;      // index of a 16-byte piece of dst
  const int num_kb = d / kTileK;
  const long long total = d_sae * (long long)d / 8;
  if (i >= total) return;
  const int piece = (int)(i & 7);                       // 8 pieces per 64-column row
  const long long row_in_all = i >> 3;                  // row of the [.., 256, 64] blocks
  const int r = (int)(row_in_all % kTileN);
  const long long blk = row_in_all / kTileN;
  const int kb = (int)(blk % num_kb);
  const long long n_tile = blk / num_kb;
  dst[i] = src[((n_tile * kTileN + r) * (long long)d + (long long)kb * kTileK) / 8 + piece];
}

// The same for 8-bit codes: [S, d] bytes -> [S/256][d/kb_bytes][256][kb_bytes] bytes (kb_bytes = 64 for the
// widening kernel, 128 for the 8-bit contraction), one thread per 16 bytes.
__global__ void retile_fp8_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, long long d_sae, int d, int kb_bytes) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int num_kb = d / kb_bytes;
  const int ppr = kb_bytes / 16;                        // 16-byte pieces per block row
  const long long total = d_sae * (long long)d / 16;
  if (i >= total) return;
  const int piece = (int)(i % ppr);
  const long long row_in_all = i / ppr;
  const int r = (int)(row_in_all % kTileN);
  const long long blk = row_in_all / kTileN;
  const int kb = (int)(blk % num_kb);
  const long long n_tile = blk / num_kb;
  dst[i] = src[((n_tile * kTileN + r) * (long long)d + (long long)kb * kb_bytes) / 16 + piece];
}

}  // namespace

cudaError_t launch_retile_fp8(const unsigned char* W_enc, unsigned char* W_tiled, long long d_sae, int d, int kb_bytes,
                              cudaStream_t s) {
  const long long total = d_sae * (long long)d / 16;
  retile_fp8_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(reinterpret_cast<const uint4*>(W_enc),
                                                                    reinterpret_cast<uint4*>(W_tiled), d_sae, d, kb_bytes);
  return cudaGetLastError();
}

cudaError_t launch_retile(const __nv_bfloat16* W_enc, __nv_bfloat16* W_tiled, long long d_sae, int d, cudaStream_t s) {
  const long long total = d_sae * (long long)d / 8;
  retile_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(reinterpret_cast<const uint4*>(W_enc),
                                                                reinterpret_cast<uint4*>(W_tiled), d_sae, d);
  return cudaGetLastError();
}

template <int kEnc, int kEpi, bool kPair>
static cudaError_t encode_tc_prepare_as() {
  return cudaFuncSetAttribute(encode_tc_kernel<kEnc, kEpi, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              TcCfg<kEnc, kEpi, kPair>::kSmemBytes);
}

cudaError_t encode_tc_prepare() {
  cudaError_t e = encode_tc_prepare_as<0, 4, false>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<0, 8, false>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<1, 4, false>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<1, 8, false>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<2, 4, false>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<2, 8, false>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<0, 4, true>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<0, 8, true>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<1, 4, true>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<1, 8, true>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<2, 4, true>();
  if (e == cudaSuccess) e = encode_tc_prepare_as<2, 8, true>();
  return e;
}

// CTA pairs or single CTAs: MIX_ENCODE_PAIR in the environment (0 / 1), read once; set by mix_set_encode_pair for A/B timing.
static int g_encode_pair = -1;
int encode_pair_mode(int set) {
  if (g_encode_pair < 0) {
    const int v = getenv("MIX_ENCODE_PAIR") ? atoi(getenv("MIX_ENCODE_PAIR")) : kEncodePairDefault;
    g_encode_pair = v == 0 || v == 1 ? v : 2;
  }
  const int old = g_encode_pair;
  if (set >= 0) g_encode_pair = set == 0 || set == 1 ? set : 2;
  return old;
}

template <int kEnc, int kEpi, bool kPair>
static cudaError_t launch_encode_tc_as(const Ctx* c, int mode, cudaStream_t s) {
  using Cfg = TcCfg<kEnc, kEpi, kPair>;
  const int w_tiled = (c->cfg.flags & MIX_FLAG_RETILE_W_ENC) ? 1 : 0;
  const int stall = (c->cfg.flags & MIX_FLAG_TEST_STALL_ENCODE) ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kPair ? (c->n_sms & ~1) : c->n_sms);
  cfg.blockDim = dim3(Cfg::kThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute at[2];
  int n_at = 0;
  if (kPair) {
    at[n_at].id = cudaLaunchAttributeClusterDimension;
    at[n_at].val.clusterDim.x = 2;
    at[n_at].val.clusterDim.y = 1;
    at[n_at].val.clusterDim.z = 1;
    ++n_at;
  }
  if (pdl_mask() & (mode == 0 ? kPdlEncode : kPdlTail)) {
    at[n_at].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n_at].val.programmaticStreamSerializationAllowed = 1;
    ++n_at;
  }
  cfg.attrs = at;
  cfg.numAttrs = n_at;
  const CUtensorMap* tmap_w = kPair ? c->d_tmap_w_half : c->d_tmap_w;
  return cudaLaunchKernelEx(&cfg, encode_tc_kernel<kEnc, kEpi, kPair>, c->tmap_panel, tmap_w,
                            static_cast<const RouteState*>(c->d_route), static_cast<const GroupEntry*>(c->d_groups),
                            c->cfg.n_groups_max, c->d_z, (long long)c->cfg.d_sae_max, c->cfg.d_model, c->d_status, mode,
                            static_cast<const int*>(c->d_mtile_flag), static_cast<const int*>(c->d_n_flagged), c->d_cand_val,
                            c->d_cand_idx, c->d_cand_ninth, c->cand_tiles, w_tiled, stall,
                            static_cast<const float*>(c->d_act_scale), c->d_tau, c->d_tau_min, c->panel_rows_cap,
                            c->d_phase_clk);
}

// Eight epilogue warps pay off for the TopK epilogue (selection work per element); the plain store of the
// pre-activations is a little faster with four.  Either form is correct for any mix of weight sets; the choice
// is made from the sets registered when the call is enqueued (or captured).
// pair: the CTA-pair kernel (256-row tiles) or the single-CTA kernel; a full pass (mode 0) launches both, and
// the one the front kernel did not choose for this call returns at once.
cudaError_t launch_encode_tc(const Ctx* c, int mode, bool pair, cudaStream_t s) {
  bool topk = false;
  for (int g = 0; g < c->cfg.n_groups_max; ++g) topk = topk || (c->h_groups[g].valid && c->h_groups[g].act == MIX_SAE_TOPK);
  if (pair) {
    if (c->cfg.flags & MIX_FLAG_FP8_ACT) return topk ? launch_encode_tc_as<2, 8, true>(c, mode, s) : launch_encode_tc_as<2, 4, true>(c, mode, s);
    if (c->cfg.flags & MIX_FLAG_FP8_W_ENC) return topk ? launch_encode_tc_as<1, 8, true>(c, mode, s) : launch_encode_tc_as<1, 4, true>(c, mode, s);
    return topk ? launch_encode_tc_as<0, 8, true>(c, mode, s) : launch_encode_tc_as<0, 4, true>(c, mode, s);
  }
  if (c->cfg.flags & MIX_FLAG_FP8_ACT) return topk ? launch_encode_tc_as<2, 8, false>(c, mode, s) : launch_encode_tc_as<2, 4, false>(c, mode, s);
  if (c->cfg.flags & MIX_FLAG_FP8_W_ENC) return topk ? launch_encode_tc_as<1, 8, false>(c, mode, s) : launch_encode_tc_as<1, 4, false>(c, mode, s);
  return topk ? launch_encode_tc_as<0, 8, false>(c, mode, s) : launch_encode_tc_as<0, 4, false>(c, mode, s);
}

bool encode_pair_possible(const Ctx* c) { return encode_pair_mode(-1) != 0 && c->cfg.T_max > kTileM; }

}  // namespace mix
