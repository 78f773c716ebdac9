// bf16 weight GEMM on the 5th-generation tensor cores (sm_100a): y[M, N] (+)= x[M, K] * W[N, K]^T.
//
// The weight matrix is the streamed operand, so it takes the 128-row side of the instruction:
// each CTA owns a tile of 128 output features (rows of W) and MT rows of x, and computes
// D^T[128, MT] = W_tile[128, K] * x_tile[MT, K]^T with tcgen05.mma (A = W tile, B = x tile, both
// K-major in shared memory under the 128-byte swizzle, staged by TMA; accumulator in TMEM).  With
// MT = 16..64 the same kernel is a bandwidth-bound skinny GEMM for decode (weights read once, MMA
// cost hidden); with MT = 256 it is the dense GEMM of prefill / PRM scoring / catch-up.
//
// Roles inside a CTA of 6 warps: warps 0-3 read the accumulator out of TMEM (lane = output feature,
// column = x row) and write y, warp 4 issues TMA loads through a ring of shared-memory stages,
// warp 5 allocates TMEM and issues the MMAs.  Small problems are split along K across CTAs; the
// partial tiles go to scratch and the last CTA to arrive adds them in split order (deterministic).
// Every wait on an mbarrier is bounded; on expiry the CTA raises an error flag and leaves cleanly.
#include <cuda.h>

#include <atomic>
#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace rsd {

static std::atomic<uint64_t> g_launches{0};
cudaError_t launched(int n_kernels) {
  g_launches.fetch_add((uint64_t)n_kernels, std::memory_order_relaxed);
  return cudaGetLastError();
}
uint64_t launches_total() { return g_launches.load(std::memory_order_relaxed); }
void note_replayed_launches(uint64_t n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

namespace {

using namespace tc;

constexpr int kTileN = 128;        // W rows per CTA (UMMA M)
constexpr int kTileK = 64;         // bf16 elements per 128-byte swizzled row
constexpr int kUmmaK = 16;
constexpr int kCounterBytes = 4096;
constexpr int kMaxSplitTiles = kCounterBytes / 4;
constexpr int kMaxSplitCtas = 640;

// DEEP: a ring of eight (six for 128-row x tiles) stages for one CTA per SM, for grids that do not reach two CTAs per SM anyway (a lone
// CTA needs about twice the bytes in flight to keep its share of the HBM stream going).
template <int MT, bool DEEP = false> struct TcCfg {
  // tiles of up to 128 x-rows leave room for two CTAs per SM (one streams while the other starts
  // up or drains); the 256-row tile of the dense regime takes the SM alone
  static constexpr int kCtasPerSm = DEEP ? 1 : (MT <= 128 ? 2 : 1);
  static constexpr int kStages = DEEP ? (MT <= 64 ? 8 : 6) : (MT <= 32 ? 5 : (MT == 64 ? 4 : (MT == 128 ? 3 : 4)));
  static constexpr int kABytes = kTileN * kTileK * 2;
  static constexpr int kBBytes = MT * kTileK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTmemCols = MT < 32 ? 32 : MT;
  static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256 + 512;   // barriers, row scales
  // gate/up mode: two exchange buffers [64 features][MT / 4 rows + 1] between the gate and the up warps; they
  // reuse the pipeline stages once the last MMA has read them
  static constexpr size_t kXchBytes = 2 * 64 * (size_t)(MT / 4 + 1) * 4;
  static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
  static_assert(kXchBytes <= (size_t)kStages * kStageBytes, "exchange buffers must fit in the stage ring");
  // instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, N = MT, M = 128
  static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(MT >> 3) << 17) | ((uint32_t)(kTileN >> 4) << 24);
};

// SPLIT: the x operand is a pair (hi, lo) of bf16 matrices whose sum is the activation; the tile
// holds MT/2 rows of hi followed by the same MT/2 rows of lo, and the epilogue adds the two halves.
// GU (gate/up mode, SPLIT only): W is the stacked matrix [Wgate | Wup] of 2 * N rows; a CTA's 128-row tile is
// 64 gate rows and the 64 up rows of the same features (two TMA boxes of 64 rows), there is no K split, and the
// epilogue writes act = silu(gate) * up as the bf16 hi + lo operand pair [M, N] of the down projection instead
// of Y.  The gate values sit in TMEM lanes 0-63 (warps 0, 1), the up values in lanes 64-127 (warps 2, 3); the
// two warp pairs swap one half of the x rows each through shared memory, so all four warps compute.
// PROBE (one instantiation, reached only through the wait-probe entry): the producer warp issues NO copy, so the
// first stage never fills; the MMA warp's wait, cut to a few thousand polls, runs out, and the kernel must take its
// failure path -- error flag raised, epilogue warps released, tensor memory freed, clean return -- with nothing in
// flight.  This is how the failure path is exercised without a fault or an endless wait.
template <int MT, bool SPLIT, bool GU = false, bool DEEP = false, bool PROBE = false>
__global__ void __launch_bounds__(192, TcCfg<MT, DEEP>::kCtasPerSm)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
               const __grid_constant__ CUtensorMap tm_x_lo, float* __restrict__ Y,
               int M, int N, int K, int accumulate, int splits, int kb_per_split, float* __restrict__ partials,
               int* __restrict__ err, const int32_t* __restrict__ n_active, RowScale rs,
               __nv_bfloat16* __restrict__ act_hi = nullptr, __nv_bfloat16* __restrict__ act_lo = nullptr) {
  // Programmatic dependent launch: the next kernel may be scheduled at once; this kernel sets itself
  // up and starts streaming its WEIGHT tiles (never written by any kernel) while its predecessors are
  // still running, and only then waits for them (griddepcontrol.wait) before it touches activations,
  // outputs or the idle flag.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  using Cfg = TcCfg<MT, DEEP>;
  constexpr int kRows = SPLIT ? MT / 2 : MT;   // distinct x rows per tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(smem + (size_t)Cfg::kStages * Cfg::kStageBytes);
  uint64_t* empty = full + Cfg::kStages;
  uint64_t* tmem_full = empty + Cfg::kStages;
  uint32_t* tmem_slot = (uint32_t*)(tmem_full + 1);
  volatile uint32_t* flags = tmem_slot + 1;   // [0] abort
  float* row_scale = (float*)(smem + (size_t)Cfg::kStages * Cfg::kStageBytes + 256);   // [kRows <= 128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Tile order.  CTAs start in the order of their linear index; with n fastest, the CTAs in flight together would
  // hold as many different weight tiles as there are SMs and the weight matrix would come from HBM once per row
  // tile of x.  With several row tiles the index is therefore walked in groups of eight row tiles, row tile
  // fastest: the CTAs in flight share eight x tiles and a few weight tiles, both of which stay in L2.
  int tile_n = blockIdx.x, tile_m = blockIdx.y;
  if (gridDim.y > 1) {
    constexpr int kGroup = 8;
    const int lin = blockIdx.y * gridDim.x + blockIdx.x, per_group = kGroup * gridDim.x;
    const int g0 = (lin / per_group) * kGroup, rem = lin % per_group;
    const int gsz = min(kGroup, (int)gridDim.y - g0);
    tile_m = g0 + rem % gsz;
    tile_n = rem / gsz;
  }
  const int n0 = tile_n * (GU ? kTileN / 2 : kTileN), m0 = tile_m * kRows, split = blockIdx.z;
  float* xch = (float*)smem;   // GU only: the exchange buffers reuse the pipeline stages, which are drained by then
  const int total_kb = (K + kTileK - 1) / kTileK;
  const int kb0 = split * kb_per_split;
  const int kb1 = min(total_kb, kb0 + kb_per_split);
  const int n_kb = kb1 - kb0;   // >= 1 by construction of the grid

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(tmem_full, 1);
    flags[0] = 0; flags[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(tmem_slot, Cfg::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (lane == 0 && !PROBE) {
      int issued = 0;
      bool ok = true;
      // weight tiles of the first ring of stages go out before the predecessors have finished
      const int pre = min(n_kb, Cfg::kStages);
      for (int i = 0; i < pre; ++i) {
        mbar_expect_tx(&full[i], Cfg::kStageBytes);
        uint8_t* a = smem + (size_t)i * Cfg::kStageBytes;
        if (GU) {
          tma_load_2d(a, &tm_w, &full[i], (kb0 + i) * kTileK, n0);
          tma_load_2d(a + Cfg::kABytes / 2, &tm_w, &full[i], (kb0 + i) * kTileK, N + n0);
        } else {
          tma_load_2d(a, &tm_w, &full[i], (kb0 + i) * kTileK, n0);
        }
      }
      issued = pre;
      asm volatile("griddepcontrol.wait;" ::: "memory");
      // every row of the decode phase has finished: complete the copies that are in flight (their
      // x halves are fetched too so that the stage barriers close), then leave without computing
      const bool idle = n_active != nullptr && *n_active == 0;
      if (idle) flags[0] = 2;
      for (int i = 0; i < pre; ++i) {
        uint8_t* a = smem + (size_t)i * Cfg::kStageBytes;
        tma_load_2d(a + Cfg::kABytes, &tm_x, &full[i], (kb0 + i) * kTileK, m0);
        if (SPLIT) tma_load_2d(a + Cfg::kABytes + kRows * kTileK * 2, &tm_x_lo, &full[i], (kb0 + i) * kTileK, m0);
      }
      if (idle) {
        for (int i = 0; i < pre; ++i) mbar_wait(&full[i], 0);
      } else {
        for (int i = pre; i < n_kb && ok; ++i) {
          const int s = i % Cfg::kStages;
          ok = mbar_wait(&empty[s], ((i / Cfg::kStages) - 1) & 1);
          if (!ok || flags[0]) { ok = false; break; }
          uint8_t* a = smem + (size_t)s * Cfg::kStageBytes;
          mbar_expect_tx(&full[s], Cfg::kStageBytes);
          if (GU) {
            tma_load_2d(a, &tm_w, &full[s], (kb0 + i) * kTileK, n0);
            tma_load_2d(a + Cfg::kABytes / 2, &tm_w, &full[s], (kb0 + i) * kTileK, N + n0);
          } else {
            tma_load_2d(a, &tm_w, &full[s], (kb0 + i) * kTileK, n0);
          }
          tma_load_2d(a + Cfg::kABytes, &tm_x, &full[s], (kb0 + i) * kTileK, m0);
          if (SPLIT) tma_load_2d(a + Cfg::kABytes + kRows * kTileK * 2, &tm_x_lo, &full[s], (kb0 + i) * kTileK, m0);
          issued = i + 1;
        }
        if (!ok) {
          if (err && flags[0] != 2) atomicCAS(err, 0, -5);
          if (flags[0] == 0) flags[0] = 1;
          // let the copies already in flight land before the CTA goes away
          for (int i = max(0, issued - Cfg::kStages); i < issued; ++i)
            mbar_wait(&full[i % Cfg::kStages], (i / Cfg::kStages) & 1);
        }
      }
    }
  } else if (warp == 5) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      bool ok = true;
      for (int i = 0; i < n_kb; ++i) {
        const int s = i % Cfg::kStages;
        ok = mbar_wait(&full[s], (i / Cfg::kStages) & 1, PROBE ? 4096u : kWaitLimit);
        if (!ok || flags[0]) { ok = false; break; }
        tc_fence_after();
        const uint32_t a = smem_u32(smem + (size_t)s * Cfg::kStageBytes);
        const uint32_t b = a + Cfg::kABytes;
#pragma unroll
        for (int k = 0; k < kTileK / kUmmaK; ++k) {
          umma_bf16(tmem_base, smem_desc_sw128(a + k * kUmmaK * 2), smem_desc_sw128(b + k * kUmmaK * 2), Cfg::kIdesc,
                    (i > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(&empty[s]);   // frees the stage once these MMAs have read it
      }
      if (ok) {
        umma_commit(tmem_full);
      } else if (flags[0] == 0) {      // a wait of this thread expired (flags[0] != 0: someone else stopped the CTA)
        if (err) atomicCAS(err, 0, -5);
        flags[0] = 1;
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> global ----------------
    asm volatile("griddepcontrol.wait;" ::: "memory");   // y and the partial sums belong to earlier kernels until now
    if (rs.ssq != nullptr) {
      // RMSNorm denominators of this tile's x rows, one per epilogue thread, while the MMAs run
      const int r = threadIdx.x;
      if (r < kRows && m0 + r < M) {
        float sum = 0.f;
        for (int c = 0; c < rs.n_chunks; ++c) sum += rs.ssq[(size_t)(m0 + r) * rs.n_chunks + c];
        row_scale[r] = rsqrtf(sum * rs.inv_d + rs.eps);
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");   // the four epilogue warps only
    }
    // the four epilogue warps sleep in hardware between polls (about 1 us at most): busy polling by 128 threads
    // crowds the shared-memory pipe that the producer and the MMA issuer need for their own barriers
    bool ok = mbar_try_wait(tmem_full, 0);
    for (uint32_t i = 0; i < (1u << 21) && !ok; ++i) {
      ok = mbar_try_wait_sleep(tmem_full, 0, 1000);
      if (!ok && flags[0]) break;                        // the CTA was stopped (idle phase or an expired wait)
    }
    if (!ok && flags[0] == 0) {
      if (err) atomicCAS(err, 0, -5);
      flags[0] = 1;
    }
    tc_fence_after();
    const int n_local = warp * 32 + lane;
    const int n = n0 + n_local;
    const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
    const int m_valid = min(kRows, M - m0);
    if (GU) {
      // SwiGLU epilogue.  Rows [0, half) of the tile are finished by the gate warps (they receive the up values
      // of those rows), rows [half, kRows) by the up warps (they receive the gate values).
      constexpr int kHalf = kRows / 2, kLd = kHalf + 1;
      const bool is_gate = warp < 2;
      const int l = (warp & 1) * 32 + lane;                    // feature within the 64-row half
      float* send = xch + (is_gate ? 64 * kLd : 0) + l * kLd;  // [0]: up values of the low rows, [1]: gate values of the high rows
      const float* recv = xch + (is_gate ? 0 : 64 * kLd) + l * kLd;
      const int send0 = is_gate ? kHalf : 0, own0 = is_gate ? 0 : kHalf;
      if (ok) {
#pragma unroll 1
        for (int c = 0; c < kHalf; c += 16) {
          float v[16], w[16];
          tmem_ld16(taddr + send0 + c, v);
          tmem_ld16(taddr + kRows + send0 + c, w);
#pragma unroll
          for (int j = 0; j < 16; ++j) send[c + j] = v[j] + w[j];
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ok && n0 + l < N) {
#pragma unroll 1
        for (int c = 0; c < kHalf; c += 16) {
          if (own0 + c >= m_valid) break;
          float v[16], w[16];
          tmem_ld16(taddr + own0 + c, v);
          tmem_ld16(taddr + kRows + own0 + c, w);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int r = own0 + c + j;
            if (r < m_valid) {
              const float sc = rs.ssq != nullptr ? row_scale[r] : 1.f;
              const float mine = (v[j] + w[j]) * sc, other = recv[c + j] * sc;
              const float gate = is_gate ? mine : other, up = is_gate ? other : mine;
              const float a = gate / (1.f + expf(-gate)) * up;
              const size_t o = (size_t)(m0 + r) * N + n0 + l;
              const __nv_bfloat16 h = __float2bfloat16_rn(a);
              act_hi[o] = h;
              act_lo[o] = __float2bfloat16_rn(a - __bfloat162float(h));
            }
          }
        }
      }
    } else if (ok) {
      // with several K-splits each CTA stores its partial sums as rows of a [split][M][N] array;
      // a reduction kernel adds the splits in order afterwards (deterministic)
      float* dst = splits == 1 ? Y : partials + (size_t)split * M * N;
      for (int c = 0; c < m_valid; c += 16) {
        float v[16];
        tmem_ld16(taddr + c, v);
        if (SPLIT) {
          if (kRows == 8) {          // hi in columns 0..7, lo in columns 8..15 of the same load
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] += v[j + 8];
          } else {
            float w[16];
            tmem_ld16(taddr + kRows + c, w);
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] += w[j];
          }
        }
        if (rs.ssq != nullptr) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c + j < m_valid) v[j] *= row_scale[c + j];
        }
        if (n < N) {
          // when adding into y, all sixteen old values are requested before the first store: written as
          // "*y += v" row by row, every load would wait for the store before it (the compiler cannot rule out
          // that two rows alias) and the epilogue would crawl at one memory round trip per element
          if (accumulate && splits == 1) {
            float old[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) old[j] = c + j < m_valid ? dst[(size_t)(m0 + c + j) * N + n] : 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] += old[j];
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            if (c + j < m_valid) dst[(size_t)(m0 + c + j) * N + n] = v[j];
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------------------
// Persistent form of the kernel above for the dense regime (more than 128 rows of x, split-precision operand, no
// K split): a CTA per SM walks the output tiles (128 weight rows x 128 x rows, the same grouped order), the TMA
// ring runs on from tile to tile, and the accumulator alternates between the two halves of tensor memory, so
// the epilogue of one tile (TMEM -> registers -> global) overlaps the MMAs of the next instead of ending the CTA.
// GU: gate/up tiles with the SwiGLU epilogue as above; the exchange buffers get shared memory of their own, since
// the ring is busy with the next tile.
// ---------------------------------------------------------------------------------------------------------
// SPLIT: the x tile is 128 rows of hi followed by the same 128 rows of lo (the epilogue adds the halves); otherwise it is
// 256 plain rows.  Either way the instruction's N is 256 and an accumulator takes 256 columns of tensor memory.
template <bool SPLIT, bool GU> struct PersistCfg {
  static constexpr int kMT = 256, kRows = SPLIT ? 128 : 256;
  static constexpr int kHalf = kRows / 2, kLd = kHalf + 1;
  static constexpr size_t kXchBytes = GU ? 2 * 64 * (size_t)kLd * 4 : 0;
  // the exchange buffers of the plain gate/up tile (2 x 64 x 129 floats) leave room for three stages
  static constexpr int kStages = (GU && !SPLIT) ? 3 : 4;
  static constexpr int kABytes = kTileN * kTileK * 2, kBBytes = kMT * kTileK * 2, kStageBytes = kABytes + kBBytes;
  static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256 + kXchBytes;
  static constexpr uint32_t kIdesc = TcCfg<256>::kIdesc;
  static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
};

// warps 0..7: epilogue, warp 8: TMA producer, warp 9: MMA issuer and owner of the tensor-memory allocation
constexpr int kPersistEpiWarps = 8, kPersistThreads = 32 * (kPersistEpiWarps + 2);

template <bool GU, bool SPLIT>
__global__ void __launch_bounds__(kPersistThreads, 1)
gemm_tc_persistent_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
                          const __grid_constant__ CUtensorMap tm_x_lo, float* __restrict__ Y, int M, int N, int K,
                          int accumulate, int n_tiles_n, int n_tiles_m, int* __restrict__ err,
                          __nv_bfloat16* __restrict__ act_hi, __nv_bfloat16* __restrict__ act_lo, int f16) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  using C = PersistCfg<SPLIT, GU>;
  // f16: both operands are fp16 (weights re-encoded at load, one fp16 activation operand); the MMA's operand-format
  // fields become 0 and a gate/up tile writes its activations as fp16.  Otherwise bf16 throughout.
  const uint32_t idesc = f16 ? (C::kIdesc & ~((1u << 7) | (1u << 10))) : C::kIdesc;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(smem + (size_t)C::kStages * C::kStageBytes);
  uint64_t* empty = full + C::kStages;
  uint64_t* acc_full = empty + C::kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
  volatile uint32_t* stop = tmem_slot + 1;
  float* xch = (float*)(smem + (size_t)C::kStages * C::kStageBytes + 256);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_kb = (K + kTileK - 1) / kTileK, n_tiles = n_tiles_n * n_tiles_m;
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], kPersistEpiWarps); }
    *stop = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kPersistEpiWarps + 1) tmem_alloc(tmem_slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // tile t -> (row tile of x, tile of W): groups of eight row tiles, row tile fastest
  auto tile_of = [&](int t, int& tm, int& tn) {
    const int per_group = 8 * n_tiles_n, g0 = (t / per_group) * 8, rem = t % per_group, gsz = min(8, n_tiles_m - g0);
    tm = g0 + rem % gsz;
    tn = rem / gsz;
  };
  auto fail = [&]() { if (*stop == 0) { if (err) atomicCAS(err, 0, -5); *stop = 1; } };

  if (warp == kPersistEpiWarps) {
    if (lane == 0) {
      uint32_t it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*stop; t += gridDim.x) {
        int tm, tn;
        tile_of(t, tm, tn);
        const int n0 = tn * (GU ? kTileN / 2 : kTileN), m0 = tm * C::kRows;
        for (int kb = 0; kb < total_kb; ++kb, ++it) {
          const uint32_t s = it % C::kStages;
          if (!mbar_wait(&empty[s], ((it / C::kStages) & 1u) ^ 1u) || *stop) { fail(); break; }
          uint8_t* a = smem + (size_t)s * C::kStageBytes;
          mbar_expect_tx(&full[s], C::kStageBytes);
          if (GU) {
            tma_load_2d(a, &tm_w, &full[s], kb * kTileK, n0);
            tma_load_2d(a + C::kABytes / 2, &tm_w, &full[s], kb * kTileK, N + n0);
          } else {
            tma_load_2d(a, &tm_w, &full[s], kb * kTileK, n0);
          }
          tma_load_2d(a + C::kABytes, &tm_x, &full[s], kb * kTileK, m0);
          if (SPLIT) tma_load_2d(a + C::kABytes + C::kRows * kTileK * 2, &tm_x_lo, &full[s], kb * kTileK, m0);
        }
      }
      if (*stop) {   // copies in flight must land before the CTA goes away
        for (uint32_t i = (it > (uint32_t)C::kStages ? it - C::kStages : 0); i < it; ++i)
          for (uint32_t k = 0; k < (1u << 16); ++k)
            if (mbar_try_wait(&full[i % C::kStages], (i / C::kStages) & 1u)) break;
      }
    }
  } else if (warp == kPersistEpiWarps + 1) {
    if (lane == 0) {
      uint32_t it = 0, n_acc = 0;
      for (int t = blockIdx.x; t < n_tiles && !*stop; t += gridDim.x, ++n_acc) {
        const uint32_t b = n_acc & 1u;
        if (!mbar_wait(&acc_empty[b], ((n_acc >> 1) & 1u) ^ 1u) || *stop) { fail(); break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + b * (uint32_t)C::kMT;
        bool ok = true;
        for (int kb = 0; kb < total_kb; ++kb, ++it) {
          const uint32_t s = it % C::kStages;
          if (!mbar_wait(&full[s], (it / C::kStages) & 1u) || *stop) { ok = false; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(smem + (size_t)s * C::kStageBytes), bb = a + C::kABytes;
#pragma unroll
          for (int k = 0; k < kTileK / kUmmaK; ++k)
            umma_bf16(d_tmem, smem_desc_sw128(a + k * kUmmaK * 2), smem_desc_sw128(bb + k * kUmmaK * 2), idesc,
                      (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(&empty[s]);
        }
        if (!ok) { fail(); break; }
        umma_commit(&acc_full[b]);
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    // eight of them: warp w reads the tensor-memory lanes of quarter w % 4 (the hardware's rule), the two warps of a
    // quarter take alternate groups of sixteen columns, which halves the time an accumulator stays occupied
    const int quarter = warp & 3, col0 = (warp >> 2) * 16;
    constexpr int kColStep = 16 * (kPersistEpiWarps / 4);
    uint32_t n_acc = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++n_acc) {
      int tm, tn;
      tile_of(t, tm, tn);
      const int n0 = tn * (GU ? kTileN / 2 : kTileN), m0 = tm * C::kRows;
      const uint32_t b = n_acc & 1u;
      bool ok = mbar_try_wait(&acc_full[b], (n_acc >> 1) & 1u);
      for (uint32_t i = 0; i < (1u << 21) && !ok && !*stop; ++i) ok = mbar_try_wait_sleep(&acc_full[b], (n_acc >> 1) & 1u, 1000);
      if (!ok) fail();
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * (uint32_t)C::kMT;
      const int m_valid = min(C::kRows, M - m0);
      if (!GU) {
        const int n = n0 + quarter * 32 + lane;
        if (ok) {
          for (int c = col0; c < m_valid; c += kColStep) {
            float v[16];
            tmem_ld16(taddr + c, v);
            if (SPLIT) {
              float w[16];
              tmem_ld16(taddr + C::kRows + c, w);
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] += w[j];
            }
            if (n < N) {
              // all sixteen old values first, then the stores (see the one-tile kernel's epilogue)
              if (accumulate) {
                float old[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) old[j] = c + j < m_valid ? Y[(size_t)(m0 + c + j) * N + n] : 0.f;
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] += old[j];
              }
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                if (c + j < m_valid) Y[(size_t)(m0 + c + j) * N + n] = v[j];
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[b]);
      } else {
        const bool is_gate = quarter < 2;
        const int l = (quarter & 1) * 32 + lane;
        float* send = xch + (is_gate ? 64 * C::kLd : 0) + l * C::kLd;
        const float* recv = xch + (is_gate ? 0 : 64 * C::kLd) + l * C::kLd;
        const int send0 = is_gate ? C::kHalf : 0, own0 = is_gate ? 0 : C::kHalf;
        if (ok) {
#pragma unroll 1
          for (int c = col0; c < C::kHalf; c += kColStep) {
            float v[16];
            tmem_ld16(taddr + send0 + c, v);
            if (SPLIT) {
              float w[16];
              tmem_ld16(taddr + C::kRows + send0 + c, w);
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] += w[j];
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) send[c + j] = v[j];
          }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kPersistEpiWarps) : "memory");
        if (ok && n0 + l < N) {
#pragma unroll 1
          for (int c = col0; c < C::kHalf; c += kColStep) {
            if (own0 + c >= m_valid) break;
            float v[16];
            tmem_ld16(taddr + own0 + c, v);
            if (SPLIT) {
              float w[16];
              tmem_ld16(taddr + C::kRows + own0 + c, w);
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] += w[j];
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int r = own0 + c + j;
              if (r < m_valid) {
                const float mine = v[j], other = recv[c + j];
                const float gate = is_gate ? mine : other, up = is_gate ? other : mine;
                const float a = gate / (1.f + expf(-gate)) * up;
                const size_t o = (size_t)(m0 + r) * N + n0 + l;
                if (!SPLIT && f16) {
                  reinterpret_cast<__half*>(act_hi)[o] = __float2half_rn(a);
                } else {
                  const __nv_bfloat16 h = __float2bfloat16_rn(a);
                  act_hi[o] = h;
                  if (SPLIT) act_lo[o] = __float2bfloat16_rn(a - __bfloat162float(h));
                }
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[b]);
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kPersistEpiWarps) : "memory");   // the exchange buffers are free for the next tile
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kPersistEpiWarps + 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// y[m, n] (+)= sum over splits of partials[s][m][n], splits added in order; 4 columns per thread.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ partials, float* __restrict__ Y, int M, int N, int splits, int accumulate,
                     const int32_t* __restrict__ n_active) {
  RSD_PDL_SYNC();
  if (n_active != nullptr && *n_active == 0) return;
  const size_t total4 = (size_t)M * N / 4, stride = (size_t)M * N / 4;
  const float4* p4 = reinterpret_cast<const float4*>(partials);
  float4* y4 = reinterpret_cast<float4*>(Y);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total4; i += (size_t)gridDim.x * blockDim.x) {
    float4 acc = accumulate ? y4[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    int sidx = 0;
    for (; sidx + 4 <= splits; sidx += 4) {
      const float4 a = __ldcg(p4 + (size_t)sidx * stride + i), b = __ldcg(p4 + (size_t)(sidx + 1) * stride + i);
      const float4 c = __ldcg(p4 + (size_t)(sidx + 2) * stride + i), d = __ldcg(p4 + (size_t)(sidx + 3) * stride + i);
      acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
      acc.x += b.x; acc.y += b.y; acc.z += b.z; acc.w += b.w;
      acc.x += c.x; acc.y += c.y; acc.z += c.z; acc.w += c.w;
      acc.x += d.x; acc.y += d.y; acc.z += d.z; acc.w += d.w;
    }
    for (; sidx < splits; ++sidx) {
      const float4 a = __ldcg(p4 + (size_t)sidx * stride + i);
      acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
    }
    y4[i] = acc;
  }
}

// ---- tensor maps (host) -----------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  });
  return fn;
}

struct MapKey {
  const void* ptr; int rows, cols, box_rows;
  bool operator==(const MapKey& o) const { return ptr == o.ptr && rows == o.rows && cols == o.cols && box_rows == o.box_rows; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = std::hash<const void*>()(k.ptr);
    h ^= std::hash<long long>()(((long long)k.rows << 32) ^ ((long long)k.cols << 8) ^ k.box_rows) + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2);
    return h;
  }
};

// Row-major bf16 matrix [rows, cols]; box = 64 columns x box_rows rows; 128-byte swizzle.  Maps are
// cached by (pointer, shape): weights and activation buffers keep their addresses for a context's life.
bool get_map(const void* ptr, int rows, int cols, int box_rows, CUtensorMap* out) {
  static std::mutex mu;
  static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  std::lock_guard<std::mutex> lock(mu);
  MapKey key{ptr, rows, cols, box_rows};
  auto it = cache.find(key);
  if (it != cache.end()) { *out = it->second; return true; }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 65536) cache.clear();
  cache.emplace(key, m);
  *out = m;
  return true;
}

// Rows of x per tile: the smallest tile that holds M, up to 128 (split operand) or 256 (plain).
int pick_rows(int M, bool split_operand) {
  if (split_operand && M <= 8) return 8;
  if (M <= 16) return 16;
  if (M <= 32) return 32;
  if (M <= 64) return 64;
  if (M <= 128 || split_operand) return 128;
  return 256;
}

struct TcPlan { int rows, mt, n_tiles, m_tiles, splits, kb_per_split; };

TcPlan plan_tc(int M, int N, int K, bool split_operand) {
  TcPlan p;
  p.rows = pick_rows(M, split_operand);
  p.mt = split_operand ? 2 * p.rows : p.rows;
  p.n_tiles = (N + kTileN - 1) / kTileN;
  p.m_tiles = (M + p.rows - 1) / p.rows;
  const int tiles = p.n_tiles * p.m_tiles;
  const int total_kb = (K + kTileK - 1) / kTileK;
  int splits = 1;
  if (tiles < 148 && tiles <= kMaxSplitTiles && p.rows <= 64 && N % 4 == 0) {
    // aim at one wave of two CTAs per SM, each with at least two k-blocks
    splits = std::max(1, (2 * 148) / tiles);
    splits = std::min(splits, std::max(1, total_kb / 2));
    splits = std::min(splits, kMaxSplitCtas / tiles);
    splits = std::max(splits, 1);
  }
  p.kb_per_split = (total_kb + splits - 1) / splits;
  p.splits = (total_kb + p.kb_per_split - 1) / p.kb_per_split;   // no empty split
  return p;
}

template <int MT, bool SPLIT, bool DEEP = false>
cudaError_t launch_mt(const CUtensorMap& tw, const CUtensorMap& tx, const CUtensorMap& txl, float* y, int M, int N, int K,
                      int accumulate, const TcPlan& p, float* partials, int* err, const int32_t* n_active,
                      bool defer_reduce, RowScale rs, cudaStream_t s) {
  using Cfg = TcCfg<MT, DEEP>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<MT, SPLIT, false, DEEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(p.n_tiles, p.m_tiles, p.splits);
  RSD_LAUNCH((gemm_tc_kernel<MT, SPLIT, false, DEEP>), grid, 192, Cfg::kSmemBytes, s, tw, tx, txl, y, M, N, K, accumulate, p.splits,
                                                                     p.kb_per_split, partials, err, n_active, rs,
                                                                     (__nv_bfloat16*)nullptr, (__nv_bfloat16*)nullptr);
  if (p.splits > 1 && !defer_reduce) {
    const size_t total4 = (size_t)M * N / 4;
    const int blocks = (int)std::min<size_t>((total4 + 255) / 256, 148 * 8);
    RSD_LAUNCH((splitk_reduce_kernel), blocks, 256, 0, s, partials, y, M, N, p.splits, accumulate, n_active);
    return launched(2);
  }
  return launched(1);
}

}  // namespace

// Row-major bf16 matrix [rows, cols] as a TMA tensor map with a 64-column x box_rows box under the 128-byte swizzle.
bool tc_tensor_map(const void* ptr, int rows, int cols, int box_rows, CUtensorMap* out) {
  return get_map(ptr, rows, cols, box_rows, out);
}

// One layer's slab of fp16 KV pages as a tensor of 4096-byte blocks (per page: the keys of every KV head
// [16 tokens][128 dims], then the values [128 dims][16 tokens]), one box per block:
//   keys    (64 dims, 8 tokens, 2 dim halves, 2 token groups, block)   128-byte swizzle: lands as
//           [token group][dim half][8 tokens][64 dims], the order the score MMA wants its operand in
//   values  (16 tokens, 128 dims, block)                               32-byte swizzle
// The block extent is a bound on what a coordinate may name, not an allocation size: only the boxes a kernel asks
// for are touched.
bool tc_tensor_map_kv(const void* pool_layer, int values, CUtensorMap* out) {
  static std::mutex mu;
  static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  std::lock_guard<std::mutex> lock(mu);
  MapKey key{pool_layer, values, 0, 0};
  auto it = cache.find(key);
  if (it != cache.end()) { *out = it->second; return true; }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  CUtensorMap m;
  const cuuint64_t blocks = 1ull << 30;
  CUresult r;
  if (values) {
    cuuint64_t dims[3] = {16, 128, blocks};
    cuuint64_t strides[2] = {32, 4096};
    cuuint32_t box[3] = {16, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(pool_layer), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    cuuint64_t dims[5] = {64, 8, 2, 2, blocks};
    cuuint64_t strides[4] = {256, 128, 2048, 4096};      // token, dim half, token group, block
    cuuint32_t box[5] = {64, 8, 2, 2, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, const_cast<void*>(pool_layer), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 65536) cache.clear();
  cache.emplace(key, m);
  *out = m;
  return true;
}

// Launches the PROBE instantiation on a 128 x 16 x 64 problem whose copies are never issued (W and x are mapped but
// not read): the kernel's bounded wait expires and *err (the int at byte 4096 of the scratch) becomes -5.
cudaError_t launch_gemm_wait_probe(const void* W, const void* x, float* y, void* scratch, size_t scratch_bytes, cudaStream_t s) {
  if (!scratch || scratch_bytes < gemm_scratch_bytes(16)) return cudaErrorInvalidValue;
  CUtensorMap tw, tx;
  if (!get_map(W, 128, 64, kTileN, &tw) || !get_map(x, 16, 64, 16, &tx)) return cudaErrorNotSupported;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<16, false, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)TcCfg<16>::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  int* err = (int*)((char*)scratch + kCounterBytes);
  float* partials = (float*)((char*)scratch + kCounterBytes + 256);
  RSD_LAUNCH((gemm_tc_kernel<16, false, false, false, true>), dim3(1, 1, 1), 192, TcCfg<16>::kSmemBytes, s, tw, tx, tx, y, 16, 128, 64, 0, 1, 1,
             partials, err, (const int32_t*)nullptr, RowScale(), (__nv_bfloat16*)nullptr, (__nv_bfloat16*)nullptr);
  return launched(1);
}

bool gemm_tc_supported(int dtype, int M, int N, int K) {
  return dtype == 1 && M >= 1 && N >= 1 && K >= 8 && K % 8 == 0;
}

static int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
  }
  return n;
}

// Dense regime (M > 128 rows, no K split, no row scale, no idle flag): persistent kernel.
template <bool GU, bool SPLIT>
static cudaError_t launch_persistent(const CUtensorMap& tw, const CUtensorMap& tx, const CUtensorMap& txl, float* y, int M, int N,
                                     int K, int accumulate, int* err, __nv_bfloat16* act_hi, __nv_bfloat16* act_lo, cudaStream_t s,
                                     int f16 = 0) {
  using C = PersistCfg<SPLIT, GU>;
  constexpr size_t smem = C::kSmemBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_persistent_kernel<GU, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int n_sm = sm_count();
  if (n_sm <= 0) return cudaErrorInvalidDevice;
  const int tiles_n = GU ? N / 64 : (N + kTileN - 1) / kTileN, tiles_m = (M + C::kRows - 1) / C::kRows;
  const int grid = std::min(tiles_n * tiles_m, n_sm);
  RSD_LAUNCH((gemm_tc_persistent_kernel<GU, SPLIT>), grid, kPersistThreads, smem, s, tw, tx, txl, y, M, N, K, accumulate, tiles_n,
             tiles_m, err, act_hi, act_lo, f16);
  return launched(1);
}

template <int MT, bool DEEP>
static cudaError_t launch_gu_mt(const CUtensorMap& tw, const CUtensorMap& tx, const CUtensorMap& txl, int M, int F, int K, int rows,
                                int* err, const int32_t* n_active, RowScale rs, __nv_bfloat16* act_hi, __nv_bfloat16* act_lo,
                                cudaStream_t s) {
  constexpr size_t smem = TcCfg<MT, DEEP>::kSmemBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<MT, true, true, DEEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int total_kb = (K + kTileK - 1) / kTileK;
  dim3 grid(F / 64, (M + rows - 1) / rows, 1);
  RSD_LAUNCH((gemm_tc_kernel<MT, true, true, DEEP>), grid, 192, smem, s, tw, tx, txl, (float*)nullptr, M, F, K, 0, 1, total_kb,
             (float*)nullptr, err, n_active, rs, act_hi, act_lo);
  return launched(1);
}

bool gemm_gu_supported(int dtype, int M, int F, int K) {
  return dtype == 1 && M >= 1 && F >= 64 && F % 64 == 0 && K >= 8 && K % 8 == 0;
}

// act (hi + lo, bf16 [M, F]) = silu(g) * u with [g | u] = rowscale * (x_hi + x_lo)[M, K] * Wgu[2F, K]^T.
cudaError_t launch_gemm_gu(const void* Wgu, const void* x, const void* x_lo, void* act_hi, void* act_lo, int M, int F, int K,
                           void* scratch, size_t scratch_bytes, const int32_t* n_active, cudaStream_t s, RowScale rs) {
  if (M <= 0) return cudaSuccess;
  if (!gemm_gu_supported(1, M, F, K) || !act_hi) return cudaErrorNotSupported;
  if (!scratch || scratch_bytes < (size_t)kCounterBytes + 256) return cudaErrorInvalidValue;
  if (((uintptr_t)Wgu & 15) || ((uintptr_t)x & 15) || ((uintptr_t)x_lo & 15)) return cudaErrorMisalignedAddress;
  int* err = (int*)((char*)scratch + kCounterBytes);
  CUtensorMap tw, tx, txl;
  if (x_lo == nullptr) {
    // plain bf16 operand: the persistent kernel only (more than 128 rows, no row scale, no idle flag)
    if (!(M > 128 && rs.ssq == nullptr && n_active == nullptr)) return cudaErrorNotSupported;
    if (!get_map(Wgu, 2 * F, K, kTileN / 2, &tw) || !get_map(x, M, K, 256, &tx)) return cudaErrorNotSupported;
    return launch_persistent<true, false>(tw, tx, tx, nullptr, M, F, K, 0, err, (__nv_bfloat16*)act_hi, nullptr, s);
  }
  if (!act_lo) return cudaErrorNotSupported;
  // at least 32 x rows per tile: each warp pair finishes one half of them, 16 at a time
  const int rows = M <= 32 ? 32 : (M <= 64 ? 64 : 128);
  if (rs.ssq != nullptr && rows > 128) return cudaErrorInvalidValue;
  if (!get_map(Wgu, 2 * F, K, kTileN / 2, &tw) || !get_map(x, M, K, rows, &tx) || !get_map(x_lo, M, K, rows, &txl))
    return cudaErrorNotSupported;
  if (M > 128 && rs.ssq == nullptr && n_active == nullptr)
    return launch_persistent<true, true>(tw, tx, txl, nullptr, M, F, K, 0, err, (__nv_bfloat16*)act_hi, (__nv_bfloat16*)act_lo, s);
  auto* hi = (__nv_bfloat16*)act_hi;
  auto* lo = (__nv_bfloat16*)act_lo;
  // fewer than ~1.5 CTAs per SM: one CTA per SM with a deep ring streams faster than a thin second wave
  const bool deep = (F / 64) * ((M + rows - 1) / rows) <= 222;
  switch (rows) {
    case 32: return deep ? launch_gu_mt<64, true>(tw, tx, txl, M, F, K, rows, err, n_active, rs, hi, lo, s)
                         : launch_gu_mt<64, false>(tw, tx, txl, M, F, K, rows, err, n_active, rs, hi, lo, s);
    case 64: return deep ? launch_gu_mt<128, true>(tw, tx, txl, M, F, K, rows, err, n_active, rs, hi, lo, s)
                         : launch_gu_mt<128, false>(tw, tx, txl, M, F, K, rows, err, n_active, rs, hi, lo, s);
    default: return launch_gu_mt<256, false>(tw, tx, txl, M, F, K, rows, err, n_active, rs, hi, lo, s);
  }
}

// Layout of the scratch: [0, 4096) tile counters (kept zero between launches), then one int error
// flag region of 256 bytes, then split-K partial tiles.
size_t gemm_scratch_bytes(int M) {
  const int rows = pick_rows(M, false);
  const size_t part = rows <= 64 ? (size_t)kMaxSplitCtas * kTileN * std::min(64, std::max(rows, 16)) * 4 : 0;
  return kCounterBytes + 256 + part;
}

// Enough for any M (split-K is only used with tiles of at most 64 rows of x).
size_t gemm_scratch_bytes_any() { return gemm_scratch_bytes(64); }

const float* gemm_partials(const void* scratch) { return (const float*)((const char*)scratch + kCounterBytes + 256); }

cudaError_t launch_gemm_tc(const void* W, const void* x, const void* x_lo, float* y, int M, int N, int K, int accumulate,
                           void* scratch, size_t scratch_bytes, const int32_t* n_active, int* deferred_splits,
                           cudaStream_t s, RowScale rs, bool no_k_split) {
  if (deferred_splits) *deferred_splits = 1;
  if (M <= 0) return cudaSuccess;
  if (rs.ssq != nullptr && accumulate) return cudaErrorInvalidValue;
  if (!scratch || scratch_bytes < gemm_scratch_bytes(M)) return cudaErrorInvalidValue;
  if (((uintptr_t)W & 15) || ((uintptr_t)x & 15) || ((uintptr_t)x_lo & 15)) return cudaErrorMisalignedAddress;
  const bool split_operand = x_lo != nullptr;
  TcPlan p = plan_tc(M, N, K, split_operand);
  if (no_k_split) { p.splits = 1; p.kb_per_split = (K + kTileK - 1) / kTileK; }
  if (rs.ssq != nullptr && p.rows > 128) return cudaErrorInvalidValue;   // one epilogue thread per x row of the tile
  if (deferred_splits) *deferred_splits = p.splits;
  const bool defer = deferred_splits != nullptr;
  CUtensorMap tw, tx, txl;
  if (!get_map(W, N, K, kTileN, &tw) || !get_map(x, M, K, p.rows, &tx)) return cudaErrorNotSupported;
  if (split_operand) { if (!get_map(x_lo, M, K, p.rows, &txl)) return cudaErrorNotSupported; }
  else txl = tx;
  int* err = (int*)((char*)scratch + kCounterBytes);
  float* partials = (float*)((char*)scratch + kCounterBytes + 256);
  if (M > 128 && p.splits == 1 && rs.ssq == nullptr && n_active == nullptr) {
    if (split_operand) return launch_persistent<false, true>(tw, tx, txl, y, M, N, K, accumulate, err, nullptr, nullptr, s);
    return launch_persistent<false, false>(tw, tx, txl, y, M, N, K, accumulate, err, nullptr, nullptr, s);
  }
#define RSD_TC(MT, SP) return launch_mt<MT, SP>(tw, tx, txl, y, M, N, K, accumulate, p, partials, err, n_active, defer, rs, s)
  // a grid of at most one CTA per SM: the deep ring (a lone CTA needs more bytes in flight to keep its stream going)
  if (split_operand && p.n_tiles * p.m_tiles * p.splits <= 148 && p.mt <= 128) {
#define RSD_TCD(MT) return launch_mt<MT, true, true>(tw, tx, txl, y, M, N, K, accumulate, p, partials, err, n_active, defer, rs, s)
    switch (p.mt) {
      case 16: RSD_TCD(16);
      case 32: RSD_TCD(32);
      case 64: RSD_TCD(64);
      default: RSD_TCD(128);
    }
#undef RSD_TCD
  }
  if (split_operand) {
    switch (p.mt) {
      case 16: RSD_TC(16, true);
      case 32: RSD_TC(32, true);
      case 64: RSD_TC(64, true);
      case 128: RSD_TC(128, true);
      default: RSD_TC(256, true);
    }
  }
  switch (p.mt) {
    case 16: RSD_TC(16, false);
    case 32: RSD_TC(32, false);
    case 64: RSD_TC(64, false);
    case 128: RSD_TC(128, false);
    default: RSD_TC(256, false);
  }
#undef RSD_TC
}

// Dense products (more than 128 rows) with fp16 weights and ONE fp16 activation operand: the persistent kernel with
// the operand formats switched.  y [M, N] fp32 (+)= x [M, K] W [N, K]^T.
cudaError_t launch_gemm_f16_dense(const void* W16, const void* x16, float* y, int M, int N, int K, int accumulate,
                                  void* scratch, size_t scratch_bytes, cudaStream_t s) {
  if (M <= 128 || !gemm_tc_supported(1, M, N, K)) return cudaErrorNotSupported;
  if (!scratch || scratch_bytes < gemm_scratch_bytes(M)) return cudaErrorInvalidValue;
  if (((uintptr_t)W16 & 15) || ((uintptr_t)x16 & 15)) return cudaErrorMisalignedAddress;
  TcPlan p = plan_tc(M, N, K, false);
  CUtensorMap tw, tx;
  if (!get_map(W16, N, K, kTileN, &tw) || !get_map(x16, M, K, p.rows, &tx)) return cudaErrorNotSupported;
  int* err = (int*)((char*)scratch + kCounterBytes);
  return launch_persistent<false, false>(tw, tx, tx, y, M, N, K, accumulate, err, nullptr, nullptr, s, 1);
}

// act [M, F] fp16 = silu(g) * u with [g | u] = x [M, K] Wgu [2F, K]^T, fp16 operands, more than 128 rows.
cudaError_t launch_gemm_gu_f16_dense(const void* Wgu16, const void* x16, void* act16, int M, int F, int K, void* scratch,
                                     size_t scratch_bytes, cudaStream_t s) {
  if (M <= 128 || !gemm_gu_supported(1, M, F, K) || !act16) return cudaErrorNotSupported;
  if (!scratch || scratch_bytes < (size_t)kCounterBytes + 256) return cudaErrorInvalidValue;
  if (((uintptr_t)Wgu16 & 15) || ((uintptr_t)x16 & 15)) return cudaErrorMisalignedAddress;
  int* err = (int*)((char*)scratch + kCounterBytes);
  CUtensorMap tw, tx;
  if (!get_map(Wgu16, 2 * F, K, kTileN / 2, &tw) || !get_map(x16, M, K, 256, &tx)) return cudaErrorNotSupported;
  return launch_persistent<true, false>(tw, tx, tx, nullptr, M, F, K, 0, err, (__nv_bfloat16*)act16, nullptr, s, 1);
}

cudaError_t launch_gemm(int dtype, const void* W, const void* x, const void* x_lo, float* y, int M, int N, int K,
                        int accumulate, int impl, void* scratch, size_t scratch_bytes, const int32_t* n_active,
                        int* deferred_splits, cudaStream_t s, RowScale rs) {
  if (deferred_splits) *deferred_splits = 1;
  const bool tc_ok = gemm_tc_supported(dtype, M, N, K) && scratch && scratch_bytes >= gemm_scratch_bytes(M);
  // the tensor-core path wins for every M (an M = 1 GEMV included: TMA streaming beats the SIMT loads)
  if (impl == 2 || impl == 3 || (impl == 0 && tc_ok))
    return launch_gemm_tc(W, x, x_lo, y, M, N, K, accumulate, scratch, scratch_bytes, n_active, deferred_splits, s, rs, impl == 3);
  if (rs.ssq != nullptr) return cudaErrorNotSupported;
  return launch_gemm_simt(dtype, W, x, dtype == 1 ? x_lo : nullptr, y, M, N, K, accumulate, n_active, s);
}

}  // namespace rsd
