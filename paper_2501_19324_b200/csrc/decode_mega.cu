// Persistent decode kernel (sm_100a): the whole layer stack of one decode iteration of a bf16 model in ONE
// launch, one CTA per SM.
//
// A decode iteration over a few dozen rows is a chain of some eight dependent stages per layer, each far too
// short to fill the machine for long; as separate kernels their fixed costs add up to several times the time
// the weights need to stream from HBM.  Here the stages are phases of one kernel separated by a grid-wide
// barrier, and the weight stream never stops at a phase boundary:
//
//   warp 8   W producer   TMA loads of weight tiles [128 rows x 64 k] into a ring of shared-memory stages.
//                         Weights depend on nothing, so this warp never takes part in a barrier: it runs
//                         ahead through phases and layers as far as the ring allows.
//   warp 9   X producer   TMA loads of the activation tiles (hi + lo bf16 rows) of the current GEMM phase.
//   warp 10  MMA issuer   tcgen05.mma, weights as the 128-row A operand, activations as B, fp32
//                         accumulators in tensor memory (two buffers, so the epilogue of one work item
//                         overlaps the MMAs of the next).
//   warps 0-3             GEMM epilogues (TMEM -> registers -> global) and, with warps 4-7, the phases
//                         that are not GEMMs.
//
// Phases of a layer (RMSNorm is folded into its neighbours: the phase that completes the residual stream
// writes x * gain as the next operand and the sums of squares, the consuming GEMM scales its result rows):
//   qkv GEMM (K-split partial sums)  |  RoPE + KV page write + paged attention + merge of the context splits
//   | wo GEMM  |  residual + norm operand  |  gate/up GEMM with SwiGLU in the epilogue (a CTA's tile holds 64
//   gate rows and the 64 matching up rows)  |  down GEMM  |  residual + norm operand.
// Every wait (mbarrier, grid barrier) is bounded; on expiry an error flag is raised, the remaining phases
// are skipped and the kernel ends in order.
#include <cuda.h>

#include <algorithm>
#include <new>
#include <vector>

#include "common.cuh"
#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace rsd {

namespace {

using namespace tc;

constexpr int kGenThreads = 256;      // warps 0-7
constexpr int kThreads = 352;         // + W producer, X producer, MMA issuer
constexpr int kWarpW = 8, kWarpX = 9, kWarpMma = 10;
constexpr int kPhaseThreads = 320;    // everyone but the W producer meets at the phase barrier
constexpr int kWStageBytes = 128 * 64 * 2;
constexpr int kGenScratchBytes = 8 * 8 * 128 * 4 + 2 * 8 * 8 * 4 + 8 * 128 * 4;   // attention: outputs, (max, sum), q
constexpr uint32_t kGridSpinLimit = 1u << 22;
constexpr int kMaxStamps = 1022;
constexpr int kXchBytes = 64 * 65 * 4;

struct GemmPlan {
  int N, K, n_tiles, splits, kbps, total_kb;
};

struct alignas(128) MegaLayer {
  CUtensorMap w[4];                    // qkv, wo, gate/up (box of 64 rows), down
  const __nv_bfloat16* norm1;
  const __nv_bfloat16* norm2;
  char* kv_layer;
};

struct alignas(128) MegaParams {
  CUtensorMap xmap[6];                 // h hi, h lo, attn hi, attn lo, act hi, act lo
  GemmPlan plan[4];
  int L, d, H, KV, F, B, rows, mt, sw, sx, attn_splits, max_pages, tmem_cols;
  float eps;
  const __nv_bfloat16* embed;
  float* x;
  __nv_bfloat16 *h_hi, *h_lo, *attn_hi, *attn_lo, *act_hi, *act_lo;
  float* partials;
  float* ssq;                          // [B][d / 128]
  float *part_o, *part_ml;             // attention context-split partials
  int32_t* attn_cnt;                   // [B * KV] arrivals of the context splits (zero between uses)
  unsigned* grid_bar;                  // [0] arrivals, [1] generation
  int* err;
  const float2* rope;
  const int32_t* page_table;
  unsigned long long* prof;            // debug: CTA 0 stamps the global timer before and after every grid barrier
};

// ---- small helpers ------------------------------------------------------------------------------
__device__ __forceinline__ void bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

struct Shared {
  uint8_t* wring;
  uint8_t* xring;
  float* gen;            // attention scratch; aliases the X ring, which is idle outside the GEMM phases
  float* xch;            // gate/up exchange of the SwiGLU epilogue [64][65]
  float* row_scale;      // [64]
  uint64_t *full_w, *empty_w, *full_x, *empty_x, *acc_full, *acc_empty;
  uint32_t* tmem_slot;
  volatile int* abort_flag;
  volatile int* go;
  volatile int* flag;
  int* pref;             // [B + 1] prefix sums of the rows' page counts, [B + 1] = the largest count
};

// Bounded wait that also gives up when another role has stopped the CTA.  Waiters sleep in hardware between
// polls (about 2 us at most, so ~2 s in all before the wait is given up).
constexpr uint32_t kSleepNs = 2000;
constexpr uint32_t kSleepPolls = 1u << 20;
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, const Shared& sh, int* err) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t i = 0; i < kSleepPolls; ++i) {
    if (mbar_try_wait_sleep(bar, parity, kSleepNs)) return true;
    if (*sh.abort_flag) return false;
  }
  *sh.abort_flag = 1;
  atomicCAS(err, 0, -5);
  return false;
}

// Grid-wide barrier for everyone but the W producer.  grid_bar[0] counts arrivals and only grows during a
// launch: barrier number k is passed once it reads k * gridDim.x.  Thread 0 arrives with a one-way release
// reduction and polls with acquire loads; the CTA barriers on both sides extend the ordering to the other
// threads.  The last CTA to leave the kernel puts the counter back to zero (finish_grid_sync).
__device__ __forceinline__ void grid_sync(const MegaParams& P, const Shared& sh, unsigned& epoch, int& n_stamps) {
  if (P.prof != nullptr && blockIdx.x == 0 && threadIdx.x == 0 && n_stamps < kMaxStamps) P.prof[n_stamps++] = global_timer();
  fence_async_proxy();          // activations written with plain stores are read by TMA after the barrier
  bar_sync(1, kPhaseThreads);
  if (threadIdx.x == 0) {
    if (!*sh.abort_flag) {
      ++epoch;
      const unsigned target = epoch * gridDim.x;
      asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(P.grid_bar) : "memory");
      bool ok = false;
      for (uint32_t i = 0; i < kGridSpinLimit; ++i) {
        if (ld_acquire(P.grid_bar) >= target) { ok = true; break; }
        if ((i & 255u) == 255u && __ldcg(P.err) != 0) break;
      }
      if (!ok) { *sh.abort_flag = 1; atomicCAS(P.err, 0, -5); }
    }
    *sh.go = *sh.abort_flag ? 0 : 1;
  }
  bar_sync(1, kPhaseThreads);
  fence_async_proxy();
  if (P.prof != nullptr && blockIdx.x == 0 && threadIdx.x == 0 && n_stamps < kMaxStamps) P.prof[n_stamps++] = global_timer();
}

// Called by thread 0 of every CTA after its last barrier: the last one to come resets both counters.
__device__ __forceinline__ void finish_grid_sync(const MegaParams& P) {
  __threadfence();
  const unsigned old = atomicAdd(P.grid_bar + 1, 1u);
  if (old == gridDim.x - 1) {
    P.grid_bar[0] = 0u;
    P.grid_bar[1] = 0u;
    __threadfence();
  }
}

struct Item { int tile, split, kb0, kb1; };
__device__ __forceinline__ Item item_of(const GemmPlan& g, int it) {
  Item r;
  r.tile = it % g.n_tiles;
  r.split = it / g.n_tiles;
  r.kb0 = r.split * g.kbps;
  r.kb1 = min(g.total_kb, r.kb0 + g.kbps);
  return r;
}

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// ---- residual + norm operand phase ----------------------------------------------------------------
// One warp per (row, 128-column chunk): x (+)= sum of the K-split partial sums (or x = embedding row);
// hi + lo = x * gain; ssq[row][chunk] = sum of x^2 over the chunk.
__device__ __forceinline__ void rn_phase(const MegaParams& P, const PassView& pv, int splits, const __nv_bfloat16* gain,
                                         bool from_embed) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp >= 8) return;
  const int d = P.d, nch = d >> 7, items = P.B * nch;
  for (int it = blockIdx.x * 8 + warp; it < items; it += gridDim.x * 8) {
    const int m = it / nch, c = it - m * nch;
    if (pv.tok_row[m] < 0) continue;
    const int col = c * 128 + lane * 4;
    const size_t o = (size_t)m * d + col;
    float4 v;
    if (from_embed) {
      const uint2 e = *reinterpret_cast<const uint2*>(P.embed + (size_t)pv.tok_id[m] * d + col);
      v.x = __uint_as_float(e.x << 16); v.y = __uint_as_float(e.x & 0xFFFF0000u);
      v.z = __uint_as_float(e.y << 16); v.w = __uint_as_float(e.y & 0xFFFF0000u);
    } else {
      v = ldcg4(P.x + o);
      const size_t stride = (size_t)P.B * d;
      int s = 0;
      for (; s + 4 <= splits; s += 4) {
        float4 a[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) a[u] = ldcg4(P.partials + (size_t)(s + u) * stride + o);
#pragma unroll
        for (int u = 0; u < 4; ++u) { v.x += a[u].x; v.y += a[u].y; v.z += a[u].z; v.w += a[u].w; }
      }
      for (; s < splits; ++s) {
        const float4 a = ldcg4(P.partials + (size_t)s * stride + o);
        v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
      }
    }
    *reinterpret_cast<float4*>(P.x + o) = v;
    const uint2 gq = *reinterpret_cast<const uint2*>(gain + col);
    const float g0 = __uint_as_float(gq.x << 16), g1 = __uint_as_float(gq.x & 0xFFFF0000u);
    const float g2 = __uint_as_float(gq.y << 16), g3 = __uint_as_float(gq.y & 0xFFFF0000u);
    const float w[4] = {v.x * g0, v.y * g1, v.z * g2, v.w * g3};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      hi[j] = __float2bfloat16_rn(w[j]);
      lo[j] = __float2bfloat16_rn(w[j] - __bfloat162float(hi[j]));
    }
    *reinterpret_cast<uint2*>(P.h_hi + o) = *reinterpret_cast<const uint2*>(hi);
    *reinterpret_cast<uint2*>(P.h_lo + o) = *reinterpret_cast<const uint2*>(lo);
    float ss = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    ss = warp_sum(ss);
    if (lane == 0) P.ssq[(size_t)m * nch + c] = ss;
  }
}

// ---- attention phase ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void pack_h2_split(float a, float b, uint32_t& hi, uint32_t& lo) {
  const __half ah = __float2half_rn(a), bh = __float2half_rn(b);
  hi = pack_h2(__half2float(ah), __half2float(bh));
  lo = pack_h2(a - __half2float(ah), b - __half2float(bh));
}
__device__ __forceinline__ void mma_f16(float& d0, float& d1, float& d2, float& d3, uint32_t a0, uint32_t a1, uint32_t a2,
                                        uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3)
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldcg_u4(const __half* p) { return __ldcg(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ uint2 ldcg_u2(const __half* p) { return __ldcg(reinterpret_cast<const uint2*>(p)); }

// Sums over the K-split partial sums of the qkv product for two columns of one slot.  All loads of a group of
// eight splits (sixteen loads) are in flight together; the sums stay in split order.
__device__ __forceinline__ void qkv_sum2(const MegaParams& P, int slot, int col_a, int col_b, float& a, float& b) {
  const GemmPlan& g = P.plan[0];
  const size_t stride = (size_t)P.B * g.N;
  const float* pa = P.partials + (size_t)slot * g.N + col_a;
  const float* pb = P.partials + (size_t)slot * g.N + col_b;
  const int splits = g.splits;
  a = 0.f; b = 0.f;
  for (int s0 = 0; s0 < splits; s0 += 8) {
    float ta[8], tb[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const bool in = s0 + u < splits;
      ta[u] = in ? __ldcg(pa + (size_t)(s0 + u) * stride) : 0.f;
      tb[u] = in ? __ldcg(pb + (size_t)(s0 + u) * stride) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) { a += ta[u]; b += tb[u]; }
  }
}

// The (row slot, KV head, page) triples of the iteration are laid end to end (slot-major, then head, then
// page) and cut into equal chunks, one per CTA, so every CTA walks the same number of pages whatever the
// rows' context lengths.  A chunk is a few segments, each a page range of one (slot, head) pair, served by
// the eight general warps: the rotated queries of the head group are rebuilt from the qkv partial sums, the
// segment that holds the pair's newest page also rotates the new key and writes it and the new value into
// that page, then every warp walks its share of the 16-token pages with m16n8k16 MMAs (queries of the group
// as rows).  A pair cut into several segments is merged by the last of them to finish.
constexpr int kMaxParts = 32;

template <bool EXT>
__device__ __forceinline__ void attn_phase(const MegaParams& P, const MegaLayer& Ly, const PassView& pv, const Shared& sh) {
  constexpr int HD = 128, KB = HD / 32, NT = HD / 8;
  const int tid = threadIdx.x;
  if (tid >= kGenThreads) return;
  const int warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int H = P.H, KV = P.KV, G = H / KV;
  float* s_o = sh.gen;                       // [8 warps][8 heads][HD]
  float* s_m = s_o + 8 * 8 * HD;             // [8][8]
  float* s_l = s_m + 64;                     // [8][8]
  float* sq = s_l + 64;                      // [8 heads][HD] rotated queries
  const __half* pool = reinterpret_cast<const __half*>(Ly.kv_layer);
  __half* pool_w = reinterpret_cast<__half*>(Ly.kv_layer);
  const size_t block_elems = (size_t)KV * kPageTokens * HD;
  const size_t page_elems = (EXT ? 4 : 2) * block_elems;
  const float scale = rsqrtf((float)HD);
  const int U = sh.pref[P.B] * KV;
  // pages per CTA: an even share, at least one page per warp, and no pair in more than kMaxParts pieces
  const int chunk = max(max((U + (int)gridDim.x - 1) / (int)gridDim.x, 8), (sh.pref[P.B + 1] + kMaxParts - 3) / (kMaxParts - 2));
  const int u_end = min(U, ((int)blockIdx.x + 1) * chunk);
  int slot = 0;
  for (int u = (int)blockIdx.x * chunk; u < u_end;) {
    while (sh.pref[slot + 1] * KV <= u) ++slot;
    const int n_pages = sh.pref[slot + 1] - sh.pref[slot];
    const int rel = u - sh.pref[slot] * KV;
    const int kvh = rel / n_pages, p_begin = rel - kvh * n_pages;
    const int p_end = min(n_pages, p_begin + (u_end - u));
    const int pair_u0 = sh.pref[slot] * KV + kvh * n_pages;
    const int first_cta = pair_u0 / chunk;
    const int S = (pair_u0 + n_pages - 1) / chunk - first_cta + 1;      // pieces of this pair
    const int split = (int)blockIdx.x - first_cta;
    const int pair = slot * KV + kvh;
    u += p_end - p_begin;
    const int row = pv.tok_row[slot];
    const int pos = pv.tok_pos[slot], ctx = pos + 1;
    const int h0 = kvh * G;
    const int32_t* pt = P.page_table + (size_t)row * P.max_pages;
    const float2* cs = P.rope + (size_t)pos * (HD / 2);
    // page indices of this warp's visits are requested first, so that they arrive under the rebuild below
    int pg[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int pp = p_begin + warp + 8 * i;
      pg[i] = pp < p_end ? __ldg(pt + pp) : 0;
    }
    // rotated queries of the group
    for (int idx = tid; idx < G * (HD / 2); idx += kGenThreads) {
      const int gg = idx >> 6, i = idx & 63;
      float a, b;
      qkv_sum2(P, slot, (h0 + gg) * HD + i, (h0 + gg) * HD + i + HD / 2, a, b);
      const float2 c = cs[i];
      sq[gg * HD + i] = a * c.x - b * c.y;
      sq[gg * HD + i + HD / 2] = b * c.x + a * c.y;
    }
    if (p_end == n_pages) {
      // the new token's key (rotated) and value go into their page before the page is read; the three upper
      // warps do it, which have the fewest queries to rebuild
      const int page = pt[pos / kPageTokens], tslot = pos % kPageTokens;
      __half* kbase = pool_w + (size_t)page * page_elems;
      __half* vbase = kbase + block_elems;
      const int r = kGenThreads - 1 - tid;        // 0..255 from the top thread down
      if (r < HD / 2) {
        const int i = r;
        float a, b;
        qkv_sum2(P, slot, (H + kvh) * HD + i, (H + kvh) * HD + i + HD / 2, a, b);
        const float2 c = cs[i];
        const float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
        __half* k = kbase + ((size_t)kvh * kPageTokens + tslot) * HD;
        const __half ka = __float2half_rn(ra), kb2 = __float2half_rn(rb);
        k[i] = ka;
        k[i + HD / 2] = kb2;
        if (EXT) {
          k[2 * block_elems + i] = __float2half_rn(ra - __half2float(ka));
          k[2 * block_elems + i + HD / 2] = __float2half_rn(rb - __half2float(kb2));
        }
      } else if (r < HD) {
        const int i = r - HD / 2;                 // value dims i and i + 64
        float v0, v1;
        qkv_sum2(P, slot, (H + KV + kvh) * HD + i, (H + KV + kvh) * HD + i + HD / 2, v0, v1);
        const __half h0v = __float2half_rn(v0), h1v = __float2half_rn(v1);
        vbase[((size_t)kvh * HD + i) * kPageTokens + tslot] = h0v;
        vbase[((size_t)kvh * HD + i + HD / 2) * kPageTokens + tslot] = h1v;
        if (EXT) {
          vbase[2 * block_elems + ((size_t)kvh * HD + i) * kPageTokens + tslot] = __float2half_rn(v0 - __half2float(h0v));
          vbase[2 * block_elems + ((size_t)kvh * HD + i + HD / 2) * kPageTokens + tslot] = __float2half_rn(v1 - __half2float(h1v));
        }
      }
    }
    bar_sync(3, kGenThreads);
    // Q fragments (rows 8..15 of the tile are padding): dims 32j + 8t + e of head h0 + g
    uint32_t qa[KB][2][2], ql[EXT ? KB : 1][2][2];
#pragma unroll
    for (int j = 0; j < KB; ++j) {
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = g < G ? sq[g * HD + 32 * j + 8 * t + e] : 0.f;
      if (EXT) {
        pack_h2_split(v[0], v[1], qa[j][0][0], ql[j][0][0]); pack_h2_split(v[2], v[3], qa[j][0][1], ql[j][0][1]);
        pack_h2_split(v[4], v[5], qa[j][1][0], ql[j][1][0]); pack_h2_split(v[6], v[7], qa[j][1][1], ql[j][1][1]);
      } else {
        qa[j][0][0] = pack_h2(v[0], v[1]); qa[j][0][1] = pack_h2(v[2], v[3]);
        qa[j][1][0] = pack_h2(v[4], v[5]); qa[j][1][1] = pack_h2(v[6], v[7]);
      }
    }
    float o[NT][2];
#pragma unroll
    for (int i = 0; i < NT; ++i) { o[i][0] = o[i][1] = 0.f; }
    float dump0 = 0.f, dump1 = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    const int tok0 = 4 * (g >> 1) + (g & 1), tok1 = tok0 + 2;
    int visit = 0;
    int page_next = 0;
    for (int p = p_begin + warp; p < p_end; p += 8, ++visit) {
      const int page = visit == 0 ? pg[0] : (visit == 1 ? pg[1] : (visit == 2 ? pg[2] : (visit == 3 ? pg[3] : page_next)));
      const __half* kb = pool + (size_t)page * page_elems + (size_t)kvh * kPageTokens * HD;
      const __half* vb = pool + (size_t)page * page_elems + block_elems + (size_t)kvh * HD * kPageTokens;
      if (visit >= 3 && p + 8 < p_end) page_next = pt[p + 8];
      uint4 k0[KB], k1[KB];
      uint2 vv[NT], vl[EXT ? NT : 1];
#pragma unroll
      for (int j = 0; j < KB; ++j) {
        k0[j] = ldcg_u4(kb + tok0 * HD + 32 * j + 8 * t);
        k1[j] = ldcg_u4(kb + tok1 * HD + 32 * j + 8 * t);
      }
#pragma unroll
      for (int i = 0; i < NT; ++i) vv[i] = ldcg_u2(vb + (size_t)(8 * i + g) * kPageTokens + 4 * t);
      if (EXT) {
#pragma unroll
        for (int i = 0; i < NT; ++i) vl[i] = ldcg_u2(vb + 2 * block_elems + (size_t)(8 * i + g) * kPageTokens + 4 * t);
      }
      float s0[2] = {0.f, 0.f}, s1[2] = {0.f, 0.f};
#pragma unroll
      for (int j = 0; j < KB; ++j) {
        mma_f16(s0[0], s0[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, k0[j].x, k0[j].y);
        mma_f16(s0[0], s0[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, k0[j].z, k0[j].w);
        mma_f16(s1[0], s1[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, k1[j].x, k1[j].y);
        mma_f16(s1[0], s1[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, k1[j].z, k1[j].w);
        if (EXT) {
          const uint4 e0 = ldcg_u4(kb + 2 * block_elems + tok0 * HD + 32 * j + 8 * t);
          const uint4 e1 = ldcg_u4(kb + 2 * block_elems + tok1 * HD + 32 * j + 8 * t);
          mma_f16(s0[0], s0[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, e0.x, e0.y);
          mma_f16(s0[0], s0[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, e0.z, e0.w);
          mma_f16(s1[0], s1[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, e1.x, e1.y);
          mma_f16(s1[0], s1[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, e1.z, e1.w);
          mma_f16(s0[0], s0[1], dump0, dump1, ql[j][0][0], 0u, ql[j][0][1], 0u, k0[j].x, k0[j].y);
          mma_f16(s0[0], s0[1], dump0, dump1, ql[j][1][0], 0u, ql[j][1][1], 0u, k0[j].z, k0[j].w);
          mma_f16(s1[0], s1[1], dump0, dump1, ql[j][0][0], 0u, ql[j][0][1], 0u, k1[j].x, k1[j].y);
          mma_f16(s1[0], s1[1], dump0, dump1, ql[j][1][0], 0u, ql[j][1][1], 0u, k1[j].z, k1[j].w);
        }
      }
      const int n_valid = min(kPageTokens, ctx - p * kPageTokens);
      float sc[4] = {s0[0] * scale, s0[1] * scale, s1[0] * scale, s1[1] * scale};
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (4 * t + e >= n_valid) sc[e] = -INFINITY;
      float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
      mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
      const float m_new = fmaxf(m_run, mx);
      const float corr = __expf(m_run - m_new);
      float pr[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) pr[e] = __expf(sc[e] - m_new);
      l_run = l_run * corr + (pr[0] + pr[1] + pr[2] + pr[3]);
      m_run = m_new;
      uint32_t pa0, pa2, pl0 = 0u, pl2 = 0u;
      if (EXT) { pack_h2_split(pr[0], pr[1], pa0, pl0); pack_h2_split(pr[2], pr[3], pa2, pl2); }
      else { pa0 = pack_h2(pr[0], pr[1]); pa2 = pack_h2(pr[2], pr[3]); }
      uint32_t mlo = 0xFFFFFFFFu, mhi = 0xFFFFFFFFu;
      if (n_valid < kPageTokens) {
        mlo = (4 * t < n_valid ? 0x0000FFFFu : 0u) | (4 * t + 1 < n_valid ? 0xFFFF0000u : 0u);
        mhi = (4 * t + 2 < n_valid ? 0x0000FFFFu : 0u) | (4 * t + 3 < n_valid ? 0xFFFF0000u : 0u);
      }
#pragma unroll
      for (int i = 0; i < NT; ++i) {
        o[i][0] *= corr; o[i][1] *= corr;
        mma_f16(o[i][0], o[i][1], dump0, dump1, pa0, 0u, pa2, 0u, vv[i].x & mlo, vv[i].y & mhi);
        if (EXT) {
          mma_f16(o[i][0], o[i][1], dump0, dump1, pl0, 0u, pl2, 0u, vv[i].x & mlo, vv[i].y & mhi);
          mma_f16(o[i][0], o[i][1], dump0, dump1, pa0, 0u, pa2, 0u, vl[i].x & mlo, vl[i].y & mhi);
        }
      }
    }
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
    if (t == 0) { s_m[warp * 8 + g] = m_run; s_l[warp * 8 + g] = l_run; }
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      s_o[(warp * 8 + g) * HD + 8 * i + 2 * t] = o[i][0];
      s_o[(warp * 8 + g) * HD + 8 * i + 2 * t + 1] = o[i][1];
    }
    bar_sync(3, kGenThreads);
    for (int idx = tid; idx < G * HD; idx += kGenThreads) {
      const int gg = idx / HD, dd = idx % HD;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < 8; ++w) M = fmaxf(M, s_m[w * 8 + gg]);
      float L = 0.f, O = 0.f;
      if (M > -INFINITY) {
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const float e = __expf(s_m[w * 8 + gg] - M);
          L += s_l[w * 8 + gg] * e;
          O += s_o[(w * 8 + gg) * HD + dd] * e;
        }
      }
      const int h = h0 + gg;
      if (S == 1) {
        store_operand<__nv_bfloat16>(P.attn_hi, P.attn_lo, ((size_t)slot * H + h) * HD + dd, O / L);
      } else {
        const size_t base = ((size_t)slot * H + h) * kMaxParts + split;
        P.part_o[base * HD + dd] = O;
        if (dd == 0) { P.part_ml[base * 2] = M; P.part_ml[base * 2 + 1] = L; }
      }
    }
    if (S > 1) {
      __threadfence();
      bar_sync(3, kGenThreads);
      if (tid == 0) {
        const int old = atomicAdd(P.attn_cnt + pair, 1);
        *sh.flag = old == S - 1;
        if (old == S - 1) P.attn_cnt[pair] = 0;
      }
      bar_sync(3, kGenThreads);
      if (*sh.flag) {
        __threadfence();
        for (int idx = tid; idx < G * HD; idx += kGenThreads) {
          const int gg = idx / HD, dd = idx % HD, h = h0 + gg;
          const size_t base = ((size_t)slot * H + h) * kMaxParts;
          float M = -INFINITY, L = 0.f, O = 0.f;
          for (int s0 = 0; s0 < S; s0 += 4) {
            float2 ml[4];
            float ov[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const bool in = s0 + u < S;
              ml[u] = in ? __ldcg(reinterpret_cast<const float2*>(P.part_ml + (base + s0 + u) * 2)) : make_float2(-INFINITY, 0.f);
              ov[u] = in ? __ldcg(P.part_o + (base + s0 + u) * HD + dd) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              if (ml[u].x > -INFINITY) {
                const float Mn = fmaxf(M, ml[u].x);
                const float e_old = __expf(M - Mn), e_new = __expf(ml[u].x - Mn);
                L = L * e_old + ml[u].y * e_new;
                O = O * e_old + ov[u] * e_new;
                M = Mn;
              }
            }
          }
          store_operand<__nv_bfloat16>(P.attn_hi, P.attn_lo, ((size_t)slot * H + h) * HD + dd, O / L);
        }
      }
    }
    bar_sync(3, kGenThreads);   // the scratch is free for the next segment
  }
}

// ---- GEMM phase ----------------------------------------------------------------------------------------
// Ring positions as (stage, parity) pairs that are stepped, never divided: the loops below run in one thread
// each, where every dependent instruction costs its full latency.
struct RingPos {
  uint32_t stage = 0, parity = 0;
  __device__ __forceinline__ void step(uint32_t n) {
    if (++stage == n) { stage = 0; parity ^= 1u; }
  }
};
struct PipeState {
  RingPos xi;        // next X stage to fill         (X producer)
  RingPos wc, xc;    // next W / X stage to consume  (MMA issuer)
  uint32_t ac = 0;   // accumulators produced        (MMA issuer)
  uint32_t ae = 0;   // accumulators read            (epilogue warps)
};

// which: 0 qkv, 1 wo, 2 gate/up (+ SwiGLU), 3 down.
__device__ __forceinline__ void gemm_phase(const MegaParams& P, int which, const Shared& sh, uint32_t tmem_base,
                                           PipeState& ps) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const GemmPlan& g = P.plan[which];
  const int n_items = g.n_tiles * g.splits;
  const int rows = P.rows, mt = P.mt;
  const uint32_t xstage = (uint32_t)mt * 128u, n_sw = (uint32_t)P.sw, n_sx = (uint32_t)P.sx;
  int* const err = P.err;
  if (warp == kWarpX) {
    if (lane == 0 && !*sh.abort_flag) {
      const int src = which == 1 ? 1 : (which == 3 ? 2 : 0);
      const CUtensorMap* mhi = &P.xmap[2 * src];
      const CUtensorMap* mlo = &P.xmap[2 * src + 1];
      for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
        const Item im = item_of(g, it);
        bool ok = true;
        for (int kb = im.kb0; kb < im.kb1 && ok; ++kb) {
          const uint32_t s = ps.xi.stage;
          ok = wait_bar(&sh.empty_x[s], ps.xi.parity ^ 1u, sh, err);
          if (!ok) break;
          uint8_t* dst = sh.xring + (size_t)s * xstage;
          mbar_expect_tx(&sh.full_x[s], xstage);
          tma_load_2d(dst, mhi, &sh.full_x[s], kb * 64, 0);
          tma_load_2d(dst + (size_t)rows * 128, mlo, &sh.full_x[s], kb * 64, 0);
          ps.xi.step(n_sx);
        }
        if (!ok) break;
      }
    }
    __syncwarp();
    return;
  }
  if (warp == kWarpMma) {
    if (lane == 0 && !*sh.abort_flag) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mt >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      // shared-memory descriptors (K-major, 128-byte swizzle): the high word is constant, the low word is the
      // tile address in 16-byte units (plus 2 per 16-element k slice) with the unused leading offset set to 1
      const uint32_t desc_hi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
      const uint32_t a_lo0 = ((smem_u32(sh.wring) >> 4) & 0x3FFFu) | (1u << 16);
      const uint32_t b_lo0 = ((smem_u32(sh.xring) >> 4) & 0x3FFFu) | (1u << 16);
      const uint32_t b_step = xstage >> 4;
      for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
        const Item im = item_of(g, it);
        const uint32_t b = ps.ac & 1u;
        bool ok = wait_bar(&sh.acc_empty[b], ((ps.ac >> 1) & 1u) ^ 1u, sh, err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + b * (uint32_t)mt;
        uint32_t acc = 0u;
        for (int kb = im.kb0; kb < im.kb1; ++kb) {
          const uint32_t ws = ps.wc.stage, xs = ps.xc.stage;
          ok = wait_bar(&sh.full_w[ws], ps.wc.parity, sh, err) && wait_bar(&sh.full_x[xs], ps.xc.parity, sh, err);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + ws * (kWStageBytes >> 4), b_lo = b_lo0 + xs * b_step;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint64_t da = ((uint64_t)desc_hi << 32) | (uint64_t)(a_lo + 2 * k);
            const uint64_t db = ((uint64_t)desc_hi << 32) | (uint64_t)(b_lo + 2 * k);
            umma_bf16(d_tmem, da, db, idesc, acc);
            acc = 1u;
          }
          umma_commit(&sh.empty_w[ws]);
          umma_commit(&sh.empty_x[xs]);
          ps.wc.step(n_sw);
          ps.xc.step(n_sx);
        }
        if (!ok) break;
        umma_commit(&sh.acc_full[b]);
        ++ps.ac;
      }
    }
    __syncwarp();
    return;
  }
  if (warp >= 4) return;
  // ---- epilogue warps ----
  const bool scaled = which == 0 || which == 2;
  if (scaled) {
    const int r = threadIdx.x;
    if (r < P.B) {
      const int nch = P.d >> 7;
      float sum = 0.f;
      for (int c = 0; c < nch; ++c) sum += __ldcg(P.ssq + (size_t)r * nch + c);
      sh.row_scale[r] = rsqrtf(sum / (float)P.d + P.eps);
    }
    bar_sync(2, 128);
  }
  const int B = P.B;
  for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
    const Item im = item_of(g, it);
    const uint32_t b = ps.ae & 1u;
    const bool ok = wait_bar(&sh.acc_full[b], (ps.ae >> 1) & 1u, sh, err);
    ++ps.ae;
    tc_fence_after();
    const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + b * (uint32_t)mt;
    if (which != 2) {
      if (ok) {
        float* dst = P.partials + (size_t)im.split * B * g.N;
        const int n = im.tile * 128 + warp * 32 + lane;
        for (int c = 0; c < rows && c < B; c += 16) {
          float v[16], w[16];
          tmem_ld16(taddr + c, v);
          tmem_ld16(taddr + rows + c, w);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            if (c + j < B) {
              float r = v[j] + w[j];
              if (scaled) r *= sh.row_scale[c + j];
              dst[(size_t)(c + j) * g.N + n] = r;
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.acc_empty[b]);
      }
    } else {
      // gate rows in TMEM lanes 0-63 (warps 0, 1), the matching up rows in lanes 64-127 (warps 2, 3)
      float* xch = sh.xch;                         // [64][65]
      const int l = (warp & 1) * 32 + lane;        // feature within the 64-row half
      if (ok && warp >= 2) {
        for (int c = 0; c < rows && c < B; c += 16) {
          float v[16], w[16];
          tmem_ld16(taddr + c, v);
          tmem_ld16(taddr + rows + c, w);
#pragma unroll
          for (int j = 0; j < 16; ++j) xch[l * 65 + c + j] = v[j] + w[j];
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.acc_empty[b]);
      }
      bar_sync(2, 128);
      if (ok && warp < 2) {
        const int f = im.tile * 64 + l;
        for (int c = 0; c < rows && c < B; c += 16) {
          float v[16], w[16];
          tmem_ld16(taddr + c, v);
          tmem_ld16(taddr + rows + c, w);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            if (c + j < B) {
              const float sc = sh.row_scale[c + j];
              const float a = (v[j] + w[j]) * sc, u = xch[l * 65 + c + j] * sc;
              store_operand<__nv_bfloat16>(P.act_hi, P.act_lo, (size_t)(c + j) * P.F + f, a / (1.f + expf(-a)) * u);
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.acc_empty[b]);
      }
      bar_sync(2, 128);
    }
  }
}

template <bool EXT>
__global__ void __launch_bounds__(kThreads, 1)
decode_mega_kernel(const MegaParams* __restrict__ Pp, const MegaLayer* __restrict__ layers, PassView pv,
                   const __nv_bfloat16* __restrict__ final_gain) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const MegaParams& P = *Pp;
  if (*pv.n_active == 0 || __ldcg(P.err) != 0) return;     // uniform over the grid

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Shared sh;
  sh.wring = smem;
  sh.xring = sh.wring + (size_t)P.sw * kWStageBytes;
  sh.gen = (float*)sh.xring;
  sh.xch = (float*)(sh.xring + (size_t)P.sx * P.mt * 128);
  sh.row_scale = (float*)((uint8_t*)sh.xch + kXchBytes);
  sh.full_w = (uint64_t*)(sh.row_scale + 64);
  sh.empty_w = sh.full_w + P.sw;
  sh.full_x = sh.empty_w + P.sw;
  sh.empty_x = sh.full_x + P.sx;
  sh.acc_full = sh.empty_x + P.sx;
  sh.acc_empty = sh.acc_full + 2;
  sh.tmem_slot = (uint32_t*)(sh.acc_empty + 2);
  sh.abort_flag = (volatile int*)(sh.tmem_slot + 1);
  sh.go = sh.abort_flag + 1;
  sh.flag = sh.abort_flag + 2;
  sh.pref = (int*)(sh.abort_flag + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < P.sw; ++s) { mbar_init(&sh.full_w[s], 1); mbar_init(&sh.empty_w[s], 1); }
    for (int s = 0; s < P.sx; ++s) { mbar_init(&sh.full_x[s], 1); mbar_init(&sh.empty_x[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&sh.acc_full[s], 1); mbar_init(&sh.acc_empty[s], 4); }
    *sh.abort_flag = 0; *sh.go = 1; *sh.flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWarpMma) tmem_alloc(sh.tmem_slot, (uint32_t)P.tmem_cols);
  if (warp == 1) {
    // page counts of the rows of this iteration (idle slots: none), as prefix sums; B <= 64
    int n0 = 0, n1 = 0;
    if (lane < P.B && pv.tok_row[lane] >= 0) n0 = (pv.tok_pos[lane] + 1 + kPageTokens - 1) / kPageTokens;
    if (lane + 32 < P.B && pv.tok_row[lane + 32] >= 0) n1 = (pv.tok_pos[lane + 32] + 1 + kPageTokens - 1) / kPageTokens;
    int i0 = n0, i1 = n1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xFFFFFFFFu, i0, o), b = __shfl_up_sync(0xFFFFFFFFu, i1, o);
      if (lane >= o) { i0 += a; i1 += b; }
    }
    const int tot0 = __shfl_sync(0xFFFFFFFFu, i0, 31);
    int mx = max(n0, n1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    if (lane == 0) { sh.pref[0] = 0; sh.pref[P.B + 1] = mx; }
    if (lane < P.B) sh.pref[lane + 1] = i0;
    if (lane + 32 < P.B) sh.pref[lane + 33] = tot0 + i1;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *sh.tmem_slot;
  const int L = P.L;

  if (warp == kWarpW) {
    // ---------------- W producer: streams every weight tile of this CTA's work items, in order ----------------
    if (lane == 0) {
      uint32_t wi = 0;
      RingPos wpos;
      bool ok = true;
      const uint32_t n_sw = (uint32_t)P.sw;
      int* const err = P.err;
      const int F = P.F;
      for (int l = 0; l < L && ok; ++l) {
        for (int which = 0; which < 4 && ok; ++which) {
          const GemmPlan& g = P.plan[which];
          const CUtensorMap* map = &layers[l].w[which];
          const int n_items = g.n_tiles * g.splits;
          for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const Item im = item_of(g, it);
            for (int kb = im.kb0; kb < im.kb1; ++kb) {
              const uint32_t s = wpos.stage;
              ok = wait_bar(&sh.empty_w[s], wpos.parity ^ 1u, sh, err);
              if (!ok) break;
              uint8_t* dst = sh.wring + (size_t)s * kWStageBytes;
              mbar_expect_tx(&sh.full_w[s], kWStageBytes);
              if (which == 2) {
                tma_load_2d(dst, map, &sh.full_w[s], kb * 64, im.tile * 64);
                tma_load_2d(dst + kWStageBytes / 2, map, &sh.full_w[s], kb * 64, F + im.tile * 64);
              } else {
                tma_load_2d(dst, map, &sh.full_w[s], kb * 64, im.tile * 128);
              }
              wpos.step(n_sw);
              ++wi;
            }
          }
        }
      }
      if (!ok) {
        // copies already requested must land before the CTA goes away
        for (uint32_t i = 0; i < min(wi, n_sw); ++i) {
          // stage filled i + 1 steps ago
          uint32_t st = wpos.stage, par = wpos.parity;
          for (uint32_t k = 0; k <= i; ++k) {
            if (st == 0) { st = n_sw - 1; par ^= 1u; } else --st;
          }
          for (uint32_t k = 0; k < (1u << 16); ++k)
            if (mbar_try_wait(&sh.full_w[st], par)) break;
        }
      }
    }
  } else {
    PipeState ps;
    int n_stamps = 1;
    unsigned epoch = 0;
    if (P.prof != nullptr && blockIdx.x == 0 && threadIdx.x == 0) P.prof[0] = global_timer();
    rn_phase(P, pv, 0, layers[0].norm1, true);
    grid_sync(P, sh, epoch, n_stamps);
    for (int l = 0; l < L; ++l) {
      const MegaLayer& Ly = layers[l];
      if (*sh.go) gemm_phase(P, 0, sh, tmem_base, ps);
      grid_sync(P, sh, epoch, n_stamps);
      if (*sh.go) attn_phase<EXT>(P, Ly, pv, sh);
      grid_sync(P, sh, epoch, n_stamps);
      if (*sh.go) gemm_phase(P, 1, sh, tmem_base, ps);
      grid_sync(P, sh, epoch, n_stamps);
      if (*sh.go) rn_phase(P, pv, P.plan[1].splits, Ly.norm2, false);
      grid_sync(P, sh, epoch, n_stamps);
      if (*sh.go) gemm_phase(P, 2, sh, tmem_base, ps);
      grid_sync(P, sh, epoch, n_stamps);
      if (*sh.go) gemm_phase(P, 3, sh, tmem_base, ps);
      grid_sync(P, sh, epoch, n_stamps);
      if (*sh.go) rn_phase(P, pv, P.plan[3].splits, l + 1 < L ? layers[l + 1].norm1 : final_gain, false);
      if (l + 1 < L) grid_sync(P, sh, epoch, n_stamps);
    }
    if (P.prof != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
      if (n_stamps < kMaxStamps) P.prof[n_stamps++] = global_timer();
      P.prof[kMaxStamps + 1] = (unsigned long long)n_stamps;
    }
    if (threadIdx.x == 0 && !*sh.abort_flag) finish_grid_sync(P);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
  }
}

GemmPlan make_plan(int N, int K, int tile_rows, int n_ctas) {
  GemmPlan p;
  p.N = N; p.K = K;
  p.n_tiles = (N + tile_rows - 1) / tile_rows;
  p.total_kb = (K + 63) / 64;
  int splits = 1;
  if (p.n_tiles < n_ctas) {
    splits = std::max(1, n_ctas / p.n_tiles);
    splits = std::min(splits, std::max(1, p.total_kb / 2));
  }
  p.kbps = (p.total_kb + splits - 1) / splits;
  p.splits = (p.total_kb + p.kbps - 1) / p.kbps;
  return p;
}

struct Geometry { int rows, sw, sx; size_t smem; };
Geometry geometry(int B) {
  Geometry g;
  g.rows = B <= 16 ? 16 : (B <= 32 ? 32 : 64);
  // The X ring is as deep as the W ring: a weight tile can only be consumed together with its activation
  // tile, and both arrive with the same latency.  What is left over goes to the W ring.
  const size_t fixed = 1024 + kXchBytes + 64 * 4 + 1024;
  const size_t avail = 227 * 1024 - fixed;
  const size_t xstage = (size_t)2 * g.rows * 128;
  size_t n = avail / (kWStageBytes + xstage);
  while (n * xstage < (size_t)kGenScratchBytes) ++n;        // the attention scratch lives in the X ring
  g.sx = (int)n;
  g.sw = (int)std::min<size_t>(16, (avail - n * xstage) / kWStageBytes);
  g.smem = fixed + n * xstage + (size_t)g.sw * kWStageBytes;
  return g;
}

int g_sm_count = 0;
size_t g_smem_set[2] = {0, 0};

}  // namespace

int mega_sm_count();

size_t mega_block_bytes(int n_layers) { return sizeof(MegaParams) + (size_t)n_layers * sizeof(MegaLayer); }

size_t mega_partials_floats(const MegaShape& m, int B) {
  const int n_ctas = std::max(1, mega_sm_count());
  size_t need = 0;
  const GemmPlan pl[3] = {make_plan((m.H + 2 * m.KV) * 128, m.d, 128, n_ctas), make_plan(m.d, m.H * 128, 128, n_ctas),
                          make_plan(m.d, m.F, 128, n_ctas)};
  for (const GemmPlan& p : pl) need = std::max(need, (size_t)p.splits * B * p.N);
  return need;
}

bool mega_supported(const MegaShape& m, int B) {
  return m.bf16 && m.hd == 128 && m.d % 128 == 0 && m.F % 64 == 0 && m.H % m.KV == 0 && m.H / m.KV <= 8 && B >= 1 && B <= 64 &&
         m.n_layers >= 1;
}

int mega_sm_count() {
  if (g_sm_count == 0) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) g_sm_count = n;
  }
  return g_sm_count;
}

cudaError_t mega_build(void* dev_block, const MegaBuild& a, cudaStream_t s) {
  const MegaShape& m = a.shape;
  if (!mega_supported(m, a.B)) return cudaErrorNotSupported;
  const int n_ctas = mega_sm_count();
  if (n_ctas <= 0) return cudaErrorInvalidDevice;
  std::vector<uint8_t> host(mega_block_bytes(m.n_layers) + 128);
  uint8_t* hb = (uint8_t*)(((uintptr_t)host.data() + 127) & ~(uintptr_t)127);
  MegaParams* P = new (hb) MegaParams();
  MegaLayer* Ls = reinterpret_cast<MegaLayer*>(hb + sizeof(MegaParams));
  const int rows = geometry(a.B).rows;
  P->L = m.n_layers; P->d = m.d; P->H = m.H; P->KV = m.KV; P->F = m.F; P->B = a.B; P->rows = rows; P->mt = 2 * rows;
  P->max_pages = a.max_pages; P->eps = m.eps;
  P->tmem_cols = std::max(32, 4 * rows);               // two accumulators of 2 * rows columns (a power of two)
  const int qkv_n = (m.H + 2 * m.KV) * 128, hq = m.H * 128;
  P->plan[0] = make_plan(qkv_n, m.d, 128, n_ctas);
  P->plan[1] = make_plan(m.d, hq, 128, n_ctas);
  P->plan[2] = make_plan(2 * m.F, m.d, 128, n_ctas);
  P->plan[2].splits = 1; P->plan[2].kbps = P->plan[2].total_kb;   // SwiGLU in the epilogue needs whole sums
  P->plan[3] = make_plan(m.d, m.F, 128, n_ctas);
  P->attn_splits = 0;
  const Geometry geo = geometry(a.B);
  P->sx = geo.sx; P->sw = geo.sw;
  if (P->sw < 3) return cudaErrorNotSupported;
  P->embed = (const __nv_bfloat16*)a.embed;
  P->x = a.x;
  P->h_hi = (__nv_bfloat16*)a.h; P->h_lo = (__nv_bfloat16*)a.h_lo;
  P->attn_hi = (__nv_bfloat16*)a.attn; P->attn_lo = (__nv_bfloat16*)a.attn_lo;
  P->act_hi = (__nv_bfloat16*)a.act; P->act_lo = (__nv_bfloat16*)a.act_lo;
  P->partials = a.partials; P->ssq = a.ssq; P->part_o = a.part_o; P->part_ml = a.part_ml;
  P->attn_cnt = a.sync_words + 16; P->grid_bar = (unsigned*)a.sync_words; P->err = a.err;
  P->rope = a.rope; P->page_table = a.page_table; P->prof = a.prof;
  const void* xs[6] = {a.h, a.h_lo, a.attn, a.attn_lo, a.act, a.act_lo};
  const int xk[6] = {m.d, m.d, hq, hq, m.F, m.F};
  for (int i = 0; i < 6; ++i)
    if (!tc_tensor_map(xs[i], a.B, xk[i], rows, &P->xmap[i])) return cudaErrorNotSupported;
  for (int l = 0; l < m.n_layers; ++l) {
    MegaLayer& Ly = Ls[l];
    if (!tc_tensor_map(a.wqkv[l], qkv_n, m.d, 128, &Ly.w[0]) || !tc_tensor_map(a.wo[l], m.d, hq, 128, &Ly.w[1]) ||
        !tc_tensor_map(a.wgu[l], 2 * m.F, m.d, 64, &Ly.w[2]) || !tc_tensor_map(a.wdown[l], m.d, m.F, 128, &Ly.w[3]))
      return cudaErrorNotSupported;
    Ly.norm1 = (const __nv_bfloat16*)a.norm1[l];
    Ly.norm2 = (const __nv_bfloat16*)a.norm2[l];
    Ly.kv_layer = a.kv_pool + (size_t)l * a.layer_stride;
  }
  cudaError_t e = cudaMemcpyAsync(dev_block, hb, mega_block_bytes(m.n_layers), cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return e;
  return cudaStreamSynchronize(s);   // the staging vector goes away
}

cudaError_t launch_decode_mega(const void* dev_block, int B, int kv_extended, PassView p, const void* final_gain,
                               cudaStream_t s) {
  const int n_ctas = mega_sm_count();
  if (n_ctas <= 0) return cudaErrorInvalidDevice;
  const size_t smem = geometry(B).smem;
  const int ext = kv_extended ? 1 : 0;
  if (g_smem_set[ext] < smem) {
    cudaError_t e = ext ? cudaFuncSetAttribute(decode_mega_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                        : cudaFuncSetAttribute(decode_mega_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    g_smem_set[ext] = smem;
  }
  const MegaParams* P = reinterpret_cast<const MegaParams*>(dev_block);
  const MegaLayer* Ls = reinterpret_cast<const MegaLayer*>((const uint8_t*)dev_block + sizeof(MegaParams));
  if (ext) RSD_LAUNCH((decode_mega_kernel<true>), n_ctas, kThreads, smem, s, P, Ls, p, (const __nv_bfloat16*)final_gain);
  else RSD_LAUNCH((decode_mega_kernel<false>), n_ctas, kThreads, smem, s, P, Ls, p, (const __nv_bfloat16*)final_gain);
  return launched(1);
}

}  // namespace rsd
