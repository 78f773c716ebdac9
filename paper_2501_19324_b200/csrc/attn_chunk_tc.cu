// Causal attention of a ragged chunk of new tokens over paged fp16 KV on the 5th-generation tensor cores
// (tcgen05.mma with the left operands and the accumulators in tensor memory, pages fetched by TMA), for the long
// passes: prefill, PRM step scoring, draft sync, target catch-up.  head_dim 128, up to 8 query heads per KV head.
//
// A CTA takes QT = 128 / G consecutive entries of the pass list and one KV head; the 128 rows of its MMA tile are
// the (entry, query head) pairs, row = entry * G + head, so every key and value is read once for the whole group.
// Entries of a tile that belong to different sequences are handled one run ("segment") at a time, the rows outside
// the segment masked; a long pass has one segment per tile almost everywhere.  Per segment the keys go by in tiles
// of 64 (four pages), twice:
//   pass 1   S = Q K^T into tensor memory; the softmax threads keep the running maximum m of the visible scores
//            of their row (causal: key position <= query position);
//   pass 2   S again, p = 2^(s - m) with the FINAL maximum (scores are in units of log 2), so the output tile
//            needs no rescaling and can stay in tensor memory: the threads add up their rows of p, write them as
//            fp16 back into tensor memory, and O += P V runs on the tensor cores.
// The second Q K^T costs half again as many flops and buys an O accumulator that is never read back or rescaled
// before the end; on tensor cores that trade is cheap.  At the end the rows of O are read, divided by the sums and
// written out (as a bf16 hi + lo pair where the next GEMM wants one).
//
// Shared-memory bandwidth is what bounds a tile (an MMA reads its shared-memory operands at 128 bytes a clock, and
// a 128 x 16 left operand re-read for every K = 16 step costs as much as the step computes), so both left operands
// live in tensor memory: Q (128 rows x 128 dims of fp16, 64 columns) is written there once, P (128 x 64 keys, 32
// columns, two buffers) by the softmax threads with tcgen05.st.  Shared memory then carries the keys and values
// only: once in by TMA, once out to the tensor cores.
//
// Roles: warps 0-7 softmax, two warpgroups that split the 64 score columns (and the 128 output columns) of every
// row, thread = tensor-memory lane = tile row; warp 8 issues the score MMAs and warp 10 the output MMAs (two
// threads, so that waiting for a tile's weights never holds up the next tiles' scores); warp 9 fetches pages.  A
// page holds, per KV head, the keys [16 tokens][128 dims] and the values transposed [128 dims][16 tokens], 4096
// bytes each, so
//   keys    one TMA box per page (five-dimensional: 64 dims, 8 tokens, 2 halves of the 128 dims, 2 groups of 8
//           tokens; 128-byte swizzle) lands as [token group][dim half][8 keys][64 dims], so either half of a tile's
//           64 keys is a K-major operand with its groups of 8 rows 2048 bytes apart;
//   values  one TMA box (16 tokens x 128 dims, 32-byte swizzle) per page is by itself the K-major operand
//           [128 dims][16 keys] of one K = 16 step of P V: four pages, four MMAs.
// Pages beyond the sequence are not fetched (their scores are masked, their weights exactly zero; the value
// buffers start zeroed and afterwards only ever hold real values, so 0 * stale stays 0).  The tokens of the last
// page that lie beyond the cached positions may hold anything, so that one page is copied by the fetch warp itself
// with those tokens zeroed.  Every wait is bounded; on expiry the CTA raises an error flag, waits for its copies in
// flight, frees its tensor memory and leaves.
#include <cuda.h>

#include "common.cuh"
#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace rsd {

namespace {

using namespace tc;

constexpr int kHd = 128;
constexpr int kKeys = 64;                           // keys per tile: four pages
constexpr int kNS = 6;                              // ring stages (keys + values of one tile)
constexpr int kKBytes = kKeys * kHd * 2;            // K tile: per page [2 token groups][2 dim halves][8 keys][64 dims]
constexpr int kVBytes = kHd * kKeys * 2;            // V tile: four page buffers [128 dims][16 keys]
constexpr int kBlockBytes = 4096;                   // keys (or values) of one page and KV head
constexpr int kStageBytes = kKBytes + kVBytes;
constexpr int kMetaBytes = 4096;                    // barriers, flags, the tile's entries, the row maxima and sums
constexpr size_t kSmemBytes = 1024 + kNS * kStageBytes + kMetaBytes;
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
constexpr int kSoftmaxWarps = 8;
constexpr int kSoftmaxThreads = 32 * kSoftmaxWarps;
constexpr int kMmaWarp = 8, kFetchWarp = 9, kOutWarp = 10;
constexpr int kThreads = 352;
// instruction descriptors (kind::f16): fp32 accumulate, fp16 A and B, both K-major, M = 128; N = 64 (scores), 128 (output)
constexpr uint32_t kIdescS = (1u << 4) | ((uint32_t)(kKeys >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t kIdescO = (1u << 4) | ((uint32_t)(kHd >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
// tensor-memory columns: S four buffers of 64 (the score issuer runs up to four tiles ahead of the softmax), O 128,
// Q 64 (fp16 pairs), P two buffers of 32 (fp16 pairs)
constexpr int kSB = 4;
constexpr uint32_t kColS = 0, kColO = 256, kColQ = 384, kColP = 448, kTmemCols = 512;
constexpr uint32_t kProbeLimit = 1u << 18;          // polls of a bounded wait (a healthy wait ends within microseconds)

// Writes of this thread to shared memory become visible to the tensor cores.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// The box of a tensor map whose first block coordinate is `blk` (all inner coordinates 0).
__device__ __forceinline__ void tma_load_block_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int blk) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(0), "r"(blk) : "memory");
}
__device__ __forceinline__ void tma_load_block_5d(void* dst, const CUtensorMap* map, uint64_t* bar, int blk) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %3, %3, %3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(0), "r"(blk) : "memory");
}

// Shared-memory matrix descriptors of K-major operands (leading byte offset unused, version 1).  A later k-step or
// half of the same tile is the descriptor plus its byte offset / 16: shared-memory addresses fit the 14-bit field.
// 128-byte swizzle: rows of 128 bytes, groups of 8 rows `sbo` bytes apart.
__device__ __forceinline__ uint64_t desc_sw128(uint32_t saddr, uint32_t sbo) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// 32-byte swizzle: rows of 32 bytes (one K = 16 step), groups of 8 rows 256 bytes apart.
__device__ __forceinline__ uint64_t desc_sw32(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(256 >> 4) << 32) | (1ull << 46) | (6ull << 61);
}

// D (tensor memory) (+)= A (tensor memory: 128 lanes x 8 columns of fp16 pairs, one K = 16 step) * B (shared memory)
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// 16 (32) registers of this thread into 16 (32) consecutive columns of its tensor-memory lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  tmem_st16(taddr, r);
  tmem_st16(taddr + 16, r + 16);
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);         // .x (the low 16 bits) = lo: the element with the even index
  return *reinterpret_cast<const uint32_t*>(&h);
}

// 32 consecutive columns of this warp's tensor-memory lanes, one per register.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Bounded wait that leaves the issue slots to the warps with work: a short spin (most waits end within a few hundred
// cycles), then suspended polls.
__device__ __forceinline__ bool wait_sleep(uint64_t* bar, uint32_t parity, volatile uint32_t* stop) {
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t i = 0; i < (1u << 19); ++i) {
    if (mbar_try_wait_sleep(bar, parity, 1000)) return true;
    if (*stop) return false;
  }
  return false;
}

struct Meta {
  uint64_t kv_full[kNS], kv_empty[kNS], s_full[kSB], s_empty[kSB], p_full[2], p_empty[2], o_full, o_empty;
  uint64_t halves;                  // the two warpgroups have posted their halves of a row's maximum (or sum)
  uint32_t tmem_slot;
  uint32_t stop;
  int32_t row[128], pos[128];
  float pmax[2][128], psum[2][128];
};
static_assert(sizeof(Meta) <= kMetaBytes, "metadata block");

template <typename OT> __device__ __forceinline__ void store16(OT* hi, OT* lo, size_t o, const float* v);
template <> __device__ __forceinline__ void store16<float>(float* hi, float*, size_t o, const float* v) {
#pragma unroll
  for (int i = 0; i < 4; ++i) *reinterpret_cast<float4*>(hi + o + 4 * i) = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
}
template <> __device__ __forceinline__ void store16<__half>(__half* hi, __half*, size_t o, const float* v) {
  __align__(16) __half2 h[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) h[i] = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
  *reinterpret_cast<uint4*>(hi + o) = *reinterpret_cast<const uint4*>(h);
  *reinterpret_cast<uint4*>(hi + o + 8) = *reinterpret_cast<const uint4*>(h + 4);
}
template <> __device__ __forceinline__ void store16<__nv_bfloat16>(__nv_bfloat16* hi, __nv_bfloat16* lo, size_t o, const float* v) {
  __align__(16) __nv_bfloat16 h[16];
  __align__(16) __nv_bfloat16 l[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    h[i] = __float2bfloat16_rn(v[i]);
    l[i] = __float2bfloat16_rn(v[i] - __bfloat162float(h[i]));
  }
  *reinterpret_cast<uint4*>(hi + o) = *reinterpret_cast<const uint4*>(h);
  *reinterpret_cast<uint4*>(hi + o + 8) = *reinterpret_cast<const uint4*>(h + 8);
  if (lo != nullptr) {
    *reinterpret_cast<uint4*>(lo + o) = *reinterpret_cast<const uint4*>(l);
    *reinterpret_cast<uint4*>(lo + o + 8) = *reinterpret_cast<const uint4*>(l + 8);
  }
}

// The values of a partly cached page (global: [128 dims][16 tokens]) into a page buffer of the value tile (rows of
// 32 bytes under the 32-byte swizzle: the 16-byte halves of a row trade places when bit 2 of the row is set), the
// tokens from `cached` on zeroed: their memory may hold anything, and 0 * NaN would poison the product.  One warp.
__device__ __noinline__ void copy_partial_values(const __half* __restrict__ src, uint8_t* dst, int cached, int lane) {
#pragma unroll 1
  for (int j = 0; j < 8; ++j) {
    const int d = lane + 32 * (j >> 1), c = j & 1;
    __align__(16) __half hv[8];
    *reinterpret_cast<uint4*>(hv) = *reinterpret_cast<const uint4*>(src + (size_t)d * kPageTokens + c * 8);
#pragma unroll
    for (int x = 0; x < 8; ++x)
      if (c * 8 + x >= cached) hv[x] = __float2half_rn(0.f);
    *reinterpret_cast<uint4*>(dst + d * 32 + ((c ^ ((d >> 2) & 1)) << 4)) = *reinterpret_cast<const uint4*>(hv);
  }
  fence_async_smem();
}

template <typename OT>
__global__ void __launch_bounds__(kThreads, 1)
attn_chunk_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     const float* __restrict__ q, PassView p, const __half* __restrict__ pool,
                     const int32_t* __restrict__ page_table, int max_pages, OT* __restrict__ out, OT* __restrict__ out_lo,
                     int H, int KV, int QT, int* __restrict__ err) {
  RSD_PDL_SYNC();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* ring = smem;
  Meta* mt = reinterpret_cast<Meta*>(ring + kNS * kStageBytes);
  volatile uint32_t* stop = &mt->stop;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = H / KV, kvh = blockIdx.y, h0 = kvh * G;
  const int t0 = blockIdx.x * QT;
  const int n_ent = min(QT, p.T - t0);

  if (threadIdx.x < 128) {
    const int i = threadIdx.x;
    mt->row[i] = i < n_ent ? p.tok_row[t0 + i] : -1;
    mt->pos[i] = i < n_ent ? p.tok_pos[t0 + i] : 0;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kNS; ++s) { mbar_init(&mt->kv_full[s], 1); mbar_init(&mt->kv_empty[s], 1); }
    for (int b = 0; b < kSB; ++b) { mbar_init(&mt->s_full[b], 1); mbar_init(&mt->s_empty[b], kSoftmaxWarps); }
    for (int b = 0; b < 2; ++b) { mbar_init(&mt->p_full[b], kSoftmaxWarps); mbar_init(&mt->p_empty[b], 1); }
    mbar_init(&mt->o_full, 1); mbar_init(&mt->o_empty, kSoftmaxWarps);
    mbar_init(&mt->halves, kSoftmaxWarps);
    mt->stop = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) tmem_alloc(&mt->tmem_slot, kTmemCols);
  // the value buffers start zeroed: a buffer no page was fetched into is multiplied by weights that are exactly zero
  for (int i = threadIdx.x; i < kNS * (kVBytes / 16); i += kThreads)
    *reinterpret_cast<uint4*>(ring + (size_t)(i / (kVBytes / 16)) * kStageBytes + kKBytes + (size_t)(i % (kVBytes / 16)) * 16) =
        make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = mt->tmem_slot;
  // Q: row r = entry r / G, head r % G, as fp16 pairs in tensor memory, a warpgroup per half of the 128 dims; rows
  // beyond the tile's entries are zero.  1 / sqrt(head_dim) and log2(e) are folded in, so the scores come out in
  // units of log 2.
  if (threadIdx.x < kSoftmaxThreads) {
    const int r = threadIdx.x & 127, half = threadIdx.x >> 7, qi = r / G, g = r % G;
    const bool valid = r < QT * G && qi < n_ent && mt->row[qi] >= 0;
    const float scale = rsqrtf((float)kHd) * 1.4426950408889634f;
    const float* src = q + ((size_t)(t0 + qi) * H + h0 + g) * kHd + half * 64;
    uint32_t packed[32];
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
      if (valid) a = *reinterpret_cast<const float4*>(src + 4 * c);
      packed[2 * c] = pack_half2(a.x * scale, a.y * scale);
      packed[2 * c + 1] = pack_half2(a.z * scale, a.w * scale);
    }
    tmem_st32(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kColQ + half * 32, packed);
    tmem_st_wait();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  auto fail = [&]() {
    if (*stop == 0) { if (err) atomicCAS(err, 0, -5); *stop = 1; }
  };

  if (warp == kFetchWarp) {
    // ---------------- fetch warp: pages -> K-major tiles ----------------
    // Lanes 0-3 issue the key boxes of a tile's four pages, lanes 4-7 the value boxes; the whole warp copies the one
    // partly cached value page of a segment.  The loop is kept short: this warp paces the CTA.
    uint32_t it = 0;
    int seg = 0;
    bool ok = true;
    while (seg < n_ent && ok) {
      const int row = mt->row[seg];
      int e = seg + 1;
      while (e < n_ent && mt->row[e] == row) ++e;
      if (row >= 0) {
        const int pos_last = mt->pos[e - 1];
        const int n_pages = pos_last / kPageTokens + 1, n_tiles = (n_pages + 3) / 4;
        const int tail = (pos_last + 1) % kPageTokens;     // cached tokens of the last page when it is not full
        const int32_t* pt = page_table + (size_t)row * max_pages;
        for (int pass = 0; pass < 2 && ok; ++pass) {
          // The page ids are read 32 at a time (eight tiles), a batch ahead of their use: a lookup that the next
          // tile waited for would put a trip to the L2 into every tile.
          int pg_cur = lane < n_pages ? __ldg(pt + lane) : -1;
          int pg_nxt = 32 + lane < n_pages ? __ldg(pt + 32 + lane) : -1;
          for (int t = 0; t < n_tiles; ++t, ++it) {
            if (t > 0 && (t & 7) == 0) {
              pg_cur = pg_nxt;
              const int ahead = (t / 8 + 1) * 32 + lane;
              pg_nxt = ahead < n_pages ? __ldg(pt + ahead) : -1;
            }
            const int st = it % kNS;
            bool got = true;
            if (lane == 0) got = wait_sleep(&mt->kv_empty[st], ((it / kNS) & 1u) ^ 1u, stop);
            got = __all_sync(0xFFFFFFFFu, got && !*stop);          // one decision for the whole warp
            if (!got) { ok = false; break; }
            uint8_t* k_st = ring + (size_t)st * kStageBytes;
            const int i = lane & 3, page = 4 * t + i;              // this lane's page of the tile (lanes 0-7 issue)
            const int pg = __shfl_sync(0xFFFFFFFFu, pg_cur, page & 31);
            const bool partial = pass == 1 && tail != 0 && page == n_pages - 1;
            if (__any_sync(0xFFFFFFFFu, partial && lane < 4)) {
              // the last page of the segment, partly cached: the warp copies its values, the tokens beyond the cache zeroed
              const int last = n_pages - 1;
              const int pg_last = __shfl_sync(0xFFFFFFFFu, pg_cur, last & 31);
              copy_partial_values(pool + ((size_t)pg_last * 2 * KV + KV + kvh) * (kPageTokens * kHd),
                                  k_st + kKBytes + (last & 3) * kBlockBytes, tail, lane);
              __syncwarp();
            }
            const bool load_k = lane < 4 && page < n_pages;
            const bool load_v = lane >= 4 && lane < 8 && pass == 1 && page < n_pages && !partial;
            const uint32_t n_boxes = __popc(__ballot_sync(0xFFFFFFFFu, load_k || load_v));
            if (lane == 0) mbar_expect_tx(&mt->kv_full[st], n_boxes * kBlockBytes);
            __syncwarp();
            const int blk = pg * 2 * KV + kvh;
            if (load_k) tma_load_block_5d(k_st + i * kBlockBytes, &tm_k, &mt->kv_full[st], blk);
            if (load_v) tma_load_block_3d(k_st + kKBytes + i * kBlockBytes, &tm_v, &mt->kv_full[st], blk + KV);
          }
        }
      }
      seg = e;
    }
    // copies in flight must have landed before the CTA may leave: the last kNS tiles (all of them consumed already
    // when nothing went wrong)
    if (lane == 0) {
      const uint32_t first = it > (uint32_t)kNS ? it - kNS : 0;
      for (uint32_t j = first; j < it; ++j) mbar_wait(&mt->kv_full[j % kNS], (j / kNS) & 1u, kProbeLimit);
      if (!ok) fail();
    }
  } else if (warp == kMmaWarp) {
    // ---------------- score issuer: S = Q K^T of every tile, both passes ----------------
    if (lane == 0) {
      uint32_t itk = 0, its = 0;
      bool ok = true;
      int seg = 0;
      while (seg < n_ent && ok && !*stop) {
        const int row = mt->row[seg];
        int e = seg + 1;
        while (e < n_ent && mt->row[e] == row) ++e;
        if (row >= 0) {
          const int pos_last = mt->pos[e - 1];
          const int n_tiles = (pos_last / kPageTokens + 1 + 3) / 4;
          for (int pass = 0; pass < 2 && ok; ++pass) {
            for (int t = 0; t < n_tiles; ++t, ++itk, ++its) {
              const int st = itk % kNS;
              const uint32_t b = its % kSB;
              if (!mbar_wait(&mt->kv_full[st], (itk / kNS) & 1u, kProbeLimit) || *stop ||
                  !mbar_wait(&mt->s_empty[b], ((its / kSB) & 1u) ^ 1u, kProbeLimit) || *stop) { ok = false; break; }
              tc_fence_after();
              const uint64_t k_desc = desc_sw128(smem_u32(ring + (size_t)st * kStageBytes), 2048);
#pragma unroll
              for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                  umma_f16_ts(tmem_base + kColS + b * kKeys, tmem_base + kColQ + (hh * 4 + kk) * 8,
                              k_desc + (uint64_t)((hh * 1024 + kk * 32) >> 4), kIdescS, (hh > 0 || kk > 0) ? 1u : 0u);
              umma_commit(&mt->s_full[b]);
              // pass 1 reads the keys only: the stage is free once these MMAs have run; in pass 2 the output
              // issuer frees it after the values have been multiplied
              if (pass == 0) umma_commit(&mt->kv_empty[st]);
            }
          }
        }
        seg = e;
      }
      if (!ok) fail();
    }
  } else if (warp == kOutWarp) {
    // ---------------- output issuer: O += P V of every tile of pass 2 ----------------
    // A thread of its own, so that the wait for a tile's weights never holds up the scores of the next tiles.
    if (lane == 0) {
      uint32_t itk = 0, itp = 0, n_seg = 0;
      bool ok = true;
      int seg = 0;
      while (seg < n_ent && ok && !*stop) {
        const int row = mt->row[seg];
        int e = seg + 1;
        while (e < n_ent && mt->row[e] == row) ++e;
        if (row >= 0) {
          const int pos_last = mt->pos[e - 1];
          const int n_tiles = (pos_last / kPageTokens + 1 + 3) / 4;
          itk += n_tiles;                                  // the stages pass 1 went through
          // the output accumulator of the previous segment must have been read out
          if (n_seg > 0) ok = mbar_wait(&mt->o_empty, (n_seg - 1) & 1u, kProbeLimit) && !*stop;
          for (int t = 0; t < n_tiles && ok; ++t, ++itk, ++itp) {
            const int st = itk % kNS;
            const uint32_t pb = itp & 1u;
            // the weights imply the scores, and those the landed keys; the wait for the stage (over at once) makes
            // the landed values visible to this thread's MMAs
            if (!mbar_wait(&mt->p_full[pb], (itp >> 1) & 1u, kProbeLimit) || *stop ||
                !mbar_wait(&mt->kv_full[st], (itk / kNS) & 1u, kProbeLimit) || *stop) { ok = false; break; }
            tc_fence_after();
            const uint64_t v_desc = desc_sw32(smem_u32(ring + (size_t)st * kStageBytes + kKBytes));
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_f16_ts(tmem_base + kColO, tmem_base + kColP + pb * 32 + kk * 8, v_desc + (uint64_t)((kk * kBlockBytes) >> 4), kIdescO,
                          (t > 0 || kk > 0) ? 1u : 0u);
            umma_commit(&mt->kv_empty[st]);
            umma_commit(&mt->p_empty[pb]);
          }
          if (ok) { umma_commit(&mt->o_full); ++n_seg; }
        }
        seg = e;
      }
      if (!ok) fail();
    }
  } else {
    // ---------------- softmax warps: thread = tile row = tensor-memory lane, warpgroup = column half ----------------
    const int wg = warp >> 2, r = threadIdx.x & 127, qi = r / G, g = r % G;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const int c0 = wg * 32;                                // this thread's score columns of a tile
    uint32_t its = 0, itp = 0, n_seg = 0, n_x = 0;
    bool ok = true;
    // the warpgroups exchange their halves of a row statistic: post, wait (bounded, like every wait) until all eight
    // warps have posted.  A slot is written again only after MMAs that need every warp's later arrival, so the
    // readers of the previous value are done by then.
    auto exchange = [&](float (*slot)[128], float mine_half, float* a, float* b) -> bool {
      slot[wg][r] = mine_half;
      __syncwarp();
      if (lane == 0) mbar_arrive(&mt->halves);
      if (!wait_sleep(&mt->halves, n_x & 1u, stop)) return false;
      ++n_x;
      *a = slot[0][r]; *b = slot[1][r];
      return true;
    };
    int seg = 0;
    while (seg < n_ent && ok) {
      const int row = mt->row[seg];
      int e = seg + 1;
      while (e < n_ent && mt->row[e] == row) ++e;
      if (row >= 0) {
        const int pos_last = mt->pos[e - 1];
        const int n_tiles = (pos_last / kPageTokens + 1 + 3) / 4;
        const bool mine = r < QT * G && qi >= seg && qi < e;
        const int pq = mine ? mt->pos[qi] : -1;           // last visible key position; -1: the row is not of this segment
        float m = -INFINITY;
        for (int t = 0; t < n_tiles && ok; ++t, ++its) {
          const uint32_t b = its % kSB;
          ok = wait_sleep(&mt->s_full[b], (its / kSB) & 1u, stop);
          if (!ok) break;
          tc_fence_after();
          {
            float v[32];
            tmem_ld32(lane_base + kColS + b * kKeys + c0, v);
            const int k0 = t * kKeys + c0;
            if (k0 + 31 <= pq) {                           // all of these keys are visible to this row
#pragma unroll
              for (int j = 0; j < 32; ++j) m = fmaxf(m, v[j]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (k0 + j <= pq) m = fmaxf(m, v[j]);
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&mt->s_empty[b]);
        }
        if (!ok) break;
        {
          float ma, mb;
          ok = exchange(mt->pmax, m, &ma, &mb);
          if (!ok) break;
          m = fmaxf(ma, mb);
        }
        const float m_use = m == -INFINITY ? 0.f : m;
        float l = 0.f;
        for (int t = 0; t < n_tiles && ok; ++t, ++its, ++itp) {
          const uint32_t b = its % kSB, pb = itp & 1u;
          ok = wait_sleep(&mt->s_full[b], (its / kSB) & 1u, stop);
          if (!ok) break;
          tc_fence_after();
          uint32_t pv[16];
          {
            float v[32];
            tmem_ld32(lane_base + kColS + b * kKeys + c0, v);
            const int k0 = t * kKeys + c0;
            if (k0 + 31 <= pq) {
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = ex2(v[j] - m_use);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = (k0 + j <= pq) ? ex2(v[j] - m_use) : 0.f;
            }
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              l += v[j] + v[j + 1];
              pv[j >> 1] = pack_half2(v[j], v[j + 1]);
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&mt->s_empty[b]);
          // the weight tile of two tiles ago must have been multiplied
          ok = wait_sleep(&mt->p_empty[pb], ((itp >> 1) & 1u) ^ 1u, stop);
          if (!ok) break;
          tmem_st16(lane_base + kColP + pb * 32 + wg * 16, pv);
          tmem_st_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&mt->p_full[pb]);
        }
        if (!ok) break;
        // output: O / l for the rows of this segment, each warpgroup its 64 columns
        {
          float la, lb;
          ok = exchange(mt->psum, l, &la, &lb);
          if (!ok) break;
          l = la + lb;
        }
        ok = wait_sleep(&mt->o_full, n_seg & 1u, stop);
        if (!ok) break;
        tc_fence_after();
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const size_t o0 = ((size_t)(t0 + qi) * H + h0 + g) * kHd + wg * 64;
#pragma unroll
        for (int c = 0; c < 64; c += 32) {
          float v[32];
          tmem_ld32(lane_base + kColO + wg * 64 + c, v);
          if (mine) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] *= inv;
            store16<OT>(out, out_lo, o0 + c, v);
            store16<OT>(out, out_lo, o0 + c + 16, v + 16);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&mt->o_empty);
        ++n_seg;
      }
      seg = e;
    }
    if (!ok) fail();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

bool attn_chunk_tc_supported(int kv_dtype, int H, int KV, int hd, int T) {
  return kv_dtype == 2 && hd == kHd && KV >= 1 && H % KV == 0 && H / KV <= 8 && T >= 64;
}

cudaError_t launch_attn_chunk_tc(const float* q, PassView p, KvView kv, void* out, void* out_lo, int out_dtype, int H, int KV,
                                 int* err, cudaStream_t s) {
  if (p.T <= 0) return cudaSuccess;
  const int G = H / KV, QT = 128 / G;
  dim3 grid((p.T + QT - 1) / QT, KV);
  CUtensorMap tm_k, tm_v;
  if (!tc_tensor_map_kv(kv.pool_layer, 0, &tm_k) || !tc_tensor_map_kv(kv.pool_layer, 1, &tm_v)) return cudaErrorInvalidValue;
  static bool configured[3] = {false, false, false};
  if (out_dtype == 2) {      // one fp16 operand (out_lo unused)
    if (!configured[2]) {
      cudaError_t e = cudaFuncSetAttribute(attn_chunk_tc_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
      if (e != cudaSuccess) return e;
      configured[2] = true;
    }
    RSD_LAUNCH((attn_chunk_tc_kernel<__half>), grid, kThreads, kSmemBytes, s, tm_k, tm_v, q, p, (const __half*)kv.pool_layer,
               kv.page_table, kv.max_pages, (__half*)out, (__half*)nullptr, H, KV, QT, err);
  } else if (out_dtype == 1) {
    if (!configured[1]) {
      cudaError_t e = cudaFuncSetAttribute(attn_chunk_tc_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
      if (e != cudaSuccess) return e;
      configured[1] = true;
    }
    RSD_LAUNCH((attn_chunk_tc_kernel<__nv_bfloat16>), grid, kThreads, kSmemBytes, s, tm_k, tm_v, q, p, (const __half*)kv.pool_layer,
               kv.page_table, kv.max_pages, (__nv_bfloat16*)out, (__nv_bfloat16*)out_lo, H, KV, QT, err);
  } else {
    if (!configured[0]) {
      cudaError_t e = cudaFuncSetAttribute(attn_chunk_tc_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
      if (e != cudaSuccess) return e;
      configured[0] = true;
    }
    RSD_LAUNCH((attn_chunk_tc_kernel<float>), grid, kThreads, kSmemBytes, s, tm_k, tm_v, q, p, (const __half*)kv.pool_layer,
               kv.page_table, kv.max_pages, (float*)out, (float*)nullptr, H, KV, QT, err);
  }
  return launched(1);
}

}  // namespace rsd
