// Causal attention of a ragged chunk of new tokens over paged KV (prefill, PRM step scoring, draft
// sync, target catch-up), sm_100a tensor cores via mma.sync m16n8k16.
//
// The pass list is sorted by (row, position).  A CTA takes 16 consecutive list entries and one KV
// head; its warps are the G = H / KV query heads that share that KV head, so the warps of a CTA read
// the same keys and values at about the same time and share them through L1.  Entries of a tile that
// belong to different rows are handled one row segment at a time (queries outside the segment are
// masked); most tiles have a single segment.  Per warp the 16 queries are the 16 rows of the MMA tile:
//   S = Q K^T  keys stream from global memory into B fragments with 128-bit loads (head dims
//              permuted identically inside Q and K), causal mask by key position, online softmax per
//              query row (two rows per lane, reduced over the 4 lanes of a row);
//   O += P V   values are stored transposed inside a page, one 64-bit load per B fragment.
// Keys and values of the chunk itself were written to the pages before this kernel runs.
#include "common.cuh"
#include "kernels.cuh"

namespace rsd {

namespace {

template <typename KT> __device__ __forceinline__ uint32_t pack2c(float lo, float hi);
template <> __device__ __forceinline__ uint32_t pack2c<__nv_bfloat16>(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
template <> __device__ __forceinline__ uint32_t pack2c<__half>(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
template <typename KT> __device__ __forceinline__ void pack2c_split(float a, float b, uint32_t& hi, uint32_t& lo) {
  const KT ah = from_f32<KT>(a), bh = from_f32<KT>(b);
  hi = pack2c<KT>(to_f32(ah), to_f32(bh));
  lo = pack2c<KT>(a - to_f32(ah), b - to_f32(bh));
}
template <typename KT>
__device__ __forceinline__ void mma_c(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1);
template <>
__device__ __forceinline__ void mma_c<__nv_bfloat16>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <>
__device__ __forceinline__ void mma_c<__half>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// The pages of the row travel through a ring of shared-memory stages filled with cp.async by all warps of the CTA
// (the warps are the query heads of one KV head, so they all need the same keys and values): the copies of the next
// pages are in flight while the MMAs of the current page run, and every warp reads its fragments from shared
// memory instead of waiting for global memory page by page.  Key rows are padded by 16 bytes against bank conflicts.
// EXT: hi + lo pairs for the queries and the softmax weights, low halves of the values in a third block
// of every page (see the decode kernel).
template <int HD, typename KT, typename OT, bool EXT>
__global__ void __launch_bounds__(256)
attn_chunk_kernel(const float* __restrict__ q, PassView p, const KT* __restrict__ pool, const int32_t* __restrict__ page_table,
                  int max_pages, OT* __restrict__ out, OT* __restrict__ out_lo, int H, int KV) {
  RSD_PDL_SYNC();
  constexpr int KB = HD / 32, NT = HD / 8;
  constexpr int NS = EXT ? 2 : 4;              // ring stages (a stage: keys + values of one page, EXT: and their low halves)
  constexpr int KP = HD + 8;                   // padded key row
  __shared__ __align__(16) KT s_k[NS][kPageTokens][KP];
  __shared__ __align__(16) KT s_v[NS][HD][kPageTokens];
  __shared__ __align__(16) KT s_kl[EXT ? NS : 1][EXT ? kPageTokens : 1][EXT ? KP : 8];
  __shared__ __align__(16) KT s_vl[EXT ? NS : 1][EXT ? HD : 1][EXT ? kPageTokens : 8];
  const int G = H / KV;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_thr = blockDim.x;                // 32 * G: every thread belongs to a working warp
  const int kvh = blockIdx.y, h = kvh * G + warp;
  const int t0 = blockIdx.x * 16;
  const int n_tile = min(16, p.T - t0);
  const int g = lane >> 2, t = lane & 3;
  const float scale = rsqrtf((float)HD);
  const size_t block_elems = (size_t)KV * kPageTokens * HD;
  const size_t page_elems = (EXT ? 4 : 2) * block_elems;
  // key tokens of a page whose scores this lane holds: 4t, 4t+1 (first MMA tile), 4t+2, 4t+3 (second)
  const int tok0 = 4 * (g >> 1) + (g & 1), tok1 = tok0 + 2;

  // rows of the 16 entries, one per lane
  const int my_row = lane < n_tile ? p.tok_row[t0 + lane] : -2;
  int seg = 0;
  while (seg < n_tile) {
    const int r = __shfl_sync(0xFFFFFFFFu, my_row, seg);
    const unsigned same = __ballot_sync(0xFFFFFFFFu, my_row == r && lane >= seg);
    // the segment is the run of equal rows starting at `seg` (the list is sorted by row)
    const int seg_end = seg + __popc(same);
    if (r < 0) { seg = seg_end; continue; }
    const int pos_last = p.tok_pos[t0 + seg_end - 1];
    // the two query rows of this lane
    const bool v0 = g >= seg && g < seg_end, v1 = g + 8 >= seg && g + 8 < seg_end;
    const int pq0 = v0 ? p.tok_pos[t0 + g] : pos_last, pq1 = v1 ? p.tok_pos[t0 + g + 8] : pos_last;
    uint32_t qa[KB][2][4], ql[EXT ? KB : 1][2][4];
#pragma unroll
    for (int j = 0; j < KB; ++j) {
      float a[8], b[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        a[e] = v0 ? q[((size_t)(t0 + g) * H + h) * HD + 32 * j + 8 * t + e] : 0.f;
        b[e] = v1 ? q[((size_t)(t0 + g + 8) * H + h) * HD + 32 * j + 8 * t + e] : 0.f;
      }
      if (EXT) {
        pack2c_split<KT>(a[0], a[1], qa[j][0][0], ql[j][0][0]); pack2c_split<KT>(b[0], b[1], qa[j][0][1], ql[j][0][1]);
        pack2c_split<KT>(a[2], a[3], qa[j][0][2], ql[j][0][2]); pack2c_split<KT>(b[2], b[3], qa[j][0][3], ql[j][0][3]);
        pack2c_split<KT>(a[4], a[5], qa[j][1][0], ql[j][1][0]); pack2c_split<KT>(b[4], b[5], qa[j][1][1], ql[j][1][1]);
        pack2c_split<KT>(a[6], a[7], qa[j][1][2], ql[j][1][2]); pack2c_split<KT>(b[6], b[7], qa[j][1][3], ql[j][1][3]);
      } else {
        qa[j][0][0] = pack2c<KT>(a[0], a[1]); qa[j][0][1] = pack2c<KT>(b[0], b[1]);
        qa[j][0][2] = pack2c<KT>(a[2], a[3]); qa[j][0][3] = pack2c<KT>(b[2], b[3]);
        qa[j][1][0] = pack2c<KT>(a[4], a[5]); qa[j][1][1] = pack2c<KT>(b[4], b[5]);
        qa[j][1][2] = pack2c<KT>(a[6], a[7]); qa[j][1][3] = pack2c<KT>(b[6], b[7]);
      }
    }
    float o[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    const int32_t* pt = page_table + (size_t)r * max_pages;
    const int n_pages = pos_last / kPageTokens + 1;
    // one page -> one ring stage: 2 * HD pieces of 16 bytes for the keys (16 rows of HD) and as many for the values
    auto issue_page = [&](int pg) {
      if (pg < n_pages) {
        const int st = pg % NS;
        const KT* kb = pool + (size_t)pt[pg] * page_elems + (size_t)kvh * kPageTokens * HD;
        const KT* vb = pool + (size_t)pt[pg] * page_elems + block_elems + (size_t)kvh * HD * kPageTokens;
        for (int c = threadIdx.x; c < 2 * HD; c += n_thr) {
          const int r = c / (HD / 8), pc = c % (HD / 8);
          cp_async16(&s_k[st][r][pc * 8], kb + r * HD + pc * 8);
          cp_async16(&s_v[st][0][0] + c * 8, vb + c * 8);
          if (EXT) {
            cp_async16(&s_kl[st][r][pc * 8], kb + 2 * block_elems + r * HD + pc * 8);
            cp_async16(&s_vl[st][0][0] + c * 8, vb + 2 * block_elems + c * 8);
          }
        }
      }
      cp_async_commit();                       // one group per page, empty beyond the last
    };
    __syncthreads();                           // every warp has left the previous segment's stages
#pragma unroll
    for (int i = 0; i < NS - 1; ++i) issue_page(i);
    for (int pg = 0; pg < n_pages; ++pg) {
      cp_async_wait<NS - 2>();                 // this thread's copies of page pg have landed
      __syncthreads();                         // everyone's have, and everyone is done with page pg - 1
      issue_page(pg + NS - 1);                 // into the stage of page pg - 1
      const int st = pg % NS;
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < KB; ++j) {
        const uint4 k0 = *reinterpret_cast<const uint4*>(&s_k[st][tok0][32 * j + 8 * t]);
        const uint4 k1 = *reinterpret_cast<const uint4*>(&s_k[st][tok1][32 * j + 8 * t]);
        mma_c<KT>(s0, qa[j][0][0], qa[j][0][1], qa[j][0][2], qa[j][0][3], k0.x, k0.y);
        mma_c<KT>(s0, qa[j][1][0], qa[j][1][1], qa[j][1][2], qa[j][1][3], k0.z, k0.w);
        mma_c<KT>(s1, qa[j][0][0], qa[j][0][1], qa[j][0][2], qa[j][0][3], k1.x, k1.y);
        mma_c<KT>(s1, qa[j][1][0], qa[j][1][1], qa[j][1][2], qa[j][1][3], k1.z, k1.w);
        if (EXT) {
          const uint4 e0 = *reinterpret_cast<const uint4*>(&s_kl[EXT ? st : 0][EXT ? tok0 : 0][EXT ? 32 * j + 8 * t : 0]);
          const uint4 e1 = *reinterpret_cast<const uint4*>(&s_kl[EXT ? st : 0][EXT ? tok1 : 0][EXT ? 32 * j + 8 * t : 0]);
          mma_c<KT>(s0, qa[j][0][0], qa[j][0][1], qa[j][0][2], qa[j][0][3], e0.x, e0.y);
          mma_c<KT>(s0, qa[j][1][0], qa[j][1][1], qa[j][1][2], qa[j][1][3], e0.z, e0.w);
          mma_c<KT>(s1, qa[j][0][0], qa[j][0][1], qa[j][0][2], qa[j][0][3], e1.x, e1.y);
          mma_c<KT>(s1, qa[j][1][0], qa[j][1][1], qa[j][1][2], qa[j][1][3], e1.z, e1.w);
          mma_c<KT>(s0, ql[j][0][0], ql[j][0][1], ql[j][0][2], ql[j][0][3], k0.x, k0.y);
          mma_c<KT>(s0, ql[j][1][0], ql[j][1][1], ql[j][1][2], ql[j][1][3], k0.z, k0.w);
          mma_c<KT>(s1, ql[j][0][0], ql[j][0][1], ql[j][0][2], ql[j][0][3], k1.x, k1.y);
          mma_c<KT>(s1, ql[j][1][0], ql[j][1][1], ql[j][1][2], ql[j][1][3], k1.z, k1.w);
        }
      }
      // scores of query g: sa[e], of query g+8: sb[e], for key tokens base + 4t + e
      const int base = pg * kPageTokens + 4 * t;
      float sa[4] = {s0[0] * scale, s0[1] * scale, s1[0] * scale, s1[1] * scale};
      float sb[4] = {s0[2] * scale, s0[3] * scale, s1[2] * scale, s1[3] * scale};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (base + e > pq0) sa[e] = -INFINITY;
        if (base + e > pq1) sb[e] = -INFINITY;
      }
      float mxa = fmaxf(fmaxf(sa[0], sa[1]), fmaxf(sa[2], sa[3]));
      float mxb = fmaxf(fmaxf(sb[0], sb[1]), fmaxf(sb[2], sb[3]));
      mxa = fmaxf(mxa, __shfl_xor_sync(0xFFFFFFFFu, mxa, 1)); mxa = fmaxf(mxa, __shfl_xor_sync(0xFFFFFFFFu, mxa, 2));
      mxb = fmaxf(mxb, __shfl_xor_sync(0xFFFFFFFFu, mxb, 1)); mxb = fmaxf(mxb, __shfl_xor_sync(0xFFFFFFFFu, mxb, 2));
      const float na = fmaxf(m0, mxa), nb = fmaxf(m1, mxb);   // finite: key 0 is visible to every query
      const float ca = __expf(m0 - na), cb = __expf(m1 - nb);
      float pa[4], pb[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) { pa[e] = __expf(sa[e] - na); pb[e] = __expf(sb[e] - nb); }
      l0 = l0 * ca + (pa[0] + pa[1] + pa[2] + pa[3]);
      l1 = l1 * cb + (pb[0] + pb[1] + pb[2] + pb[3]);
      m0 = na; m1 = nb;
      uint32_t a0, a1, a2, a3, l0p = 0u, l1p = 0u, l2p = 0u, l3p = 0u;
      if (EXT) {
        pack2c_split<KT>(pa[0], pa[1], a0, l0p); pack2c_split<KT>(pb[0], pb[1], a1, l1p);
        pack2c_split<KT>(pa[2], pa[3], a2, l2p); pack2c_split<KT>(pb[2], pb[3], a3, l3p);
      } else {
        a0 = pack2c<KT>(pa[0], pa[1]); a1 = pack2c<KT>(pb[0], pb[1]);
        a2 = pack2c<KT>(pa[2], pa[3]); a3 = pack2c<KT>(pb[2], pb[3]);
      }
      // values of tokens beyond the last cached position of the row may be uninitialised memory
      const int n_valid = min(kPageTokens, pos_last + 1 - pg * kPageTokens);
      uint32_t mlo = 0xFFFFFFFFu, mhi = 0xFFFFFFFFu;
      if (n_valid < kPageTokens) {
        mlo = (4 * t < n_valid ? 0x0000FFFFu : 0u) | (4 * t + 1 < n_valid ? 0xFFFF0000u : 0u);
        mhi = (4 * t + 2 < n_valid ? 0x0000FFFFu : 0u) | (4 * t + 3 < n_valid ? 0xFFFF0000u : 0u);
      }
#pragma unroll
      for (int i = 0; i < NT; ++i) {
        const uint2 vv = *reinterpret_cast<const uint2*>(&s_v[st][8 * i + g][4 * t]);
        o[i][0] *= ca; o[i][1] *= ca; o[i][2] *= cb; o[i][3] *= cb;
        mma_c<KT>(o[i], a0, a1, a2, a3, vv.x & mlo, vv.y & mhi);
        if (EXT) {
          const uint2 vl = *reinterpret_cast<const uint2*>(&s_vl[EXT ? st : 0][EXT ? 8 * i + g : 0][EXT ? 4 * t : 0]);
          mma_c<KT>(o[i], l0p, l1p, l2p, l3p, vv.x & mlo, vv.y & mhi);
          mma_c<KT>(o[i], a0, a1, a2, a3, vl.x & mlo, vl.y & mhi);
        }
      }
    }
    l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 1); l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 2);
    l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 1); l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 2);
    const float i0 = 1.f / l0, i1 = 1.f / l1;
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      if (v0) {
        const size_t o0 = ((size_t)(t0 + g) * H + h) * HD + 8 * i + 2 * t;
        store_operand<OT>(out, out_lo, o0, o[i][0] * i0);
        store_operand<OT>(out, out_lo, o0 + 1, o[i][1] * i0);
      }
      if (v1) {
        const size_t o1 = ((size_t)(t0 + g + 8) * H + h) * HD + 8 * i + 2 * t;
        store_operand<OT>(out, out_lo, o1, o[i][2] * i1);
        store_operand<OT>(out, out_lo, o1 + 1, o[i][3] * i1);
      }
    }
    seg = seg_end;
  }
}

}  // namespace

cudaError_t launch_attn_chunk(int kv_dtype, const float* q, PassView p, KvView kv, void* out, void* out_lo,
                              int out_dtype, int H, int KV, int hd, cudaStream_t s, int* err) {
  if (p.T <= 0) return cudaSuccess;
  if (attn_chunk_tc_supported(kv_dtype, H, KV, hd, p.T))
    return launch_attn_chunk_tc(q, p, kv, out, out_lo, out_dtype, H, KV, err, s);
  if (out_dtype == 2) return cudaErrorNotSupported;   // a single fp16 operand is written by the tcgen05 kernel only
  const int G = H / KV;
  if (kv_dtype == 3) kv.v_extra = 1;
  if (kv_dtype == 0 || G > 8)
    return launch_attn_generic(kv_dtype == 3 ? 2 : kv_dtype, q, p, kv, out, out_lo, out_dtype, H, KV, hd, s);
  dim3 grid((p.T + 15) / 16, KV);
  const int threads = 32 * G;
#define RSD_CH(HD, KT, OT, EXTV) \
  RSD_LAUNCH((attn_chunk_kernel<HD, KT, OT, EXTV>), grid, threads, 0, s, q, p, (const KT*)kv.pool_layer, kv.page_table, kv.max_pages, (OT*)out, (OT*)out_lo, H, KV)
#define RSD_CH_O(HD, KT, EXTV) do { if (out_dtype == 1) RSD_CH(HD, KT, __nv_bfloat16, EXTV); else RSD_CH(HD, KT, float, EXTV); } while (0)
  if (kv_dtype == 3) { if (hd == 128) RSD_CH_O(128, __half, true); else RSD_CH_O(64, __half, true); }
  else if (kv_dtype == 2) { if (hd == 128) RSD_CH_O(128, __half, false); else RSD_CH_O(64, __half, false); }
  else { if (hd == 128) RSD_CH_O(128, __nv_bfloat16, false); else RSD_CH_O(64, __nv_bfloat16, false); }
#undef RSD_CH_O
#undef RSD_CH
  return launched(1);
}

}  // namespace rsd
