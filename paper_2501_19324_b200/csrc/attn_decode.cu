// Paged-KV grouped-query decode attention (one query token per row), sm_100a.
//
// A CTA of 4 warps serves one (row slot, KV head, context split): the G = H / KV query heads that
// share the KV head are the rows of a 16-row MMA tile, so every key / value is read once from HBM for
// the whole group.  Each warp walks its share of the 16-token pages:
//   S  = Q K^T   with mma.sync m16n8k16 (bf16 in, fp32 out): keys stream from global memory straight
//        into B fragments with 128-bit loads (the order of the head dims inside a 32-dim block is
//        permuted identically for Q and K, which a dot product does not see);
//   softmax statistics per head are kept on line (running max / sum), reduced over the 4 lanes that
//        share a row with warp shuffles;
//   O += P V     with the same MMA: values are stored transposed inside a page ([hd][16 tokens]), so a
//        B fragment is one 64-bit load; the order of the tokens inside a page is permuted identically
//        for P and V.
// The warps' partial (max, sum, O) meet in shared memory.  With 2 to 8 context splits the splits of a (slot, KV
// head) are the CTAs of one thread-block cluster: each leaves its partial in its own shared memory, and after a
// cluster barrier every CTA merges a slice of the G x HD outputs out of all the CTAs' shared memory (in split
// order) and writes it: no second launch and no trip through global memory.  With more splits than a cluster
// holds the CTA writes its partial to scratch and a second kernel merges them.
#include <cooperative_groups.h>

#include "common.cuh"
#include "kernels.cuh"

namespace rsd {

namespace {

constexpr int kMaxSplits = 32;

// Two fp32 values rounded to the cache's 16-bit type and packed into one MMA operand register.
template <typename KT> __device__ __forceinline__ uint32_t pack2(float lo, float hi);
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
template <> __device__ __forceinline__ uint32_t pack2<__half>(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// The same pair split into a high and a low 16-bit part: (a, b) = hi + lo up to ~2^-22 relative.
template <typename KT> __device__ __forceinline__ void pack2_split(float a, float b, uint32_t& hi, uint32_t& lo) {
  const KT ah = from_f32<KT>(a), bh = from_f32<KT>(b);
  hi = pack2<KT>(to_f32(ah), to_f32(bh));
  lo = pack2<KT>(a - to_f32(ah), b - to_f32(bh));
}

template <typename KT>
__device__ __forceinline__ void mma_16816(float& d0, float& d1, float& d2, float& d3, uint32_t a0, uint32_t a1, uint32_t a2,
                                          uint32_t a3, uint32_t b0, uint32_t b1);
template <>
__device__ __forceinline__ void mma_16816<__nv_bfloat16>(float& d0, float& d1, float& d2, float& d3, uint32_t a0, uint32_t a1,
                                                         uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3)
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <>
__device__ __forceinline__ void mma_16816<__half>(float& d0, float& d1, float& d2, float& d3, uint32_t a0, uint32_t a1,
                                                  uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3)
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// part_o: [slot][head][split][HD] un-normalised outputs; part_ml: [slot][head][split][2] (max, sum).
// EXT: queries and softmax weights enter the products as hi + lo pairs and every page carries the low
// halves of its keys and values in two more blocks: the attention is accurate to about 2^-20.
template <int HD, typename KT, typename OT, bool EXT, bool CL>
__global__ void __launch_bounds__(128, EXT ? 2 : 4)
attn_decode_kernel(const float* __restrict__ q, const KT* __restrict__ pool, const int32_t* __restrict__ page_table,
                   int max_pages, const int32_t* __restrict__ slot_row, const int32_t* __restrict__ len_or_pos, int len_offset,
                   OT* __restrict__ out, OT* __restrict__ out_lo, float* __restrict__ part_o, float* __restrict__ part_ml, int H, int KV, int n_splits,
                   const int32_t* __restrict__ n_active) {
  RSD_PDL_SYNC();
  if (n_active != nullptr && *n_active == 0) return;
  constexpr int KB = HD / 32;    // 32-dim blocks of the head dimension
  constexpr int NT = HD / 8;     // 8-dim output tiles
  __shared__ float s_m[4][8], s_l[4][8];
  __shared__ float s_o[4][8][HD];
  const int kvh = blockIdx.x, slot = blockIdx.y, split = blockIdx.z;
  const int row = slot_row ? slot_row[slot] : slot;
  if (row < 0) return;
  const int ctx = len_or_pos[slot] + len_offset;
  if (ctx <= 0) return;
  const int G = H / KV, h0 = kvh * G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const float scale = rsqrtf((float)HD);

  const int n_pages = (ctx + kPageTokens - 1) / kPageTokens;
  const int pps = (n_pages + n_splits - 1) / n_splits;
  const int p_begin = split * pps, p_end = min(n_pages, p_begin + pps);

  // Q fragments (rows 8..15 of the tile are padding): dims 32j + 8t + e of head h0 + g
  uint32_t qa[KB][2][2], ql[EXT ? KB : 1][2][2];
#pragma unroll
  for (int j = 0; j < KB; ++j) {
    float v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = g < G ? q[((size_t)slot * H + h0 + g) * HD + 32 * j + 8 * t + e] : 0.f;
    if (EXT) {
      pack2_split<KT>(v[0], v[1], qa[j][0][0], ql[j][0][0]); pack2_split<KT>(v[2], v[3], qa[j][0][1], ql[j][0][1]);
      pack2_split<KT>(v[4], v[5], qa[j][1][0], ql[j][1][0]); pack2_split<KT>(v[6], v[7], qa[j][1][1], ql[j][1][1]);
    } else {
      qa[j][0][0] = pack2<KT>(v[0], v[1]); qa[j][0][1] = pack2<KT>(v[2], v[3]);
      qa[j][1][0] = pack2<KT>(v[4], v[5]); qa[j][1][1] = pack2<KT>(v[6], v[7]);
    }
  }
  // Rows 8..15 of every MMA tile are padding (their A rows are zero), so all tiles share two dump
  // registers for those rows instead of carrying 2 x (NT + 2) dead accumulators.
  float o[NT][2];
#pragma unroll
  for (int i = 0; i < NT; ++i) { o[i][0] = o[i][1] = 0.f; }
  float dump0 = 0.f, dump1 = 0.f;
  float m_run = -INFINITY, l_run = 0.f;

  const int32_t* pt = page_table + (size_t)row * max_pages;
  const size_t block_elems = (size_t)KV * kPageTokens * HD;
  const size_t page_elems = (EXT ? 4 : 2) * block_elems;
  // tokens whose keys this lane loads: tile 0 -> 4(g/2) + g%2, tile 1 -> that + 2
  const int tok0 = 4 * (g >> 1) + (g & 1), tok1 = tok0 + 2;
  int page = (p_begin + warp < p_end) ? pt[p_begin + warp] : 0;
  for (int p = p_begin + warp; p < p_end; p += 4) {
    const KT* kb = pool + (size_t)page * page_elems + (size_t)kvh * kPageTokens * HD;
    const KT* vb = pool + (size_t)page * page_elems + (size_t)KV * kPageTokens * HD + (size_t)kvh * HD * kPageTokens;
    if (p + 4 < p_end) page = pt[p + 4];     // next page's index is fetched while this page is worked on
    // all of the page's keys and values are requested up front (8 KB per warp in flight)
    uint4 k0[KB], k1[KB];
    uint2 vv[NT], vl[EXT ? NT : 1];
#pragma unroll
    for (int j = 0; j < KB; ++j) {
      k0[j] = *reinterpret_cast<const uint4*>(kb + tok0 * HD + 32 * j + 8 * t);
      k1[j] = *reinterpret_cast<const uint4*>(kb + tok1 * HD + 32 * j + 8 * t);
    }
#pragma unroll
    for (int i = 0; i < NT; ++i) vv[i] = *reinterpret_cast<const uint2*>(vb + (size_t)(8 * i + g) * kPageTokens + 4 * t);
    if (EXT) {
#pragma unroll
      for (int i = 0; i < NT; ++i) vl[i] = *reinterpret_cast<const uint2*>(vb + 2 * block_elems + (size_t)(8 * i + g) * kPageTokens + 4 * t);
    }
    float s0[2] = {0.f, 0.f}, s1[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < KB; ++j) {
      mma_16816<KT>(s0[0], s0[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, k0[j].x, k0[j].y);
      mma_16816<KT>(s0[0], s0[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, k0[j].z, k0[j].w);
      mma_16816<KT>(s1[0], s1[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, k1[j].x, k1[j].y);
      mma_16816<KT>(s1[0], s1[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, k1[j].z, k1[j].w);
      if (EXT) {
        const uint4 e0 = *reinterpret_cast<const uint4*>(kb + 2 * block_elems + tok0 * HD + 32 * j + 8 * t);
        const uint4 e1 = *reinterpret_cast<const uint4*>(kb + 2 * block_elems + tok1 * HD + 32 * j + 8 * t);
        mma_16816<KT>(s0[0], s0[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, e0.x, e0.y);
        mma_16816<KT>(s0[0], s0[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, e0.z, e0.w);
        mma_16816<KT>(s1[0], s1[1], dump0, dump1, qa[j][0][0], 0u, qa[j][0][1], 0u, e1.x, e1.y);
        mma_16816<KT>(s1[0], s1[1], dump0, dump1, qa[j][1][0], 0u, qa[j][1][1], 0u, e1.z, e1.w);
        mma_16816<KT>(s0[0], s0[1], dump0, dump1, ql[j][0][0], 0u, ql[j][0][1], 0u, k0[j].x, k0[j].y);
        mma_16816<KT>(s0[0], s0[1], dump0, dump1, ql[j][1][0], 0u, ql[j][1][1], 0u, k0[j].z, k0[j].w);
        mma_16816<KT>(s1[0], s1[1], dump0, dump1, ql[j][0][0], 0u, ql[j][0][1], 0u, k1[j].x, k1[j].y);
        mma_16816<KT>(s1[0], s1[1], dump0, dump1, ql[j][1][0], 0u, ql[j][1][1], 0u, k1[j].z, k1[j].w);
      }
    }
    // this lane's scores of head g: tokens 4t, 4t+1 (tile 0) and 4t+2, 4t+3 (tile 1) of the page
    const int n_valid = min(kPageTokens, ctx - p * kPageTokens);
    float sc[4] = {s0[0] * scale, s0[1] * scale, s1[0] * scale, s1[1] * scale};
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (4 * t + e >= n_valid) sc[e] = -INFINITY;
    float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
    const float m_new = fmaxf(m_run, mx);          // finite: token 0 of the page is always valid
    const float corr = __expf(m_run - m_new);
    float pr[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) pr[e] = __expf(sc[e] - m_new);
    l_run = l_run * corr + (pr[0] + pr[1] + pr[2] + pr[3]);
    m_run = m_new;
    uint32_t pa0, pa2, pl0 = 0u, pl2 = 0u;
    if (EXT) { pack2_split<KT>(pr[0], pr[1], pa0, pl0); pack2_split<KT>(pr[2], pr[3], pa2, pl2); }
    else { pa0 = pack2<KT>(pr[0], pr[1]); pa2 = pack2<KT>(pr[2], pr[3]); }
    // mask of the 16-bit halves of a value fragment that belong to cached tokens
    uint32_t mlo = 0xFFFFFFFFu, mhi = 0xFFFFFFFFu;
    if (n_valid < kPageTokens) {
      mlo = (4 * t < n_valid ? 0x0000FFFFu : 0u) | (4 * t + 1 < n_valid ? 0xFFFF0000u : 0u);
      mhi = (4 * t + 2 < n_valid ? 0x0000FFFFu : 0u) | (4 * t + 3 < n_valid ? 0xFFFF0000u : 0u);
    }
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      o[i][0] *= corr; o[i][1] *= corr;
      mma_16816<KT>(o[i][0], o[i][1], dump0, dump1, pa0, 0u, pa2, 0u, vv[i].x & mlo, vv[i].y & mhi);
      if (EXT) {
        mma_16816<KT>(o[i][0], o[i][1], dump0, dump1, pl0, 0u, pl2, 0u, vv[i].x & mlo, vv[i].y & mhi);
        mma_16816<KT>(o[i][0], o[i][1], dump0, dump1, pa0, 0u, pa2, 0u, vl[i].x & mlo, vl[i].y & mhi);
      }
    }
  }
  // the 4 lanes of a row hold partial sums of l
  l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
  l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
  if (t == 0) { s_m[warp][g] = m_run; s_l[warp][g] = l_run; }
#pragma unroll
  for (int i = 0; i < NT; ++i) {
    s_o[warp][g][8 * i + 2 * t] = o[i][0];
    s_o[warp][g][8 * i + 2 * t + 1] = o[i][1];
  }
  __syncthreads();
  __shared__ float c_m[8], c_l[8];               // cluster mode: this CTA's (max, sum) per head; its O goes to s_o[0]
  for (int idx = threadIdx.x; idx < G * HD; idx += blockDim.x) {
    const int gg = idx / HD, dd = idx % HD;
    float M = fmaxf(fmaxf(s_m[0][gg], s_m[1][gg]), fmaxf(s_m[2][gg], s_m[3][gg]));
    float L = 0.f, O = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float e = __expf(s_m[w][gg] - M);
        L += s_l[w][gg] * e;
        O += s_o[w][gg][dd] * e;
      }
    }
    const int h = h0 + gg;
    if (CL) {
      // (gg, dd) is this thread's alone: it has read the four warps' values and may overwrite the first
      s_o[0][gg][dd] = O;
      if (dd == 0) { c_m[gg] = M; c_l[gg] = L; }
    } else if (n_splits == 1) {
      store_operand<OT>(out, out_lo, ((size_t)slot * H + h) * HD + dd, O / L);
    } else {
      const size_t base = ((size_t)slot * H + h) * n_splits + split;
      part_o[base * HD + dd] = O;
      if (dd == 0) { part_ml[base * 2] = M; part_ml[base * 2 + 1] = L; }
    }
  }
  if (CL) {
    // Every CTA of the cluster gets here (the early returns above depend on the slot alone, which the cluster
    // shares).  Rank = split.  A CTA merges the outputs [rank * per, rank * per + per) of the G x HD.
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();
    const int n_rank = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int total = G * HD, per = (total + n_rank - 1) / n_rank;
    const int end = min(total, (rank + 1) * per);
    for (int idx = rank * per + threadIdx.x; idx < end; idx += blockDim.x) {
      const int gg = idx / HD, dd = idx % HD;
      float pm[8], pl[8], po[8];
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        if (r < n_rank) {
          pm[r] = *cluster.map_shared_rank(&c_m[gg], r);
          pl[r] = *cluster.map_shared_rank(&c_l[gg], r);
          po[r] = *cluster.map_shared_rank(&s_o[0][gg][dd], r);
        } else {
          pm[r] = -INFINITY; pl[r] = 0.f; po[r] = 0.f;
        }
      }
      float M = -INFINITY, L = 0.f, O = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        if (pm[r] > -INFINITY) {
          const float Mn = fmaxf(M, pm[r]);
          const float e_old = __expf(M - Mn), e_new = __expf(pm[r] - Mn);
          L = L * e_old + pl[r] * e_new;
          O = O * e_old + po[r] * e_new;
          M = Mn;
        }
      }
      store_operand<OT>(out, out_lo, ((size_t)slot * H + h0 + gg) * HD + dd, O / L);
    }
    cluster.sync();                              // nobody leaves while its shared memory may still be read
  }
}

template <int HD, typename OT>
__global__ void __launch_bounds__(HD)
attn_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml, const int32_t* __restrict__ slot_row,
                  const int32_t* __restrict__ len_or_pos, int len_offset, OT* __restrict__ out, OT* __restrict__ out_lo,
                  int H, int n_splits, const int32_t* __restrict__ n_active) {
  RSD_PDL_SYNC();
  if (n_active != nullptr && *n_active == 0) return;
  const int slot = blockIdx.y, h = blockIdx.x, dd = threadIdx.x;
  if ((slot_row && slot_row[slot] < 0) || len_or_pos[slot] + len_offset <= 0) return;
  const size_t base = ((size_t)slot * H + h) * n_splits;
  // four splits at a time with every load of the group in flight together; running maximum as in the kernel above
  float M = -INFINITY, L = 0.f, O = 0.f;
  for (int s0 = 0; s0 < n_splits; s0 += 4) {
    float2 ml[4];
    float ov[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const bool in = s0 + u < n_splits;
      ml[u] = in ? *reinterpret_cast<const float2*>(part_ml + (base + s0 + u) * 2) : make_float2(-INFINITY, 0.f);
      ov[u] = in ? part_o[(base + s0 + u) * HD + dd] : 0.f;
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
  store_operand<OT>(out, out_lo, ((size_t)slot * H + h) * HD + dd, O / L);
}

__global__ void decode_slots_kernel(const int32_t* slot_row, const int32_t* len_or_pos, int len_offset, int32_t* row,
                                    int32_t* pos, int B) {
  RSD_PDL_SYNC();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B) return;
  const int r = slot_row ? slot_row[i] : i;
  const int ctx = len_or_pos[i] + len_offset;
  row[i] = (r >= 0 && ctx >= 1) ? r : -1;
  pos[i] = ctx - 1;
}

constexpr int kClusterSplits = 8;   // the portable cluster size

int pick_splits(int B, int KV, int max_ctx) {
  const int ctas = B * KV;
  int splits = (4 * 148) / ctas;   // one wave of at most four CTAs per SM: a second, partial wave would double the time
  const int max_by_ctx = std::max(1, (max_ctx / kPageTokens) / 4);   // at least 4 pages per split (one per warp)
  splits = std::min(splits, max_by_ctx);
  splits = std::max(1, std::min(splits, kMaxSplits));
  // a few splits more than a cluster holds are not worth the second launch: 8 splits of 16 or more (slot, KV head)
  // pairs already put a CTA on most SMs
  if (splits > kClusterSplits && ctas * kClusterSplits >= 128) splits = kClusterSplits;
  return splits;
}

// Launch with programmatic stream serialisation and, when cluster_z > 1, clusters of cluster_z CTAs along z.
template <typename... KArgs, typename... Args>
cudaError_t launch_decode(void (*kernel)(KArgs...), dim3 grid, int cluster_z, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(128);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.numAttrs = 1;
  if (cluster_z > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = (unsigned)cluster_z;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

}  // namespace

size_t attn_decode_scratch_bytes(int B, int H, int hd, int max_ctx) {
  (void)max_ctx;
  const size_t partials = (size_t)B * H * kMaxSplits * (hd + 2) * sizeof(float);
  return sizeof(int32_t) * 2 * (size_t)B + 256 + partials;
}

cudaError_t launch_attn_decode(int kv_dtype, const float* q, const void* pool_layer, const int32_t* page_table,
                               int max_pages, const int32_t* slot_row, const int32_t* len_or_pos, int len_offset,
                               void* out, void* out_lo, int out_dtype, int B, int H, int KV, int hd, int max_ctx,
                               void* scratch, size_t scratch_bytes, const int32_t* n_active, cudaStream_t s, int active_rows) {
  if (B <= 0) return cudaSuccess;
  if (!scratch || scratch_bytes < attn_decode_scratch_bytes(B, H, hd, max_ctx)) return cudaErrorInvalidValue;
  const int G = H / KV;
  int32_t* row = (int32_t*)scratch;
  int32_t* pos = row + B;
  if (kv_dtype == 0 || G > 8) {
    // fp32 caches and wide groups take the generic kernel
    RSD_LAUNCH((decode_slots_kernel), (B + 255) / 256, 256, 0, s, slot_row, len_or_pos, len_offset, row, pos, B);
    launched(1);
    PassView p{nullptr, row, pos, B, n_active};
    KvView kv{const_cast<void*>(pool_layer), page_table, max_pages, kv_dtype == 3 ? 1 : 0};
    return launch_attn_generic(kv_dtype == 3 ? 2 : kv_dtype, q, p, kv, out, out_lo, out_dtype, H, KV, hd, s);
  }
  const size_t head = ((sizeof(int32_t) * 2 * (size_t)B + 255) / 256) * 256;
  float* part_ml = (float*)((char*)scratch + head);
  float* part_o = part_ml + (size_t)B * H * kMaxSplits * 2;
  const int splits = pick_splits(active_rows > 0 ? std::min(active_rows, B) : B, KV, max_ctx);
  const bool clustered = splits >= 2 && splits <= kClusterSplits;
  dim3 grid(KV, B, splits);
#define RSD_DEC(HD, KT, OT, EXTV)                                                                                          \
  do {                                                                                                               \
    if (clustered)                                                                                                   \
      (void)launch_decode(attn_decode_kernel<HD, KT, OT, EXTV, true>, grid, splits, s, q, (const KT*)pool_layer, page_table,       \
                          max_pages, slot_row, len_or_pos, len_offset, (OT*)out, (OT*)out_lo, part_o, part_ml, H, KV, splits, n_active); \
    else                                                                                                             \
      (void)launch_decode(attn_decode_kernel<HD, KT, OT, EXTV, false>, grid, 1, s, q, (const KT*)pool_layer, page_table,           \
                          max_pages, slot_row, len_or_pos, len_offset, (OT*)out, (OT*)out_lo, part_o, part_ml, H, KV, splits, n_active); \
    if (splits > 1 && !clustered)                                                                                    \
      RSD_LAUNCH((attn_merge_kernel<HD, OT>), dim3(H, B), HD, 0, s, part_o, part_ml, slot_row, len_or_pos, len_offset, (OT*)out, \
                                                          (OT*)out_lo, H, splits, n_active);                         \
  } while (0)
#define RSD_DEC_O(HD, KT, EXTV) do { if (out_dtype == 1) RSD_DEC(HD, KT, __nv_bfloat16, EXTV); else RSD_DEC(HD, KT, float, EXTV); } while (0)
  if (kv_dtype == 3) { if (hd == 128) RSD_DEC_O(128, __half, true); else RSD_DEC_O(64, __half, true); }
  else if (kv_dtype == 2) { if (hd == 128) RSD_DEC_O(128, __half, false); else RSD_DEC_O(64, __half, false); }
  else { if (hd == 128) RSD_DEC_O(128, __nv_bfloat16, false); else RSD_DEC_O(64, __nv_bfloat16, false); }
#undef RSD_DEC_O
#undef RSD_DEC
  return launched(splits > 1 && !clustered ? 2 : 1);
}

}  // namespace rsd
