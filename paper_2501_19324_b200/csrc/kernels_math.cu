// Element-wise, normalisation, rotary, SIMT GEMV, attention, sampling and reward kernels of the RSD
// step loop (sm_100a).  The residual stream and every reduction are fp32; weights, GEMM inputs and
// the KV cache are stored in the model's element type (fp32 or bfloat16).
#include "common.cuh"
#include "kernels.cuh"

namespace rsd {

#define RSD_SKIP_IF_IDLE(n_active) \
  if ((n_active) != nullptr && *(n_active) == 0) return;

// ---------------------------------------------------------------------------------------------
// Embedding gather: x[t, :] = E[tok_id[t], :]
// ---------------------------------------------------------------------------------------------
template <typename WT>
__global__ void embed_kernel(const WT* __restrict__ E, PassView p, float* __restrict__ x, int d) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(p.n_active);
  const int t = blockIdx.x;
  if (p.tok_row[t] < 0) return;
  const WT* src = E + (size_t)p.tok_id[t] * d;
  float* dst = x + (size_t)t * d;
  constexpr int N = Vec16<WT>::N;
  for (int i = threadIdx.x * N; i < d; i += blockDim.x * N) {
    Vec16<WT> v;
    v.load(src + i);
#pragma unroll
    for (int j = 0; j < N; ++j) dst[i + j] = v.v[j];
  }
}

cudaError_t launch_embed(int dtype, const void* embed, PassView p, float* x, int d, cudaStream_t s) {
  if (p.T <= 0) return cudaSuccess;
  if (dtype == 1) RSD_LAUNCH((embed_kernel<__nv_bfloat16>), p.T, 128, 0, s, (const __nv_bfloat16*)embed, p, x, d);
  else RSD_LAUNCH((embed_kernel<float>), p.T, 128, 0, s, (const float*)embed, p, x, d);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// RMSNorm: out = x * gain / sqrt(mean(x^2) + eps), one block per token, x kept in registers
// ---------------------------------------------------------------------------------------------
template <typename OT, typename GT>
__global__ void rmsnorm_kernel(float* __restrict__ x, const GT* __restrict__ gain, OT* __restrict__ out,
                               OT* __restrict__ out_lo, int d, float eps, const int32_t* __restrict__ src,
                               const int32_t* n_active, const float* __restrict__ partials, int splits, int T) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(n_active);
  __shared__ float red[33];
  const int t = blockIdx.x;
  int st = t;
  if (src != nullptr) {
    st = src[t];
    if (st < 0) return;
  }
  float* xr = x + (size_t)st * d;
  float ss = 0.f;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(xr + i);
    if (splits > 1) {
      // the producing GEMM left K-split partial sums: fold them into the residual stream here
      int sidx = 0;
      for (; sidx + 8 <= splits; sidx += 8) {
        float4 a[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) a[u] = __ldcg(reinterpret_cast<const float4*>(partials + ((size_t)(sidx + u) * T + st) * d + i));
#pragma unroll
        for (int u = 0; u < 8; ++u) { v.x += a[u].x; v.y += a[u].y; v.z += a[u].z; v.w += a[u].w; }
      }
      for (; sidx < splits; ++sidx) {
        const float4 a = __ldcg(reinterpret_cast<const float4*>(partials + ((size_t)sidx * T + st) * d + i));
        v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
      }
      *reinterpret_cast<float4*>(xr + i) = v;
    }
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, red);
  const float inv = rsqrtf(ss / (float)d + eps);
  const size_t o = (size_t)t * d;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(xr + i);
    store_operand<OT>(out, out_lo, o + i, v.x * inv * to_f32(gain[i]));
    store_operand<OT>(out, out_lo, o + i + 1, v.y * inv * to_f32(gain[i + 1]));
    store_operand<OT>(out, out_lo, o + i + 2, v.z * inv * to_f32(gain[i + 2]));
    store_operand<OT>(out, out_lo, o + i + 3, v.w * inv * to_f32(gain[i + 3]));
  }
}

// bf16 -> fp16, element by element (n a multiple of 8: weight matrices are).
__global__ void bf16_to_f16_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n8) {
  RSD_PDL_SYNC();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
    uint4 v = src[i];
    const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&v);
    uint4 o;
    __half2* h = reinterpret_cast<__half2*>(&o);
#pragma unroll
    for (int k = 0; k < 4; ++k) h[k] = __floats2half2_rn(__low2float(b[k]), __high2float(b[k]));
    dst[i] = o;
  }
}

cudaError_t launch_bf16_to_f16(const void* src, void* dst, size_t n, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  if (n % 8 != 0 || ((uintptr_t)src & 15) || ((uintptr_t)dst & 15)) return cudaErrorInvalidValue;
  const size_t n8 = n / 8;
  const int blocks = (int)std::min<size_t>((n8 + 255) / 256, 148 * 16);
  RSD_LAUNCH((bf16_to_f16_kernel), blocks, 256, 0, s, (const uint4*)src, (uint4*)dst, n8);
  return launched(1);
}

cudaError_t launch_rmsnorm(int dtype, float* x, const void* gain, void* out, void* out_lo, int T, int d, float eps,
                           const int32_t* src, const int32_t* n_active, SplitSum pending, cudaStream_t s, bool out_f16) {
  if (T <= 0) return cudaSuccess;
  const int threads = d >= 2048 ? 512 : 256;
  if (dtype == 1 && out_f16)
    RSD_LAUNCH((rmsnorm_kernel<__half, __nv_bfloat16>), T, threads, 0, s, x, (const __nv_bfloat16*)gain, (__half*)out, (__half*)nullptr, d, eps, src, n_active, pending.partials, pending.splits, T);
  else if (dtype == 1)
    RSD_LAUNCH((rmsnorm_kernel<__nv_bfloat16, __nv_bfloat16>), T, threads, 0, s, x, (const __nv_bfloat16*)gain, (__nv_bfloat16*)out, (__nv_bfloat16*)out_lo, d, eps, src, n_active, pending.partials, pending.splits, T);
  else
    RSD_LAUNCH((rmsnorm_kernel<float, float>), T, threads, 0, s, x, (const float*)gain, (float*)out, nullptr, d, eps, src, n_active, pending.partials, pending.splits, T);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Residual update + un-normalised RMSNorm operand (decode path of bf16 models).  One block per (row,
// 256-column chunk): x (+)= sum of the K-split partial sums of the GEMM that feeds the residual stream;
// hi + lo = x * gain (two bf16 arrays, the operand of the next GEMM); ssq[row][chunk] = sum of x^2
// over the chunk.  The next GEMM multiplies its result rows by rsqrt(sum_chunk ssq / d + eps)
// (RowScale), which is RMSNorm applied after the product instead of before it.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(64)
reduce_norm_kernel(const float* __restrict__ partials, int splits, float* __restrict__ x,
                   const __nv_bfloat16* __restrict__ gain, __nv_bfloat16* __restrict__ hi,
                   __nv_bfloat16* __restrict__ lo, float* __restrict__ ssq, int M, int d, int n_chunks,
                   const int32_t* n_active) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(n_active);
  __shared__ float red[2];
  const int m = blockIdx.y, c = blockIdx.x;
  const int col = c * 256 + threadIdx.x * 4;
  float ss = 0.f;
  if (col < d) {
    const size_t o = (size_t)m * d + col;
    float4 v = *reinterpret_cast<const float4*>(x + o);
    if (splits > 1) {
      const size_t stride = (size_t)M * d;
      // twelve loads in flight at a time (tail predicated): each group is one L2 round trip, and 10-24 splits
      // are the rule; the sums stay in split order
      for (int s0 = 0; s0 < splits; s0 += 12) {
        float4 a[12];
#pragma unroll
        for (int u = 0; u < 12; ++u)
          a[u] = s0 + u < splits ? __ldcg(reinterpret_cast<const float4*>(partials + (size_t)(s0 + u) * stride + o))
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 12; ++u) { v.x += a[u].x; v.y += a[u].y; v.z += a[u].z; v.w += a[u].w; }
      }
      *reinterpret_cast<float4*>(x + o) = v;
    }
    ss = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    store_operand<__nv_bfloat16>(hi, lo, o, v.x * to_f32(gain[col]));
    store_operand<__nv_bfloat16>(hi, lo, o + 1, v.y * to_f32(gain[col + 1]));
    store_operand<__nv_bfloat16>(hi, lo, o + 2, v.z * to_f32(gain[col + 2]));
    store_operand<__nv_bfloat16>(hi, lo, o + 3, v.w * to_f32(gain[col + 3]));
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) ssq[(size_t)m * n_chunks + c] = red[0] + red[1];
}

cudaError_t launch_reduce_norm(const float* partials, int splits, float* x, const void* gain, void* hi, void* lo,
                               float* ssq, int M, int d, const int32_t* n_active, cudaStream_t s) {
  if (M <= 0) return cudaSuccess;
  if (d % 4 != 0) return cudaErrorInvalidValue;
  const int n_chunks = norm_chunks(d);
  RSD_LAUNCH((reduce_norm_kernel), dim3(n_chunks, M), 64, 0, s, partials, splits, x, (const __nv_bfloat16*)gain,
             (__nv_bfloat16*)hi, (__nv_bfloat16*)lo, ssq, M, d, n_chunks, n_active);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Split-K SIMT GEMV / skinny GEMM:  y[m, n] (+)= sum_k x[m, k] W[n, k]
// A block of 8 warps covers nb = 8/ks output columns; the ks warps of one column each stream a
// strided share of the row with 16-byte loads and their partial sums meet in shared memory, in a
// fixed order (deterministic).  Rows of x are taken MT at a time.
// ---------------------------------------------------------------------------------------------
template <typename WT, int MT>
__global__ void __launch_bounds__(256)
gemv_splitk_kernel(const WT* __restrict__ W, const WT* __restrict__ X, const WT* __restrict__ X_lo, float* __restrict__ Y,
                   int M, int N, int K, int ks, int accumulate, const int32_t* n_active) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(n_active);
  constexpr int VN = Vec16<WT>::N;
  __shared__ float part[8][MT];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nb = 8 / ks;
  const int col = warp / ks, split = warp % ks;
  const int n = blockIdx.x * nb + col;
  const int m0 = blockIdx.y * MT;
  float acc[MT];
#pragma unroll
  for (int m = 0; m < MT; ++m) acc[m] = 0.f;
  if (n < N) {
    const WT* wrow = W + (size_t)n * K;
    const int nvec = K / VN;
    for (int v = split * 32 + lane; v < nvec; v += ks * 32) {
      Vec16<WT> w;
      w.load_stream(wrow + (size_t)v * VN);
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        if (m0 + m < M) {
          Vec16<WT> xv;
          xv.load(X + (size_t)(m0 + m) * K + (size_t)v * VN);
          if (X_lo != nullptr) {
            Vec16<WT> xl;
            xl.load(X_lo + (size_t)(m0 + m) * K + (size_t)v * VN);
#pragma unroll
            for (int j = 0; j < VN; ++j) xv.v[j] += xl.v[j];
          }
#pragma unroll
          for (int j = 0; j < VN; ++j) acc[m] = fmaf(w.v[j], xv.v[j], acc[m]);
        }
      }
    }
  }
#pragma unroll
  for (int m = 0; m < MT; ++m) acc[m] = warp_sum(acc[m]);
  if (lane == 0) {
#pragma unroll
    for (int m = 0; m < MT; ++m) part[warp][m] = acc[m];
  }
  __syncthreads();
  // one thread per (column, m): add the ks partial sums in split order
  const int idx = threadIdx.x;
  if (idx < nb * MT) {
    const int c = idx / MT, m = idx % MT;
    const int nn = blockIdx.x * nb + c;
    if (nn < N && m0 + m < M) {
      float sum = 0.f;
      for (int sidx = 0; sidx < ks; ++sidx) sum += part[c * ks + sidx][m];
      float* y = Y + (size_t)(m0 + m) * N + nn;
      *y = accumulate ? (*y + sum) : sum;
    }
  }
}

cudaError_t launch_gemm_simt(int dtype, const void* W, const void* x, const void* x_lo, float* y, int M, int N, int K,
                             int accumulate, const int32_t* n_active, cudaStream_t s) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  // pick the split so that the grid covers the 148 SMs a few times over
  int ks = 1;
  while (ks < 8 && (long)N * ks / 8 < 148L * 4 && K / (ks * 2) >= 256) ks *= 2;
  constexpr int MT = 8;
  dim3 grid((N + (8 / ks) - 1) / (8 / ks), (M + MT - 1) / MT);
  if (dtype == 1)
    RSD_LAUNCH((gemv_splitk_kernel<__nv_bfloat16, MT>), grid, 256, 0, s, (const __nv_bfloat16*)W, (const __nv_bfloat16*)x, (const __nv_bfloat16*)x_lo, y, M, N, K, ks, accumulate, n_active);
  else
    RSD_LAUNCH((gemv_splitk_kernel<float, MT>), grid, 256, 0, s, (const float*)W, (const float*)x, nullptr, y, M, N, K, ks, accumulate, n_active);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Rotary table: table[pos, i] = (cos, sin)(pos * theta^(-2i/hd)), evaluated in fp64
// ---------------------------------------------------------------------------------------------
__global__ void rope_table_kernel(float2* table, int n_pos, int half, double theta, double hd) {
  RSD_PDL_SYNC();
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pos * half) return;
  const int pos = idx / half, i = idx % half;
  const double ang = (double)pos * pow(theta, -2.0 * (double)i / hd);
  double sn, cs;
  sincos(ang, &sn, &cs);
  table[idx] = make_float2((float)cs, (float)sn);
}

cudaError_t launch_rope_table(float2* table, int n_pos, int hd, float theta, cudaStream_t s) {
  const int n = n_pos * (hd / 2);
  if (n <= 0) return cudaSuccess;
  RSD_LAUNCH((rope_table_kernel), (n + 255) / 256, 256, 0, s, table, n_pos, hd / 2, (double)theta, (double)hd);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// RoPE on q and k, KV page write.  One block per token slot; threads walk the (head, pair) grid.
// Pair (i, i + hd/2) of a head turns by the angle of (position, i).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float split_sum(const float* __restrict__ direct, const float* __restrict__ partials, int splits,
                                           size_t idx, size_t stride) {
  if (splits <= 1) return direct[idx];
  // loads go out twelve at a time (tail predicated) so their latencies overlap; the sums stay in split order
  float v = 0.f;
  for (int s0 = 0; s0 < splits; s0 += 12) {
    float t[12];
#pragma unroll
    for (int u = 0; u < 12; ++u) t[u] = s0 + u < splits ? __ldcg(partials + (size_t)(s0 + u) * stride + idx) : 0.f;
#pragma unroll
    for (int u = 0; u < 12; ++u) v += t[u];
  }
  return v;
}

template <typename KT>
__global__ void rope_kv_kernel(const float* __restrict__ qkv, const float* __restrict__ partials, int splits,
                               PassView p, float* __restrict__ q_out, KT* pool,
                               const int32_t* __restrict__ page_table, int max_pages,
                               const float2* __restrict__ rope, int H, int KV, int hd, int pf) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(p.n_active);
  const int t = blockIdx.x;
  const int row = p.tok_row[t];
  if (row < 0) return;
  const int pos = p.tok_pos[t];
  const int half = hd / 2;
  const int width = (H + 2 * KV) * hd;
  const size_t src0 = (size_t)t * width;                 // offset of this token's row in qkv / a partial
  const size_t sstride = (size_t)gridDim.x * width;      // one partial array = [T][width]
  const float2* cs = rope + (size_t)pos * half;
  const int page = page_table[(size_t)row * max_pages + pos / kPageTokens];
  const int slot = pos % kPageTokens;
  // page = K block [KV][16][hd] followed by V block [KV][hd][16] (V transposed within the page)
  // (pf = 4: two more blocks hold the low halves of the keys and of the values)
  const size_t block = (size_t)KV * kPageTokens * hd;
  KT* kbase = pool + (size_t)page * pf * block;
  KT* vbase = kbase + block;
  // one block per (token, head): query and key heads are rotated, value heads copied
  const int head = blockIdx.y;
  if (head < H + KV) {
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
      const float a = split_sum(qkv, partials, splits, src0 + head * hd + i, sstride);
      const float b = split_sum(qkv, partials, splits, src0 + head * hd + i + half, sstride);
      const float2 c = cs[i];
      const float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
      if (head < H) {
        q_out[(size_t)t * H * hd + head * hd + i] = ra;
        q_out[(size_t)t * H * hd + head * hd + i + half] = rb;
      } else {
        KT* k = kbase + ((size_t)(head - H) * kPageTokens + slot) * hd;
        const KT ka = from_f32<KT>(ra), kb2 = from_f32<KT>(rb);
        k[i] = ka;
        k[i + half] = kb2;
        if (pf == 4) {
          k[2 * block + i] = from_f32<KT>(ra - to_f32(ka));
          k[2 * block + i + half] = from_f32<KT>(rb - to_f32(kb2));
        }
      }
    }
  } else {
    const int vh_idx = head - H - KV;
    for (int i = threadIdx.x; i < hd; i += blockDim.x) {
      const float v = split_sum(qkv, partials, splits, src0 + (size_t)head * hd + i, sstride);
      const KT vh = from_f32<KT>(v);
      vbase[((size_t)vh_idx * hd + i) * kPageTokens + slot] = vh;
      if (pf == 4) vbase[2 * block + ((size_t)vh_idx * hd + i) * kPageTokens + slot] = from_f32<KT>(v - to_f32(vh));
    }
  }
}

// The same for the long passes (prefill, scoring, sync, catch-up: thousands of tokens, no K-split sums): a block takes
// kRopeTokens consecutive list entries.  Their rows, positions and pages are looked up once into shared memory, so the
// data loads of all entries go out together instead of after a chain of three dependent loads per (token, head)
// block; and when the entries are consecutive positions of one row inside one page (the rule in a long pass), a thread
// writes the eight transposed value elements of a (head, dim) as ONE 16-byte store instead of eight 2-byte ones.
constexpr int kRopeTokens = 8;

template <typename KT>
__global__ void __launch_bounds__(256)
rope_kv_long_kernel(const float* __restrict__ qkv, PassView p, float* __restrict__ q_out, KT* pool,
                    const int32_t* __restrict__ page_table, int max_pages, const float2* __restrict__ rope, int H, int KV,
                    int hd, int pf) {
  RSD_PDL_SYNC();
  __shared__ int s_row[kRopeTokens], s_pos[kRopeTokens], s_page[kRopeTokens];
  __shared__ int s_run;            // 1: the entries are eight consecutive positions of one row within one page
  const int t0 = blockIdx.x * kRopeTokens;
  const int n_tok = min(kRopeTokens, p.T - t0);
  if (threadIdx.x < kRopeTokens) {
    const int i = threadIdx.x;
    int row = -1, pos = 0, page = 0;
    if (i < n_tok) {
      row = p.tok_row[t0 + i];
      pos = p.tok_pos[t0 + i];
      if (row >= 0) page = page_table[(size_t)row * max_pages + pos / kPageTokens];
    }
    s_row[i] = row; s_pos[i] = pos; s_page[i] = page;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = n_tok == kRopeTokens && s_row[0] >= 0 && (s_pos[0] % kRopeTokens) == 0;
    for (int i = 1; i < kRopeTokens && run; ++i) run = s_row[i] == s_row[0] && s_pos[i] == s_pos[0] + i;
    s_run = run;
  }
  __syncthreads();
  const int half = hd / 2;
  const int width = (H + 2 * KV) * hd;
  const size_t block = (size_t)KV * kPageTokens * hd;
  const int n_rot = (H + KV) * half;            // rotated pairs of one token
  // queries and keys: one (token, head, pair) per step
  for (int idx = threadIdx.x; idx < n_tok * n_rot; idx += blockDim.x) {
    const int tk = idx / n_rot, e = idx % n_rot;
    if (s_row[tk] < 0) continue;
    const int head = e / half, i = e % half;
    const int t = t0 + tk, pos = s_pos[tk];
    const float a = qkv[(size_t)t * width + head * hd + i], b = qkv[(size_t)t * width + head * hd + i + half];
    const float2 c = rope[(size_t)pos * half + i];
    const float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
    if (head < H) {
      q_out[(size_t)t * H * hd + head * hd + i] = ra;
      q_out[(size_t)t * H * hd + head * hd + i + half] = rb;
    } else {
      KT* k = pool + (size_t)s_page[tk] * pf * block + ((size_t)(head - H) * kPageTokens + pos % kPageTokens) * hd;
      const KT ka = from_f32<KT>(ra), kb2 = from_f32<KT>(rb);
      k[i] = ka;
      k[i + half] = kb2;
      if (pf == 4) {
        k[2 * block + i] = from_f32<KT>(ra - to_f32(ka));
        k[2 * block + i + half] = from_f32<KT>(rb - to_f32(kb2));
      }
    }
  }
  // values, transposed inside the page: [KV][hd][16 tokens]
  if (s_run && sizeof(KT) == 2) {
    const int slot0 = s_pos[0] % kPageTokens;                     // 0 or 8: the 16-byte store is aligned
    KT* vbase = pool + (size_t)s_page[0] * pf * block + block;
    for (int e = threadIdx.x; e < KV * hd; e += blockDim.x) {
      __align__(16) KT hi8[kRopeTokens];
      __align__(16) KT lo8[kRopeTokens];
#pragma unroll
      for (int tk = 0; tk < kRopeTokens; ++tk) {
        const float v = qkv[(size_t)(t0 + tk) * width + (size_t)(H + KV) * hd + e];
        hi8[tk] = from_f32<KT>(v);
        lo8[tk] = from_f32<KT>(v - to_f32(hi8[tk]));
      }
      *reinterpret_cast<uint4*>(vbase + (size_t)e * kPageTokens + slot0) = *reinterpret_cast<const uint4*>(hi8);
      if (pf == 4) *reinterpret_cast<uint4*>(vbase + 2 * block + (size_t)e * kPageTokens + slot0) = *reinterpret_cast<const uint4*>(lo8);
    }
  } else {
    for (int idx = threadIdx.x; idx < n_tok * KV * hd; idx += blockDim.x) {
      const int tk = idx / (KV * hd), e = idx % (KV * hd);
      if (s_row[tk] < 0) continue;
      const float v = qkv[(size_t)(t0 + tk) * width + (size_t)(H + KV) * hd + e];
      KT* vbase = pool + (size_t)s_page[tk] * pf * block + block;
      const int slot = s_pos[tk] % kPageTokens;
      const KT vh = from_f32<KT>(v);
      vbase[(size_t)e * kPageTokens + slot] = vh;
      if (pf == 4) vbase[2 * block + (size_t)e * kPageTokens + slot] = from_f32<KT>(v - to_f32(vh));
    }
  }
}

cudaError_t launch_rope_kv(int kv_dtype, const float* qkv, SplitSum pending, PassView p, float* q_out, KvView kv,
                           const float2* rope, int H, int KV, int hd, cudaStream_t s) {
  if (p.T <= 0) return cudaSuccess;
  const int pf = 2 + 2 * kv.v_extra;
  if (pending.splits <= 1 && p.n_active == nullptr && p.T >= 64) {
    // long pass: eight list entries per block
    const int blocks = (p.T + kRopeTokens - 1) / kRopeTokens;
    if (kv_dtype == 2 || kv_dtype == 3)
      RSD_LAUNCH((rope_kv_long_kernel<__half>), blocks, 256, 0, s, qkv, p, q_out, (__half*)kv.pool_layer, kv.page_table, kv.max_pages, rope, H, KV, hd, pf);
    else if (kv_dtype == 1)
      RSD_LAUNCH((rope_kv_long_kernel<__nv_bfloat16>), blocks, 256, 0, s, qkv, p, q_out, (__nv_bfloat16*)kv.pool_layer, kv.page_table, kv.max_pages, rope, H, KV, hd, pf);
    else
      RSD_LAUNCH((rope_kv_long_kernel<float>), blocks, 256, 0, s, qkv, p, q_out, (float*)kv.pool_layer, kv.page_table, kv.max_pages, rope, H, KV, hd, pf);
    return launched(1);
  }
  if (kv_dtype == 2 || kv_dtype == 3)
    RSD_LAUNCH((rope_kv_kernel<__half>), dim3(p.T, H + 2 * KV), 64, 0, s, qkv, pending.partials, pending.splits, p, q_out, (__half*)kv.pool_layer, kv.page_table, kv.max_pages, rope, H, KV, hd, pf);
  else if (kv_dtype == 1)
    RSD_LAUNCH((rope_kv_kernel<__nv_bfloat16>), dim3(p.T, H + 2 * KV), 64, 0, s, qkv, pending.partials, pending.splits, p, q_out, (__nv_bfloat16*)kv.pool_layer, kv.page_table, kv.max_pages, rope, H, KV, hd, pf);
  else
    RSD_LAUNCH((rope_kv_kernel<float>), dim3(p.T, H + 2 * KV), 64, 0, s, qkv, pending.partials, pending.splits, p, q_out, (float*)kv.pool_layer, kv.page_table, kv.max_pages, rope, H, KV, hd, pf);
  return launched(1);
}

// Stand-alone rotary kernel on [T, n_heads, hd] fp32 (angles in fp64).
__global__ void rope_only_kernel(float* v, const int32_t* pos, int n_heads, int hd, double theta) {
  RSD_PDL_SYNC();
  const int t = blockIdx.x, half = hd / 2;
  const int p = pos[t];
  for (int idx = threadIdx.x; idx < n_heads * half; idx += blockDim.x) {
    const int head = idx / half, i = idx % half;
    double sn, cs;
    sincos((double)p * pow(theta, -2.0 * (double)i / (double)hd), &sn, &cs);
    float* h = v + ((size_t)t * n_heads + head) * hd;
    const float a = h[i], b = h[i + half];
    h[i] = a * (float)cs - b * (float)sn;
    h[i + half] = b * (float)cs + a * (float)sn;
  }
}

cudaError_t launch_rope_only(float* v, const int32_t* pos, int T, int n_heads, int hd, float theta, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  RSD_LAUNCH((rope_only_kernel), T, 128, 0, s, v, pos, n_heads, hd, (double)theta);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Generic causal attention over paged KV: one warp per (slot, query head), online softmax.
// Each lane owns hd/32 consecutive dims; query head j reads KV head j / (H / KV).
// ---------------------------------------------------------------------------------------------
template <typename KT, typename OT, int HD>
__global__ void __launch_bounds__(128)
attn_generic_kernel(const float* __restrict__ q, PassView p, const KT* __restrict__ pool,
                    const int32_t* __restrict__ page_table, int max_pages, OT* __restrict__ out, OT* __restrict__ out_lo,
                    int H, int KV, int pf) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(p.n_active);
  constexpr int DPL = HD / 32;
  const int lane = threadIdx.x & 31;
  const int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (w >= p.T * H) return;
  const int t = w / H, h = w % H;
  const int row = p.tok_row[t];
  if (row < 0) return;
  const int pos = p.tok_pos[t];
  const int g = h / (H / KV);
  const float scale = rsqrtf((float)HD);
  float qv[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) qv[i] = q[((size_t)t * H + h) * HD + lane * DPL + i] * scale;
  float m = -INFINITY, l = 0.f, acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  const int32_t* pt = page_table + (size_t)row * max_pages;
  for (int p0 = 0; p0 <= pos; p0 += kPageTokens) {
    const int page = pt[p0 / kPageTokens];
    const size_t block = (size_t)KV * kPageTokens * HD;
    const KT* kb = pool + (size_t)page * pf * block + (size_t)g * kPageTokens * HD;
    const KT* vb = kb + block;
    const int n = min(kPageTokens, pos + 1 - p0);
    float sc[kPageTokens];
#pragma unroll
    for (int j = 0; j < kPageTokens; ++j) {
      float a = 0.f;
      if (j < n) {
#pragma unroll
        for (int i = 0; i < DPL; ++i) {
          float kk = to_f32(kb[j * HD + lane * DPL + i]);
          if (pf == 4) kk += to_f32(kb[2 * block + j * HD + lane * DPL + i]);
          a = fmaf(qv[i], kk, a);
        }
      }
      sc[j] = a;
    }
#pragma unroll
    for (int j = 0; j < kPageTokens; ++j) sc[j] = warp_sum(sc[j]);
    float mx = m;
#pragma unroll
    for (int j = 0; j < kPageTokens; ++j)
      if (j < n) mx = fmaxf(mx, sc[j]);
    const float corr = __expf(m - mx);
    l *= corr;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] *= corr;
#pragma unroll
    for (int j = 0; j < kPageTokens; ++j) {
      if (j < n) {
        const float pj = __expf(sc[j] - mx);
        l += pj;
#pragma unroll
        for (int i = 0; i < DPL; ++i) {
          float vv = to_f32(vb[(lane * DPL + i) * kPageTokens + j]);
          if (pf == 4) vv += to_f32(vb[2 * block + (lane * DPL + i) * kPageTokens + j]);
          acc[i] = fmaf(pj, vv, acc[i]);
        }
      }
    }
    m = mx;
  }
  const float inv = 1.f / l;
#pragma unroll
  for (int i = 0; i < DPL; ++i) store_operand<OT>(out, out_lo, ((size_t)t * H + h) * HD + lane * DPL + i, acc[i] * inv);
}

cudaError_t launch_attn_generic(int kv_dtype, const float* q, PassView p, KvView kv, void* out, void* out_lo,
                                int out_dtype, int H, int KV, int hd, cudaStream_t s) {
  if (p.T <= 0) return cudaSuccess;
  const int warps = p.T * H;
  const int blocks = (warps + 3) / 4;
#define RSD_ATTN(KT, OT, HD) \
  RSD_LAUNCH((attn_generic_kernel<KT, OT, HD>), blocks, 128, 0, s, q, p, (const KT*)kv.pool_layer, kv.page_table, kv.max_pages, (OT*)out, (OT*)out_lo, H, KV, 2 + 2 * kv.v_extra)
#define RSD_ATTN_HD(KT, OT) do { if (hd == 128) RSD_ATTN(KT, OT, 128); else RSD_ATTN(KT, OT, 64); } while (0)
  using bf = __nv_bfloat16;
  if (kv_dtype == 2) { if (out_dtype == 1) RSD_ATTN_HD(__half, bf); else RSD_ATTN_HD(__half, float); }
  else if (kv_dtype == 1) { if (out_dtype == 1) RSD_ATTN_HD(bf, bf); else RSD_ATTN_HD(bf, float); }
  else RSD_ATTN_HD(float, float);
#undef RSD_ATTN_HD
#undef RSD_ATTN
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// SwiGLU: out[t, f] = silu(gu[t, f]) * gu[t, F + f]
// ---------------------------------------------------------------------------------------------
template <typename OT>
__global__ void swiglu_kernel(const float* __restrict__ gu, const float* __restrict__ partials, int splits,
                              OT* __restrict__ out, OT* __restrict__ out_lo, int T, int F, const int32_t* n_active) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(n_active);
  const size_t n = (size_t)T * F;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const size_t t = i / F, f = i % F;
    const size_t sstride = (size_t)T * 2 * F;
    const float a = split_sum(gu, partials, splits, t * 2 * F + f, sstride);
    const float b = split_sum(gu, partials, splits, t * 2 * F + F + f, sstride);
    store_operand<OT>(out, out_lo, i, a / (1.f + expf(-a)) * b);
  }
}

cudaError_t launch_swiglu(int dtype, const float* gu, SplitSum pending, void* out, void* out_lo, int T, int F,
                          const int32_t* n_active, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  const size_t n = (size_t)T * F;
  int blocks = (int)((n + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (dtype == 1) RSD_LAUNCH((swiglu_kernel<__nv_bfloat16>), blocks, 256, 0, s, gu, pending.partials, pending.splits, (__nv_bfloat16*)out, (__nv_bfloat16*)out_lo, T, F, n_active);
  else RSD_LAUNCH((swiglu_kernel<float>), blocks, 256, 0, s, gu, pending.partials, pending.splits, (float*)out, nullptr, T, F, n_active);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Sampling: greedy argmax, or Gumbel-max with Philox noise keyed by (seed; vocab id / 4, position
// of the generated token, row, model id).  One block per slot; ties go to the lowest id.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void better(float& bs, int& bi, float s, int i) {
  if (s > bs || (s == bs && i < bi)) { bs = s; bi = i; }
}

// (score, id) packed so that an unsigned 64-bit maximum picks the highest score and, among equal
// scores, the lowest id: high word = order-preserving image of the float, low word = ~id.
__device__ __forceinline__ unsigned long long pack_best(float sc, int id) {
  const uint32_t b = __float_as_uint(sc);
  const uint32_t key = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return ((unsigned long long)key << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
}

// Grid (slots, chunks): every block scans one chunk of the vocabulary and folds its best candidate
// into best[slot] with an atomic maximum (order-independent, hence deterministic).
__global__ void __launch_bounds__(1024) sample_kernel(SampleArgs a) {
  RSD_PDL_SYNC();
  RSD_SKIP_IF_IDLE(a.n_active);
  __shared__ float s_sc[32];
  __shared__ int s_ix[32];
  const int slot = blockIdx.x;
  const int row = a.slot_row[slot];
  if (row < 0) return;
  const float* lg = a.logits + (size_t)slot * a.V;
  const uint32_t position = (uint32_t)(a.slot_pos[slot] + 1);
  const uint2 key = make_uint2((uint32_t)(a.seed & 0xFFFFFFFFull), (uint32_t)(a.seed >> 32));
  const float inv_t = a.temperature > 0.f ? 1.f / a.temperature : 1.f;
  float bs = -INFINITY;
  int bi = 0x7FFFFFFF;
  const int n_v4 = (a.v_limit + 3) / 4;
  const int per_chunk = (n_v4 + gridDim.y - 1) / gridDim.y;
  const int v4_end = min(n_v4, (int)(blockIdx.y + 1) * per_chunk);
  for (int v4 = blockIdx.y * per_chunk + threadIdx.x; v4 < v4_end; v4 += blockDim.x) {
    float g[4] = {0.f, 0.f, 0.f, 0.f};
    if (a.temperature > 0.f) {
      const uint4 r = philox4x32_10(make_uint4((uint32_t)v4, position, (uint32_t)row, (uint32_t)a.model_id), key);
      const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) g[j] = -logf(-logf(uniform_from_bits(w[j])));
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int v = v4 * 4 + j;
      if (v < a.v_limit) better(bs, bi, lg[v] * inv_t + g[j], v);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float os = __shfl_xor_sync(0xFFFFFFFFu, bs, o);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
    better(bs, bi, os, oi);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { s_sc[warp] = bs; s_ix[warp] = bi; }
  __syncthreads();
  if (warp == 0) {
    const int nw = blockDim.x >> 5;
    bs = lane < nw ? s_sc[lane] : -INFINITY;
    bi = lane < nw ? s_ix[lane] : 0x7FFFFFFF;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float os = __shfl_xor_sync(0xFFFFFFFFu, bs, o);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
      better(bs, bi, os, oi);
    }
    if (lane == 0 && bi != 0x7FFFFFFF) atomicMax(a.best + slot, pack_best(bs, bi));
  }
}

// token[slot] = id held in best[slot]; best is cleared for the next use.
__global__ void sample_finalize_kernel(unsigned long long* best, const int32_t* slot_row, int32_t* token, int n) {
  RSD_PDL_SYNC();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  if (slot_row[i] >= 0) token[i] = (int32_t)(0xFFFFFFFFu - (uint32_t)(best[i] & 0xFFFFFFFFull));
  best[i] = 0ull;
}

int sample_chunks(int v_limit) { return v_limit >= 65536 ? 16 : (v_limit >= 8192 ? 4 : 1); }

// Leaves the winners packed in a.best (which must be zero on entry); when a.token is given a second
// kernel unpacks them into a.token and clears a.best.
cudaError_t launch_sample(const SampleArgs& a, cudaStream_t s) {
  if (a.n_slots <= 0) return cudaSuccess;
  const int threads = a.v_limit >= 16384 ? 1024 : 256;
  RSD_LAUNCH((sample_kernel), dim3(a.n_slots, sample_chunks(a.v_limit)), threads, 0, s, a);
  if (a.token == nullptr) return launched(1);
  RSD_LAUNCH((sample_finalize_kernel), (a.n_slots + 255) / 256, 256, 0, s, a.best, a.slot_row, a.token, a.n_slots);
  return launched(2);
}

__global__ void philox_kernel(const uint32_t* ctr, const uint32_t* key, uint32_t* out, int n) {
  RSD_PDL_SYNC();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint4 r = philox4x32_10(make_uint4(ctr[4 * i], ctr[4 * i + 1], ctr[4 * i + 2], ctr[4 * i + 3]),
                                make_uint2(key[0], key[1]));
  out[4 * i] = r.x; out[4 * i + 1] = r.y; out[4 * i + 2] = r.z; out[4 * i + 3] = r.w;
}

cudaError_t launch_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out, int n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  RSD_LAUNCH((philox_kernel), (n + 255) / 256, 256, 0, s, ctr, key, out, n);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// PRM step scoring head: gathers the hidden state of each row's last step token, applies the final
// RMSNorm, projects to a scalar and squashes it (Appendix B.3; score in [0,1], Section 3 "Models").
// ---------------------------------------------------------------------------------------------
template <typename WT>
__global__ void reward_kernel(const float* __restrict__ x, const WT* __restrict__ final_norm, const WT* __restrict__ w_r,
                              int head_kind, const int32_t* __restrict__ last_idx, int t0, int T, int d, float eps,
                              float* __restrict__ reward) {
  RSD_PDL_SYNC();
  __shared__ float red[33];
  const int row = blockIdx.x;
  const int idx = last_idx[row];
  if (idx < t0 || idx >= t0 + T) return;
  const float* xr = x + (size_t)(idx - t0) * d;
  float ss = 0.f, dot = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = xr[i];
    ss += v * v;
    dot += v * to_f32(final_norm[i]) * to_f32(w_r[i]);
  }
  ss = block_sum(ss, red);
  dot = block_sum(dot, red);
  if (threadIdx.x == 0) {
    const float a = dot * rsqrtf(ss / (float)d + eps);
    reward[row] = head_kind == 2 ? a : 1.f / (1.f + expf(-a));
  }
}

cudaError_t launch_reward(int dtype, const float* x, const void* final_norm, const void* w_r, int head_kind,
                          const int32_t* last_idx, int t0, int T, int d, float eps, float* reward, int n_rows,
                          cudaStream_t s) {
  if (n_rows <= 0) return cudaSuccess;
  if (dtype == 1)
    RSD_LAUNCH((reward_kernel<__nv_bfloat16>), n_rows, 256, 0, s, x, (const __nv_bfloat16*)final_norm, (const __nv_bfloat16*)w_r, head_kind, last_idx, t0, T, d, eps, reward);
  else
    RSD_LAUNCH((reward_kernel<float>), n_rows, 256, 0, s, x, (const float*)final_norm, (const float*)w_r, head_kind, last_idx, t0, T, d, eps, reward);
  return launched(1);
}

}  // namespace rsd
