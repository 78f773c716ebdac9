// Integer side of the RSD step loop (Algorithm 1 batched over rows): page reservation, ragged pass
// lists, decode-phase control, the threshold gate with warp-ballot compaction of rejected rows,
// and the commit of y_i.  All state lives on the device; every kernel here runs as ONE block of
// 1024 threads (thread b <-> row b, rows <= 1024), which keeps the ascending-row order of page
// hand-out and of the rejected-row list deterministic.
#include "common.cuh"
#include "kernels.cuh"

namespace rsd {

// ---------------------------------------------------------------------------------------------
// Page reservation.  Row b needs capacity for `need` cached positions; missing pages are taken
// from a bump counter, rows served in ascending order, each row's new pages consecutive.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) reserve_pages_kernel(RowState st, int which, int mode, int min_target_rows) {
  RSD_PDL_SYNC();
  __shared__ int scan[33];
  const int b = threadIdx.x;
  int need = 0;
  if (b < st.B) {
    const int z = st.z_len[b];
    const bool live = st.live[b] != 0;
    const bool runs = live && !st.waiting[b];     // takes a draft step in this call
    switch (mode) {
      case kReservePrefillDraft: need = live ? z - 1 : 0; break;
      case kReservePrefillPrm: need = live ? z : 0; break;
      case kReserveStepDraft: need = runs ? z - 1 + st.C + st.prm_shared : 0; break;   // merged PRM: + the step's last token
      case kReserveScorePrm: need = runs ? z + st.gen_len[0][b] : 0; break;
      case kReserveTarget:
        need = (live && st.waiting[b] && target_pass_due(st.n_rej[0], st.n_live[0], min_target_rows)) ? z - 1 + st.C : 0;
        break;
    }
  }
  const int have = b < st.B ? st.n_pages[which][b] : 0;
  int more = (need + kPageTokens - 1) / kPageTokens - have;
  if (more < 0) more = 0;
  int total;
  const int off = block_exclusive_scan(more, scan, &total);
  const int base = st.next_page[which];
  if (base + total > st.pool_pages[which] || (b < st.B && have + more > st.max_pages)) {
    st.err[0] = -3;  // pool exhausted: leave the tables untouched
  }
  __syncthreads();
  if (st.err[0] != 0) return;
  if (b < st.B) {
    for (int i = 0; i < more; ++i) st.page_table[which][(size_t)b * st.max_pages + have + i] = base + off + i;
    st.n_pages[which][b] = have + more;
  }
  __syncthreads();
  if (b == 0) st.next_page[which] = base + total;
}

cudaError_t launch_reserve_pages(const RowState& st, int which, ReserveMode mode, int min_target_rows, cudaStream_t s) {
  RSD_LAUNCH((reserve_pages_kernel), 1, 1024, 0, s, st, which, (int)mode, min_target_rows);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Ragged pass list: for every participating row the positions [kv_len, end) not yet cached by model
// `which`, flattened in (row, position) order.  Advances kv_len to `end`.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) build_pass_kernel(RowState st, int which, int mode, int min_target_rows) {
  RSD_PDL_SYNC();
  __shared__ int scan[33];
  __shared__ int s_off[kMaxBatch + 1];
  __shared__ int s_start[kMaxBatch];
  const int b = threadIdx.x;
  int start = 0, cnt = 0;
  if (b < st.B) {
    const int z = st.z_len[b];
    const bool live = st.live[b] != 0;
    const bool runs = live && !st.waiting[b];
    start = st.kv_len[which][b];
    int end = start;
    switch (mode) {
      case kPassIngestDraft: end = runs ? z - 1 : start; break;
      case kPassScorePrm: end = runs ? z + st.gen_len[0][b] : start; break;
      case kPassCatchupTarget:
        end = (live && st.waiting[b] && target_pass_due(st.n_rej[0], st.n_live[0], min_target_rows)) ? z - 1 : start;
        break;
    }
    cnt = max(0, end - start);
  }
  int total;
  const int off = block_exclusive_scan(cnt, scan, &total);
  if (b < kMaxBatch) { s_off[b] = off; s_start[b] = start; }
  if (total > st.pass_capacity) {
    // the list does not fit: raise the error and leave cursors and the list as they were
    if (b == 0) { st.n_tok[0] = 0; st.err[0] = -3; }
    return;
  }
  if (b == 0) {
    s_off[kMaxBatch] = total;
    st.n_tok[0] = total;
  }
  if (b < st.B) {
    st.last_idx[b] = cnt > 0 ? off + cnt - 1 : -1;
    st.kv_len[which][b] = start + cnt;
    if (mode == kPassScorePrm) {
      // the pass also caches a step the target wrote last time: its last token is the row's last committed one
      const int z = st.z_len[b];
      st.prev_idx[b] = (cnt > 0 && start < z) ? off + (z - 1 - start) : -1;
    }
  }
  __syncthreads();
  for (int t = threadIdx.x; t < total; t += blockDim.x) {
    // largest row with s_off[row] <= t (rows with no tokens share an offset with their successor)
    int lo = 0, hi = st.B - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (s_off[mid] <= t) lo = mid; else hi = mid - 1;
    }
    const int pos = s_start[lo] + (t - s_off[lo]);
    st.pass_tok_row[t] = lo;
    st.pass_tok_pos[t] = pos;
    st.pass_tok_id[t] = st.tok[(size_t)lo * st.S + pos];
  }
}

cudaError_t launch_build_pass(const RowState& st, int which, PassMode mode, int min_target_rows, cudaStream_t s) {
  RSD_LAUNCH((build_pass_kernel), 1, 1024, 0, s, st, which, (int)mode, min_target_rows);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Decode-phase control.  Phase 0: the draft writes y^_i for every live row that is not waiting for
// the target (slot b = row b).  Phase 1: the target writes y_i for the waiting rows (slot i = rej_idx[i]).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) decode_begin_kernel(RowState st, int phase) {
  RSD_PDL_SYNC();
  __shared__ int scan[33];
  const int b = threadIdx.x;
  int part = 0;
  if (b < st.B) {
    part = st.live[b] != 0 && (phase == 0 ? st.waiting[b] == 0 : st.waiting[b] != 0);
    st.gen_active[b] = part;
    st.gen_len[phase][b] = 0;
  }
  int total;
  block_exclusive_scan(part, scan, &total);
  if (b == 0) { st.n_active[0] = total; st.iter[0] = 0; st.sd_stats[3] = 0; st.sd_stats[4] = 0; }
  const int n_slots = phase == 0 ? st.B : st.n_rej[0];
  if (b == 0) st.n_slots[0] = n_slots;
  if (b < st.B) st.slot_row[b] = phase == 0 ? b : (b < n_slots ? st.rej_idx[b] : -1);
  for (int i = threadIdx.x; i < st.B * st.C; i += blockDim.x) {
    st.gen_tok[phase][i] = 0;
    st.sampled[phase][i] = 0;
  }
}

cudaError_t launch_decode_begin(const RowState& st, int phase, cudaStream_t s) {
  RSD_LAUNCH((decode_begin_kernel), 1, 1024, 0, s, st, phase);
  return launched(1);
}

__global__ void __launch_bounds__(1024) score_prepare_kernel(RowState st) {
  RSD_PDL_SYNC();
  const int b = threadIdx.x;
  int part = 0;
  if (b < st.B) {
    const int n = st.gen_len[0][b];
    part = st.live[b] != 0 && st.waiting[b] == 0 && n > 0;
    if (part) {
      st.pass_tok_id[b] = st.gen_tok[0][(size_t)b * st.C + n - 1];
      st.pass_tok_pos[b] = st.kv_len[0][b];     // position of the step's last token; the cursor does not move
      st.pass_tok_row[b] = b;
      st.last_idx[b] = b;
    } else {
      st.pass_tok_row[b] = -1;
      st.last_idx[b] = -1;
    }
  }
  const int total = __syncthreads_count(part);
  if (b == 0) st.n_active[0] = total;
}

cudaError_t launch_score_prepare(const RowState& st, cudaStream_t s) {
  RSD_LAUNCH((score_prepare_kernel), 1, 1024, 0, s, st);
  return launched(1);
}

__global__ void __launch_bounds__(1024) decode_prepare_kernel(RowState st, int which, int n_slots) {
  RSD_PDL_SYNC();
  if (st.n_active[0] == 0) return;
  const int i = threadIdx.x;
  if (i >= n_slots) return;
  const int row = st.slot_row[i];
  if (row >= 0 && st.gen_active[row]) {
    const int pos = st.kv_len[which][row];
    st.pass_tok_id[i] = st.tok[(size_t)row * st.S + pos];
    st.pass_tok_pos[i] = pos;
    st.pass_tok_row[i] = row;
  } else {
    st.pass_tok_row[i] = -1;
  }
}

cudaError_t launch_decode_prepare(const RowState& st, int which, int n_slots, cudaStream_t s) {
  if (n_slots <= 0) return cudaSuccess;
  RSD_LAUNCH((decode_prepare_kernel), 1, 1024, 0, s, st, which, n_slots);
  return launched(1);
}

__device__ __forceinline__ bool ends_step(int t, const LoopParams& lp) {
  if (lp.eos_id >= 0 && t == lp.eos_id) return true;
  if (lp.step_end_mod > 0) return (t % lp.step_end_mod) == (lp.step_end_id % lp.step_end_mod);
  return t == lp.step_end_id;
}

// Appends the current iteration's token of every active slot to its row and stops rows whose step ended.
__global__ void __launch_bounds__(1024)
decode_update_kernel(RowState st, int which, int phase, unsigned long long* best, int n_slots, LoopParams lp) {
  RSD_PDL_SYNC();
  if (st.n_active[0] == 0) return;
  const int iter = st.iter[0];   // iteration of the current decode phase, kept on the device
  const int i = threadIdx.x;
  int ended = 0;
  if (i < n_slots) {
    const int row = st.pass_tok_row[i];
    const unsigned long long packed = best[i];
    best[i] = 0ull;
    if (row >= 0) {
      // packed == 0: no candidate was comparable (all scores NaN); fall back to id 0
      int t = packed ? (int)(0xFFFFFFFFu - (uint32_t)(packed & 0xFFFFFFFFull)) : 0;
      st.sampled[phase][(size_t)row * st.C + iter] = t;
      const int flen = st.forced_len[phase][row];
      if (flen > 0) t = st.forced_tok[phase][(size_t)row * st.C + iter];
      const int pos = st.pass_tok_pos[i];
      st.tok[(size_t)row * st.S + pos + 1] = t;
      st.gen_tok[phase][(size_t)row * st.C + iter] = t;
      st.kv_len[which][row] = pos + 1;
      st.gen_len[phase][row] = iter + 1;
      if (ends_step(t, lp) || iter + 1 == st.C || (flen > 0 && iter + 1 == flen)) {
        st.gen_active[row] = 0;
        ended = 1;
      }
    }
  }
  const int n_ended = __syncthreads_count(ended);
  if (threadIdx.x == 0) {
    st.n_active[0] -= n_ended;
    st.iter[0] = iter + 1;
  }
}

cudaError_t launch_decode_update(const RowState& st, int which, int phase, unsigned long long* best,
                                 int n_slots, const LoopParams& lp, cudaStream_t s) {
  if (n_slots <= 0) return cudaSuccess;
  RSD_LAUNCH((decode_update_kernel), 1, 1024, 0, s, st, which, phase, best, n_slots, lp);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Speculative decoding of rejected steps (the paper's discussion of combining RSD with speculative decoding:
// a rejected step is regenerated by draft + target).  Slot i serves row slot_row[i]; gen_len[1][row] tokens
// of the row's step are written so far; the row's last written token sits at the cursor of both caches.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int sd_round_tokens(const RowState& st, int row) {
  // proposals (and evaluated positions) of the running round for this row: up to sd_k, not beyond the step cap
  return min(st.sd_k, st.C - st.gen_len[1][row]);
}

__global__ void __launch_bounds__(1024) sd_propose_prepare_kernel(RowState st, int n_slots) {
  RSD_PDL_SYNC();
  if (st.n_active[0] == 0) return;
  const int j = st.sd_stats[4];   // proposal index within the round, kept on the device so one graph serves every j
  const int i = threadIdx.x;
  if (i >= n_slots) return;
  const int row = st.slot_row[i];
  if (row >= 0 && st.gen_active[row] && j < sd_round_tokens(st, row)) {
    const int pos = st.kv_len[0][row];
    st.pass_tok_id[i] = st.tok[(size_t)row * st.S + pos];
    st.pass_tok_pos[i] = pos;
    st.pass_tok_row[i] = row;
  } else {
    st.pass_tok_row[i] = -1;
  }
}

cudaError_t launch_sd_propose_prepare(const RowState& st, int n_slots, cudaStream_t s) {
  if (n_slots <= 0) return cudaSuccess;
  RSD_LAUNCH((sd_propose_prepare_kernel), 1, 1024, 0, s, st, n_slots);
  return launched(1);
}

__global__ void __launch_bounds__(1024)
sd_propose_update_kernel(RowState st, unsigned long long* best, int n_slots) {
  RSD_PDL_SYNC();
  if (st.n_active[0] == 0) return;
  const int j = st.sd_stats[4];
  const int i = threadIdx.x;
  __syncthreads();                              // every thread has read j
  if (i == 0) st.sd_stats[4] = j + 1;
  if (i >= n_slots) return;
  const int row = st.pass_tok_row[i];
  const unsigned long long packed = best[i];
  best[i] = 0ull;
  if (row < 0) return;
  int t = packed ? (int)(0xFFFFFFFFu - (uint32_t)(packed & 0xFFFFFFFFull)) : 0;
  if (st.sd_forced_props != nullptr && st.sd_forced_on[row])
    t = st.sd_forced_props[((size_t)row * st.C + st.sd_stats[3]) * st.sd_k + j];
  const int pos = st.pass_tok_pos[i];
  st.tok[(size_t)row * st.S + pos + 1] = t;     // proposal j of the round; the target's choice replaces it later
  st.kv_len[0][row] = pos + 1;
}

cudaError_t launch_sd_propose_update(const RowState& st, unsigned long long* best, int n_slots, cudaStream_t s) {
  if (n_slots <= 0) return cudaSuccess;
  RSD_LAUNCH((sd_propose_update_kernel), 1, 1024, 0, s, st, best, n_slots);
  return launched(1);
}

// One block; thread i lays out the sd_k token slots of decode slot i.
__global__ void __launch_bounds__(1024) sd_verify_prepare_kernel(RowState st, int n_slots) {
  RSD_PDL_SYNC();
  if (st.n_active[0] == 0) return;
  const int i = threadIdx.x;
  if (i >= n_slots) return;
  const int row = st.slot_row[i];
  const bool on = row >= 0 && st.gen_active[row];
  const int kk = on ? sd_round_tokens(st, row) : 0;
  const int pos0 = on ? st.kv_len[2][row] : 0;
  const int e = on ? st.gen_len[1][row] : 0;
  for (int j = 0; j < st.sd_k; ++j) {
    const int t = i * st.sd_k + j;
    if (j < kk) {
      st.pass_tok_id[t] = st.tok[(size_t)row * st.S + pos0 + j];   // the last written token, then the proposals
      st.pass_tok_pos[t] = pos0 + j;
      st.pass_tok_row[t] = row;
      st.sd_out_idx[t] = e + j;
    } else {
      st.pass_tok_row[t] = -1;
      st.sd_out_idx[t] = -1;
    }
  }
}

cudaError_t launch_sd_verify_prepare(const RowState& st, int n_slots, cudaStream_t s) {
  if (n_slots <= 0) return cudaSuccess;
  RSD_LAUNCH((sd_verify_prepare_kernel), 1, 1024, 0, s, st, n_slots);
  return launched(1);
}

__global__ void __launch_bounds__(1024)
sd_accept_kernel(RowState st, unsigned long long* best, int n_slots, LoopParams lp) {
  RSD_PDL_SYNC();
  if (st.n_active[0] == 0) return;
  const int i = threadIdx.x;
  int ended = 0, proposed = 0, matched = 0, rounds = 0;
  if (i < n_slots) {
    const int row = st.slot_row[i];
    const bool on = row >= 0 && st.gen_active[row];
    if (on) {
      const int kk = sd_round_tokens(st, row);
      const int pos0 = st.kv_len[2][row];
      const int e = st.gen_len[1][row];
      const int flen = st.forced_len[1][row];
      const int limit = flen > 0 ? flen : st.C;
      int n_emit = 0;
      bool done = false;
      for (int j = 0; j < kk; ++j) {
        const unsigned long long packed = best[i * st.sd_k + j];
        int t = packed ? (int)(0xFFFFFFFFu - (uint32_t)(packed & 0xFFFFFFFFull)) : 0;
        st.sampled[1][(size_t)row * st.C + e + j] = t;
        if (flen > 0) t = st.forced_tok[1][(size_t)row * st.C + e + j];
        const int prop = st.tok[(size_t)row * st.S + pos0 + 1 + j];
        st.tok[(size_t)row * st.S + pos0 + 1 + j] = t;
        st.gen_tok[1][(size_t)row * st.C + e + j] = t;
        ++n_emit;
        if (ends_step(t, lp) || e + n_emit == limit) done = true;
        if (t == prop) ++matched;
        if (done || t != prop) break;
      }
      // both caches hold the positions whose input tokens stand: the old last token and all written but the newest
      st.kv_len[2][row] = pos0 + n_emit;
      st.kv_len[0][row] = pos0 + n_emit;
      st.gen_len[1][row] = e + n_emit;
      if (done) { st.gen_active[row] = 0; ended = 1; }
      proposed = kk;
      rounds = 1;
    }
    for (int j = 0; j < st.sd_k; ++j) best[i * st.sd_k + j] = 0ull;
  }
  __shared__ int sums[4];
  if (threadIdx.x < 4) sums[threadIdx.x] = 0;
  __syncthreads();
  if (rounds) { atomicAdd(&sums[0], rounds); atomicAdd(&sums[1], proposed); atomicAdd(&sums[2], matched); atomicAdd(&sums[3], ended); }
  __syncthreads();
  if (threadIdx.x == 0) {
    st.sd_stats[0] += sums[0];
    st.sd_stats[1] += sums[1];
    st.sd_stats[2] += sums[2];
    st.sd_stats[3] += 1;
    st.sd_stats[4] = 0;
    st.n_active[0] -= sums[3];
  }
}

cudaError_t launch_sd_accept(const RowState& st, unsigned long long* best, int n_slots, const LoopParams& lp, cudaStream_t s) {
  if (n_slots <= 0) return cudaSuccess;
  RSD_LAUNCH((sd_accept_kernel), 1, 1024, 0, s, st, best, n_slots, lp);
  return launched(1);
}

// ---------------------------------------------------------------------------------------------
// Gate + compaction.  Acceptance criterion of Algorithm 2 with the weighting functions of Table 1
// (binary step: accept iff r >= delta) for the rows that took a draft step; a rejected row starts
// waiting for the target and its draft / PRM caches are rolled back to the step start.  All waiting
// rows (those of earlier calls included) are listed in ascending order by a warp ballot + popcount
// prefix.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float omega_weight(int kind, float r, float delta, float alpha) {
  switch (kind) {
    case 0: return delta;
    case 1: return r >= delta ? 1.f : 0.f;
    case 2: return fminf(1.f, fmaxf(0.f, r));
    case 3: return fmaxf(0.f, r / (1.f + r));
    case 4: return 1.f / (1.f + expf(-alpha * (r - delta)));
    default: return 0.f;
  }
}

// Ascending compaction of the flagged threads of a 1024-thread block: returns this thread's rank
// among flagged threads and the total; `wsum` holds 33 ints.
__device__ __forceinline__ int ballot_rank(bool flag, int* wsum, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned ballot = __ballot_sync(0xFFFFFFFFu, flag);
  const int in_warp = __popc(ballot & ((1u << lane) - 1u));
  __syncthreads();
  if (lane == 0) wsum[warp] = __popc(ballot);
  __syncthreads();
  if (warp == 0) {
    const int nw = blockDim.x >> 5;
    const int c = lane < nw ? wsum[lane] : 0;
    int inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if (lane >= o) inc += n;
    }
    wsum[lane] = inc - c;
    if (lane == 31) wsum[32] = inc;
  }
  __syncthreads();
  *total = wsum[32];
  return wsum[warp] + in_warp;
}

__global__ void __launch_bounds__(1024) gate_kernel(RowState st, float delta, LoopParams lp) {
  RSD_PDL_SYNC();
  __shared__ int wsum[33];
  const int b = threadIdx.x;
  bool live = false, waits = false;
  if (b < st.B) {
    live = st.live[b] != 0;
    waits = live && st.waiting[b] != 0;
    int code = 0;                      // rows that took no draft step in this call keep 0
    if (live && !waits) {
      const float r = st.rewards[b];
      const float w = omega_weight(lp.omega_kind, r, delta, lp.omega_alpha);
      int acc;
      if (w == 0.f) acc = 0;
      else if (w == 1.f) acc = 1;
      else {
        const uint4 rnd = philox4x32_10(make_uint4(0u, (uint32_t)st.z_len[b], (uint32_t)b, 3u),
                                        make_uint2((uint32_t)(lp.seed & 0xFFFFFFFFull), (uint32_t)(lp.seed >> 32)));
        acc = w >= uniform_from_bits(rnd.x) ? 1 : 0;
      }
      const uint8_t f = st.forced_accept[b];
      if (f <= 1) acc = f;
      code = acc ? 1 : 2;
      if (!acc) {
        waits = true;
        st.waiting[b] = 1;
        st.kv_len[0][b] = st.z_len[b] - 1;   // draft: drop y^_i, keep z_i minus its newest token
        if (!st.prm_shared) st.kv_len[1][b] = st.z_len[b];   // PRM: drop y^_i
      }
    } else if (!live) {
      st.rewards[b] = 0.f;
    }
    st.accept[b] = (uint8_t)code;
  }
  const int n_live = __syncthreads_count(live);
  int total;
  const int rank = ballot_rank(waits, wsum, &total);
  if (waits) st.rej_idx[rank] = b;
  if (b == 0) { st.n_rej[0] = total; st.n_live[0] = n_live; }
}

cudaError_t launch_gate(const RowState& st, float delta, const LoopParams& lp, cudaStream_t s) {
  RSD_LAUNCH((gate_kernel), 1, 1024, 0, s, st, delta, lp);
  return launched(1);
}

// Stand-alone gate + compaction for any B: per-block ballot counts, a scan of the block counts,
// then the ascending write.
__global__ void __launch_bounds__(1024)
gate_count_kernel(const float* rewards, const uint8_t* live, float delta, uint8_t* accept, int32_t* block_cnt, int B) {
  RSD_PDL_SYNC();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  bool rej = false;
  if (b < B) {
    const bool lv = live[b] != 0;
    const bool acc = lv && rewards[b] >= delta;
    accept[b] = acc ? 1 : 0;
    rej = lv && !acc;
  }
  const int n = __syncthreads_count(rej);
  if (threadIdx.x == 0) block_cnt[blockIdx.x] = n;
}

__global__ void __launch_bounds__(1024) gate_scan_kernel(int32_t* block_cnt, int n_blocks, int32_t* n_rej) {
  RSD_PDL_SYNC();
  // exclusive scan of up to 2^24 / 1024 = 16384 block counts by one block, 16 per thread
  __shared__ int scan[33];
  int local[16];
  int sum = 0;
  for (int i = 0; i < 16; ++i) {
    const int idx = threadIdx.x * 16 + i;
    local[i] = idx < n_blocks ? block_cnt[idx] : 0;
    sum += local[i];
  }
  int total;
  int off = block_exclusive_scan(sum, scan, &total);
  for (int i = 0; i < 16; ++i) {
    const int idx = threadIdx.x * 16 + i;
    if (idx < n_blocks) block_cnt[idx] = off;
    off += local[i];
  }
  if (threadIdx.x == 0) n_rej[0] = total;
}

__global__ void __launch_bounds__(1024)
gate_write_kernel(const uint8_t* live, const uint8_t* accept, const int32_t* block_off, int32_t* rej_idx, int B) {
  RSD_PDL_SYNC();
  __shared__ int wsum[33];
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  const bool rej = b < B && live[b] != 0 && accept[b] == 0;
  int total;
  const int rank = ballot_rank(rej, wsum, &total);
  if (rej) rej_idx[block_off[blockIdx.x] + rank] = b;
}

cudaError_t launch_gate_compact_large(const float* rewards, const uint8_t* live, float delta, uint8_t* accept,
                                      int32_t* rej_idx, int32_t* n_rej, int32_t* block_cnt, int B, cudaStream_t s) {
  const int n_blocks = (B + 1023) / 1024;
  RSD_LAUNCH((gate_count_kernel), n_blocks, 1024, 0, s, rewards, live, delta, accept, block_cnt, B);
  RSD_LAUNCH((gate_scan_kernel), 1, 1024, 0, s, block_cnt, n_blocks, n_rej);
  RSD_LAUNCH((gate_write_kernel), n_blocks, 1024, 0, s, live, accept, block_cnt, rej_idx, B);
  return launched(3);
}

// ---------------------------------------------------------------------------------------------
// Commit: y_i <- accept ? y^_i : target step; the row stops when EOS is in y_i, after max_steps
// steps, or when another step would not fit.  One block per row.
// ---------------------------------------------------------------------------------------------
__global__ void commit_kernel(RowState st, LoopParams lp, int target_ran, int32_t* out_tokens, int32_t* out_len,
                              float* out_rewards, uint8_t* out_accept, uint8_t* out_live, uint8_t* out_role,
                              uint8_t* out_waiting, int32_t* out_gen) {
  RSD_PDL_SYNC();
  const int b = blockIdx.x;
  const bool live = st.live[b] != 0;
  const int code = st.accept[b];
  const bool waits = live && st.waiting[b] != 0;
  // the step this row commits now: the accepted draft step, the target's step, or none (it waits)
  const int phase = (live && code == 1) ? 0 : (waits && target_ran) ? 1 : -1;
  const int n = phase >= 0 ? st.gen_len[phase][b] : 0;
  const int32_t* y = st.gen_tok[phase >= 0 ? phase : 0] + (size_t)b * st.C;
  int has_eos = 0;
  for (int j = threadIdx.x; j < st.C; j += blockDim.x) {
    const int t = j < n ? y[j] : 0;
    out_tokens[(size_t)b * st.C + j] = t;
    if (j < n && lp.eos_id >= 0 && t == lp.eos_id) has_eos = 1;
  }
  has_eos = __syncthreads_or(has_eos);
  if (threadIdx.x == 0) {
    out_len[b] = n;
    out_gen[b] = st.gen_len[0][b];
    out_gen[gridDim.x + b] = st.gen_len[1][b];
    out_rewards[b] = live ? st.rewards[b] : 0.f;
    out_accept[b] = (live && code == 1) ? 1 : 0;
    out_role[b] = (uint8_t)((live ? code : 0) | (phase == 1 ? 4 : 0));
    int still = live ? 1 : 0, still_waits = waits ? 1 : 0;
    if (phase >= 0) {
      const int z = st.z_len[b] + n;
      const int steps = st.n_steps[b] + 1;
      st.z_len[b] = z;
      st.n_steps[b] = steps;
      still = !(has_eos || steps >= lp.max_steps || z + st.C > st.S);
      st.live[b] = still;
      if (phase == 1) { st.waiting[b] = 0; still_waits = 0; }
    }
    out_live[b] = (uint8_t)still;
    out_waiting[b] = (uint8_t)(still && still_waits);
  }
}

cudaError_t launch_commit(const RowState& st, const LoopParams& lp, int target_ran, int32_t* out_tokens,
                          int32_t* out_len, float* out_rewards, uint8_t* out_accept, uint8_t* out_live,
                          uint8_t* out_role, uint8_t* out_waiting, int32_t* out_gen, cudaStream_t s) {
  if (st.B <= 0) return cudaSuccess;
  RSD_LAUNCH((commit_kernel), st.B, 128, 0, s, st, lp, target_ran, out_tokens, out_len, out_rewards, out_accept,
             out_live, out_role, out_waiting, out_gen);
  return launched(1);
}

}  // namespace rsd
