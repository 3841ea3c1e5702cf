// Algorithm 1 "in parallel on P workers: update beta_j using Eq. 2" + SAP step 4 (progress monitoring).
//
// With r = y - X beta, Eq. 2's argument x_j^T y - sum_{k != j} x_j^T x_k beta_k equals
// x_j^T r + n_j beta_j, so for every kept j, all from the SAME pre-round r:
//     g_j = x_j^T r,   beta_j' = S(beta_j + g_j / n_j, lambda / n_j),   S(a, k) = sign(a) max(|a| - k, 0)
// then beta_j <- beta_j', delta_j <- |beta_j' - beta_j|, r <- r - sum_j x_j (beta_j' - beta_j).
//
// "dot" streams the kept columns once against r (FP64 accumulation in a fixed order; the last CTA of a
// column sums the partials in index order and applies the soft threshold).  The residual update has every
// dense row owned by exactly one CTA and summed over the kept columns in list order; CSC contributions are
// added as 64-bit fixed-point integers with integer atomics (integer addition is associative, so hot rows
// shared by thousands of columns still give the same bits whatever the order) -- no floating-point atomics
// anywhere.
#include <climits>

#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Soft threshold + bookkeeping for kept entry a (one thread).
__device__ void finish_coefficient(const Problem& p, int a, int j, double g) {
  const double n = p.n2[j];
  const float b_old = p.beta[j];
  float b_new = b_old;
  if (n > 0.0) {
    const double c = step_scale(p);
    const double z = (double)b_old + c * g / n;
    const double m = fabs(z) - c * (double)p.lambda / n;
    b_new = (float)(m <= 0.0 ? 0.0 : (z > 0.0 ? m : -m));
  }
  const double d = (double)b_new - (double)b_old;        // the change that beta (FP32) really makes
  p.beta[j] = b_new;
  const float d_old = p.delta[j], d_new = (float)fabs(d);
  p.delta_prev[a] = d_old;
  p.delta[j] = d_new;
  if (p.patch_keys != nullptr)                           // (the round advances in a later kernel)
    next_round_keys(p, (uint32_t)j, d_old, d_new, &p.patch_keys[a], &p.patch_keys[p.n_keep + a]);
  p.dbeta[a] = (float)d;
  p.dbeta64[a] = d;
  if (d != 0.0) atomicAdd(&p.st->counts[3], 1);
  if (!isfinite(g)) atomicOr(&p.st->status, STRADS_STATUS_NONFINITE);
}

// ------------------------------------------------------------------------------------------------
// dense
// ------------------------------------------------------------------------------------------------
// Where the kept columns are read from: X itself.
struct ColumnSource {
  const float* base;
  long long pitch;
  const int* index;     // [n_kept] coefficient index
};

__global__ void __launch_bounds__(kThreads) k_dot_dense(Problem p, const int* __restrict__ kept, ColumnSource src) {
  chain_begin();
  const int a = blockIdx.y;
  if (a >= p.st->counts[2]) {
    if (blockIdx.x == 0 && threadIdx.x == 0) p.dbeta[a] = 0.f;
    return;
  }
  const int part = blockIdx.x, parts = gridDim.x;
  const int j = kept[a];
  const float* x = src.base + (long long)src.index[a] * src.pitch;
  const long long n4 = (p.N + 3) >> 2;                       // float4 groups (the last may be partial)
  const long long per = (n4 + parts - 1) / parts;
  const long long g0 = part * per, g1 = min(n4, g0 + per);
  double acc0 = 0.0, acc1 = 0.0;
  for (long long g = g0 + threadIdx.x; g < g1; g += kThreads) {
    const long long i = g << 2;
    float4 xv = __ldg(reinterpret_cast<const float4*>(x) + g);
    float4 rv;
    if (i + 3 < p.N) {
      rv = *(reinterpret_cast<const float4*>(p.resid) + g);
    } else {
      rv.x = p.resid[i];
      rv.y = i + 1 < p.N ? p.resid[i + 1] : 0.f;
      rv.z = i + 2 < p.N ? p.resid[i + 2] : 0.f;
      rv.w = 0.f;
      if (i + 1 >= p.N) xv.y = 0.f;
      if (i + 2 >= p.N) xv.z = 0.f;
      xv.w = 0.f;
    }
    acc0 += (double)xv.x * (double)rv.x + (double)xv.z * (double)rv.z;
    acc1 += (double)xv.y * (double)rv.y + (double)xv.w * (double)rv.w;
  }
  __shared__ double wsum[kThreads / 32];
  double v = warp_sum(acc0 + acc1);
  if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) s += wsum[w];
    p.dot_partial[(long long)a * parts + part] = s;
    __threadfence();
    if (atomicAdd(&p.dot_ticket[a], 1u) == (unsigned)parts - 1) {   // last part of this column: finish it
      __threadfence();
      double g = 0.0;
      for (int q = 0; q < parts; ++q) g += __ldcg(&p.dot_partial[(long long)a * parts + q]);
      p.dot_ticket[a] = 0;
      finish_coefficient(p, a, j, g);
    }
  }
}

// r <- r - sum_a x_a dbeta_a with every row owned by one CTA: 32 rows per CTA, a quarter-warp per column
// (8 lanes x float4 = one 128-byte line), so a warp reads four columns per instruction and the 32 quarter-warps
// of the CTA take the columns round-robin, eight loads in flight each: many small CTAs with shallow loops, which
// measured as fast as streaming the same columns whole (16.4 us for c3's 41 MB from a cold cache; 128- to 512-row
// blocks with a warp per column segment and the columns split into groups ran 1.4 to 6 times slower).
// Only the kept columns whose change is not zero are read (a coefficient that stays where it is moves nothing):
// their addresses and changes are compacted into shared memory first, in list order, so the column loads depend
// on nothing.  The per-row sums of the quarter-warps are added in a fixed order.
// proposals = 1: the changes were formed by the pack kernel for every candidate (cand_dbeta64 / cand_bnew by
// position in the list, p.kept_pos = positions of the kept ones); this kernel then also does the bookkeeping of
// the kept coefficients (beta, delta, dbeta), spread over its CTAs.  No other thread reads beta or delta here.
constexpr int kRowsPerCta = 32;
constexpr int kColSlots = kThreads / 8;    // quarter-warps per CTA
constexpr int kStageCols = 2048;           // moving columns staged per pass (32 KB of shared memory)

// gate: 0 always; 1 only if the window's Gram kernel settled the walk and P were kept inside the window
// (DeviceState::route == 0); 2 only otherwise (the update is then enqueued twice, behind the window's Gram and at the
// end of the branch that holds the walk kernel and the whole-list retry, and exactly one runs).
__global__ void __launch_bounds__(kThreads) k_apply_dense(Problem p, const int* __restrict__ kept, ColumnSource src,
                                                          int advance, int proposals, int gate) {
  chain_begin();
  if (gate != 0 && (p.st->route != 0) != (gate == 2)) return;
  __shared__ double part[kColSlots][kRowsPerCta];
  __shared__ double s_d[kStageCols];
  __shared__ long long s_off[kStageCols];
  __shared__ int s_scan[kThreads / 32];
  const int n_kept = p.st->counts[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int slot = tid >> 3, l8 = tid & 7;
  const long long i = (long long)blockIdx.x * kRowsPerCta + l8 * 4;

  // ranks of the kept entries whose change is not zero: thread t owns the entries [t c, (t + 1) c)
  const int per_thread = (n_kept + kThreads - 1) / kThreads;
  const int a_lo = min(tid * per_thread, n_kept), a_hi = min(a_lo + per_thread, n_kept);
  auto change_of = [&](int a) { return proposals ? p.cand_dbeta64[p.kept_pos[a]] : p.dbeta64[a]; };
  double d_first[4] = {0.0, 0.0, 0.0, 0.0};               // the first four stay in registers (all of them up to P = 1,024)
  int mine = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k)
    if (a_lo + k < a_hi) { d_first[k] = change_of(a_lo + k); mine += d_first[k] != 0.0; }
  for (int a = a_lo + 4; a < a_hi; ++a) mine += change_of(a) != 0.0;
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_scan[warp] = incl;
  __syncthreads();
  int before = 0, n_moving = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) { const int v = s_scan[w]; if (w < warp) before += v; n_moving += v; }
  const int rank0 = before + incl - mine;                 // rank of this thread's first moving entry

  double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
  for (int base = 0; base < n_moving; base += kStageCols) {
    const int n_here = min(kStageCols, n_moving - base);
    if (base > 0) __syncthreads();
    {
      int rank = rank0;
      auto place = [&](int a, double d) {
        if (d != 0.0) {
          if (rank >= base && rank < base + n_here) { s_d[rank - base] = d; s_off[rank - base] = (long long)src.index[a] * src.pitch; }
          ++rank;
        }
      };
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (a_lo + k < a_hi) place(a_lo + k, d_first[k]);
      for (int a = a_lo + 4; a < a_hi; ++a) place(a, change_of(a));
    }
    __syncthreads();
    if (i < p.N) {
      for (int a0 = slot; a0 < n_here; a0 += kColSlots * 8) {
        float4 xv[8];
        double d[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int a = a0 + u * kColSlots;
          d[u] = a < n_here ? s_d[a] : 0.0;
          xv[u] = __ldg(reinterpret_cast<const float4*>(src.base + s_off[a < n_here ? a : a0] + i));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          s0 += (double)xv[u].x * d[u]; s1 += (double)xv[u].y * d[u];
          s2 += (double)xv[u].z * d[u]; s3 += (double)xv[u].w * d[u];
        }
      }
    }
  }
  part[slot][l8 * 4 + 0] = s0; part[slot][l8 * 4 + 1] = s1;
  part[slot][l8 * 4 + 2] = s2; part[slot][l8 * 4 + 3] = s3;
  __syncthreads();
  if (tid < kRowsPerCta) {
    const long long r = (long long)blockIdx.x * kRowsPerCta + tid;
    if (r < p.N) {
      double s = 0.0;
#pragma unroll
      for (int w = 0; w < kColSlots; ++w) s += part[w][tid];
      if (s != 0.0) apply_row(p, r, s);
    }
  }
  DeviceState* st = p.st;
  const int cta = blockIdx.x, n_ctas = gridDim.x;
  if (proposals) {
    for (int a = cta * kThreads + tid; a < p.n_keep; a += n_ctas * kThreads) {
      if (a >= n_kept) { p.dbeta[a] = 0.f; continue; }
      const int pos = p.kept_pos[a], j = kept[a];
      const double d = p.cand_dbeta64[pos];
      p.beta[j] = p.cand_bnew[pos];
      p.delta_prev[a] = p.delta[j];
      p.delta[j] = (float)fabs(d);
      if (p.patch_keys != nullptr) {                   // formed by the pack kernel (this kernel advances the round)
        p.patch_keys[a] = p.cand_keys[pos];
        p.patch_keys[p.n_keep + a] = p.cand_keys[p.n_cand + pos];
      }
      p.dbeta[a] = (float)d;
      p.dbeta64[a] = d;
      if (d != 0.0) {                                    // counted here and in the running total: CTA 0 may be done already
        atomicAdd(&st->counts[3], 1);
        if (advance) atomicAdd(&st->totals[3], 1ull);
      }
      if (!isfinite(d)) atomicOr(&st->status, STRADS_STATUS_NONFINITE);
    }
  }
  if (cta == 0 && tid == 0 && advance) {
    st->totals[0] += 1; st->totals[1] += st->counts[1]; st->totals[2] += st->counts[2];
    if (!proposals) st->totals[3] += st->counts[3];
    st->round += (unsigned long long)p.part_count;       // this scheduler's next turn
  }
}

// ------------------------------------------------------------------------------------------------
// CSC
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_dot_csc(Problem p, const int* __restrict__ kept) {
  chain_begin();
  const int lane = threadIdx.x & 31;
  const int a = (blockIdx.x * kThreads + threadIdx.x) >> 5;
  if (a >= p.n_keep) return;
  if (a >= p.st->counts[2]) {
    if (lane == 0) p.dbeta[a] = 0.f;
    return;
  }
  const int j = kept[a];
  double acc = 0.0;
  for (long long q = p.xptr[j] + lane; q < p.xptr[j + 1]; q += 32)
    acc += (double)__ldg(p.xv + q) * (double)p.resid[__ldg(p.xrow + q)];
  acc = warp_sum(acc);
  if (lane == 0) {
    finish_coefficient(p, a, j, acc);
    atomicMax(&p.st->dmax_bits, (unsigned long long)__double_as_longlong(fabs(p.dbeta64[a])));
  }
}

// r <- r - sum_a x_a dbeta_a for sparse columns, in two kernels.  Contributions are added as 64-bit fixed-point
// integers with atomics into one accumulator per row (integer addition is associative: a row shared by
// thousands of columns gets the same bits in any order); then every row with a non-zero accumulator is
// updated once and its accumulator cleared.  Scale: every row sum is below n_kept * max|x| * max|dbeta| < 2^e;
// the unit is 2^-(61 - e).
__device__ __forceinline__ int csc_resid_shift(const Problem& p, int n_kept) {
  const double m = __longlong_as_double((long long)p.st->dmax_bits);
  if (!(m > 0.0) || !isfinite(m)) return INT_MIN;
  int e = 0;
  frexp(m * (double)p.st->x_abs_max * (double)max(n_kept, 1), &e);
  return 61 - e;
}

__global__ void __launch_bounds__(kThreads) k_scatter_csc(Problem p, const int* __restrict__ kept) {
  chain_begin();
  const int n_kept = p.st->counts[2];
  const int shift = csc_resid_shift(p, n_kept);
  if (blockIdx.x == 0 && threadIdx.x == 0) p.st->resid_shift = shift;     // for the apply kernel (nobody here reads it)
  if (shift == INT_MIN) return;
  const int lane = threadIdx.x & 31;
  const int a = (blockIdx.x * kThreads + threadIdx.x) >> 5;             // a warp per kept column
  if (a >= n_kept) return;
  const double d = p.dbeta64[a];
  if (d == 0.0) return;
  const int j = kept[a];
  const long long q1 = p.xptr[j + 1];
  for (long long q = p.xptr[j] + lane; q < q1; q += 32) {
    const long long fx = __double2ll_rn(ldexp((double)__ldg(p.xv + q) * d, shift));
    atomicAdd(reinterpret_cast<unsigned long long*>(p.resid_acc + __ldg(p.xrow + q)), (unsigned long long)fx);
  }
}

__global__ void __launch_bounds__(kThreads) k_apply_csc(Problem p, int advance) {
  chain_begin();
  const int shift = p.st->resid_shift;
  if (shift != INT_MIN) {
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long r = (long long)blockIdx.x * kThreads + threadIdx.x; r < p.N; r += stride) {
      const long long v = p.resid_acc[r];
      if (v != 0) {
        apply_row(p, r, ldexp((double)v, -shift));
        p.resid_acc[r] = 0;
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    DeviceState* st = p.st;
    st->dmax_bits = 0ull;                                // (read by the scatter kernel only)
    if (advance) {
      st->totals[0] += 1; st->totals[1] += st->counts[1]; st->totals[2] += st->counts[2]; st->totals[3] += st->counts[3];
      st->round += (unsigned long long)p.part_count;     // this scheduler's next turn
    }
  }
}

__global__ void k_set_counts(Problem p, int n_cand, int n_examined, int n_kept) {
  chain_begin();
  p.st->counts[0] = n_cand; p.st->counts[1] = n_examined; p.st->counts[2] = n_kept; p.st->counts[3] = 0;
}

__global__ void k_export(Problem p, const int* kept, int* kept_out, float* dbeta_out, int* counts_out) {
  chain_begin();
  const int n_kept = p.st->counts[2];
  for (int a = blockIdx.x * blockDim.x + threadIdx.x; a < p.n_keep; a += gridDim.x * blockDim.x) {
    if (kept_out != nullptr) kept_out[a] = a < n_kept ? kept[a] : -1;
    if (dbeta_out != nullptr) dbeta_out[a] = a < n_kept ? p.dbeta[a] : 0.f;
  }
  if (counts_out != nullptr && blockIdx.x == 0 && threadIdx.x < 4) counts_out[threadIdx.x] = p.st->counts[threadIdx.x];
}

}  // namespace

// after_pack: this round's pack kernel ran (dense, tensor-core Gram); with p.proposals it has left the changes of all
// candidates, and p.kept_pos says where the kept ones are in the list.
cudaError_t launch_update(const Problem& p, const int* kept, int advance, bool after_pack, cudaStream_t s, int gate) {
  if (p.layout == STRADS_DENSE_COLMAJOR) {
    ColumnSource src;
    src.base = p.xv; src.pitch = p.ld; src.index = kept;           // the kept columns, from X itself
    cudaError_t e;
    const int proposals = after_pack && p.proposals ? 1 : 0;     // the pack kernel of this round left the changes
    if (gate != 0 && !proposals) return cudaErrorInvalidValue;    // (only the single-kernel update is gated)
    if (!proposals && (e = launch_chained(k_dot_dense, dim3(p.dot_parts, p.n_keep), kThreads, 0, s, p, kept, src)) != cudaSuccess)
      return e;
    return launch_chained(k_apply_dense, (unsigned)((p.N + kRowsPerCta - 1) / kRowsPerCta), kThreads, 0, s, p, kept, src,
                          advance, proposals, gate);
  } else {
    cudaError_t e;
    if ((e = launch_chained(k_dot_csc, (p.n_keep * 32 + kThreads - 1) / kThreads, kThreads, 0, s, p, kept)) != cudaSuccess) return e;
    if ((e = launch_chained(k_scatter_csc, (p.n_keep * 32 + kThreads - 1) / kThreads, kThreads, 0, s, p, kept)) != cudaSuccess) return e;
    long long grid = (p.N + kThreads - 1) / kThreads;
    if (grid > (long long)p.sm_count * 8) grid = (long long)p.sm_count * 8;
    return launch_chained(k_apply_csc, (unsigned)grid, kThreads, 0, s, p, advance);
  }
}

cudaError_t launch_set_counts(const Problem& p, int n_cand, int n_examined, int n_kept, cudaStream_t s) {
  return launch_chained(k_set_counts, 1, 1, 0, s, p, n_cand, n_examined, n_kept);
}

cudaError_t launch_export(const Problem& p, const int* kept, int* kept_out, float* dbeta_out, int* counts_out,
                          cudaStream_t s) {
  return launch_chained(k_export, (p.n_keep + 255) / 256, 256, 0, s, p, kept, kept_out, dbeta_out, counts_out);
}

}  // namespace strads
