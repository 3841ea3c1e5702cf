// SAP step 2, CSC X: conflict bits of all candidate pairs.  x_a^T x_b of two sparse columns is the
// intersection of two ascending row lists.  One CTA owns candidate a and stages its column in shared
// memory; each warp takes 32 consecutive later candidates b (one per lane), every lane merges its own
// column b against the staged column a, and one ballot yields the 32 conflict bits of that mask word.
// Products are accumulated in row order, so the result does not depend on the launch shape.
//
// That all-pairs kernel does one merge per pair, although two sparse columns rarely share a row at all (the
// paper's point about sparse designs: most pairs are exactly uncorrelated).  So the pairs worth a merge are found
// first, by rows: every candidate is entered into the bucket of each row it has an entry in, every row then
// emits the pairs of candidates in its bucket, and only those pairs are merged (by the same routine, so with
// the same bits) and their conflict bits set.  A bucket holds kBucketSlots candidates and the pair list is
// finite: when either overflows (rows shared by very many columns), the all-pairs kernel, launched behind,
// redoes the round's bits, and the buckets are left alone for the next 63 rounds of that scheduler.
#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;
constexpr int kStage = 1024;          // entries of column a staged in shared memory (longer columns: global)

// Whether this launch has anything to do (same test in every kernel of the step).
__device__ __forceinline__ bool gram_wanted(const Problem& p, int only_if_short, int window) {
  if (only_if_short && !p.st->window_short) return false;
  if (window && window_skipped(p)) return false;
  return true;
}

// Buckets, step 1: a warp per candidate a clears its conflict row and enters a into the bucket of each of its rows.
__global__ void __launch_bounds__(kThreads) k_csc_bucket_fill(Problem p, const int* __restrict__ cand, int n_cand,
                                                               int only_if_short, int window) {
  chain_begin();
  DeviceState* st = p.st;
  const bool wanted = gram_wanted(p, only_if_short, window);
  const bool use = wanted && !(st->bucket_avoid && ((st->round / (unsigned)p.part_count) & 63ull) != 0);
  if (blockIdx.x == 0 && threadIdx.x == 0) { st->bucket_used = use ? 1 : 0; st->pair_count = 0; st->bucket_failed = 0; }
  if (!use) return;
  const int lane = threadIdx.x & 31;
  const int words = (n_cand + 31) >> 5;
  const int n_warps = (int)(gridDim.x * (unsigned)kThreads) >> 5;
  for (int a = (int)((blockIdx.x * (unsigned)kThreads + threadIdx.x) >> 5); a < n_cand; a += n_warps) {
    for (int w = lane; w < words; w += 32) p.conflict[(long long)a * p.mask_words + w] = 0u;
    const int ja = cand[a];
    const long long q1 = p.xptr[ja + 1];
    for (long long q = p.xptr[ja] + lane; q < q1; q += 32) {
      const int r = __ldg(p.xrow + q);
      const unsigned int slot = atomicAdd(&p.bucket_count[r], 1u);
      if (slot < (unsigned)kBucketSlots) p.bucket_items[(long long)r * kBucketSlots + slot] = a;
    }
  }
}

// Step 2: a thread per row emits the pairs of its bucket (and empties it for the next round).
__global__ void __launch_bounds__(kThreads) k_csc_bucket_pairs(Problem p) {
  chain_begin();
  DeviceState* st = p.st;
  if (!st->bucket_used) return;
  const int lane = threadIdx.x & 31;
  // (the grid is capped, so that a launch with nothing to do costs little: a thread takes several rows in turn; the
  //  trip count is the same for all lanes of a warp)
  for (long long r0 = (long long)blockIdx.x * kThreads; r0 < p.N; r0 += (long long)gridDim.x * kThreads) {
  const long long r = r0 + threadIdx.x;
  unsigned int c = 0;
  if (r < p.N) {
    c = p.bucket_count[r];
    if (c) p.bucket_count[r] = 0u;
    if (c > (unsigned)kBucketSlots) { st->bucket_failed = 1; c = 0; }
  }
  const unsigned int mine = c * (c - (c ? 1u : 0u)) / 2u;
  unsigned int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  const unsigned int total = __shfl_sync(0xffffffffu, incl, 31);
  if (total == 0) continue;
  unsigned int base = 0;
  if (lane == 31) base = atomicAdd(&st->pair_count, total);
  base = __shfl_sync(0xffffffffu, base, 31);
  if (base + total > (unsigned)p.pair_cap) {          // the list is full: this round falls back to all pairs
    if (lane == 31) st->bucket_failed = 1;
    continue;
  }
  if (mine == 0) continue;
  unsigned int at = base + incl - mine;
  const int* items = p.bucket_items + r * kBucketSlots;
  int it[kBucketSlots];
#pragma unroll
  for (int i = 0; i < kBucketSlots; ++i) it[i] = i < (int)c ? items[i] : 0;
#pragma unroll
  for (int i = 0; i < kBucketSlots; ++i)
#pragma unroll
    for (int j = i + 1; j < kBucketSlots; ++j)
      if (j < (int)c) {
        const int lo = min(it[i], it[j]), hi = max(it[i], it[j]);
        p.pair_list[at++] = ((unsigned int)lo << 16) | (unsigned int)hi;
      }
  }
}

// Step 3: a thread per listed pair merges the two columns and sets the pair's conflict bit in the row of the
// earlier candidate (a pair that shares several rows is listed as often and gives the same bit each time).
__global__ void __launch_bounds__(kThreads) k_csc_pair_bits(Problem p, const int* __restrict__ cand) {
  chain_begin();
  const DeviceState* st = p.st;
  if (!st->bucket_used || st->bucket_failed) return;
  const unsigned int n = st->pair_count;
  const double rho = (double)p.rho;
  for (unsigned int i = blockIdx.x * (unsigned)kThreads + threadIdx.x; i < n; i += gridDim.x * (unsigned)kThreads) {
    const unsigned int pr = __ldcg(p.pair_list + i);
    const int a = (int)(pr >> 16), b = (int)(pr & 0xffffu);
    if (a == b) continue;                               // (a row never lists a column twice; defensive)
    const int ja = cand[a], jb = cand[b];
    const long long a0 = p.xptr[ja];
    const float dot = sparse_dot(p.xrow + a0, p.xv + a0, (int)(p.xptr[ja + 1] - a0), p, jb);
    const double den = sqrt(coupling_n2(p, ja) * coupling_n2(p, jb));
    if (den > 0.0 && fabs((double)dot) >= rho * den) {
      atomicOr(&p.conflict[(long long)a * p.mask_words + (b >> 5)], 1u << (b & 31));
      list_conflict(p, a, b);                             // (a pair listed twice is listed twice here too: harmless)
    }
  }
}

// All pairs.  after_buckets: launched behind the bucket kernels; it then only runs when they were not used this
// round or gave up, and it records whether the next rounds should try them at all.
__global__ void __launch_bounds__(kThreads) k_gram_csc(Problem p, const int* __restrict__ cand, int n_cand,
                                                        float* __restrict__ gram_dbg, int only_if_short, int window,
                                                        int after_buckets) {
  chain_begin();
  if (!gram_wanted(p, only_if_short, window)) return;
  if (after_buckets) {
    const int used = p.st->bucket_used, failed = p.st->bucket_failed;
    if (blockIdx.x == 0 && threadIdx.x == 0 && used) p.st->bucket_avoid = failed;   // (nobody reads it in this kernel)
    if (used && !failed) return;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) p.st->edges_off = 1;     // this kernel sets bits without listing the pairs
  __shared__ int arow[kStage];
  __shared__ float aval[kStage];
  for (int a = blockIdx.x; a < n_cand; a += gridDim.x) {   // (capped grid: the CTAs take the candidates in turn)
  if (a != (int)blockIdx.x) __syncthreads();               // the staged column of the last candidate is no longer read
  const int ja = cand[a];
  const long long a0 = p.xptr[ja];
  const int na = (int)(p.xptr[ja + 1] - a0);
  const bool staged = na <= kStage;
  if (staged)
    for (int q = threadIdx.x; q < na; q += kThreads) { arow[q] = p.xrow[a0 + q]; aval[q] = p.xv[a0 + q]; }
  __syncthreads();
  const int* ar = staged ? arow : p.xrow + a0;
  const float* av = staged ? aval : p.xv + a0;
  const double n2a = coupling_n2(p, ja);
  const double rho = (double)p.rho;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  for (int w = (a >> 5) + warp; w < p.mask_words; w += kThreads / 32) {
    const int b = w * 32 + lane;
    bool hit = false;
    if (b < n_cand && b != a) {
      const int jb = cand[b];
      const float dot = sparse_dot(ar, av, na, p, jb);
      const double den = sqrt(n2a * coupling_n2(p, jb));
      hit = den > 0.0 && fabs((double)dot) >= rho * den;
      if (gram_dbg != nullptr) {
        gram_dbg[(long long)a * n_cand + b] = dot;
        if (b > a) gram_dbg[(long long)b * n_cand + a] = dot;
      }
    } else if (b == a && gram_dbg != nullptr) {
      gram_dbg[(long long)a * n_cand + a] = (float)n2a;
    }
    const unsigned int word = __ballot_sync(0xffffffffu, hit);
    if (lane == 0) p.conflict[(long long)a * p.mask_words + w] = word;
  }
  }
}

}  // namespace

cudaError_t launch_gram_csc(const Problem& p, const int* cand, int n_cand, float* gram_dbg, bool only_if_short,
                            bool window, cudaStream_t s) {
  const int ois = only_if_short ? 1 : 0, win = window ? 1 : 0;
  // grids of at most eight CTAs per SM: in many rounds (a window that keeps failing is skipped) these launches have
  // nothing to do, and what an idle launch costs is the launching of its CTAs
  const long long cap = (long long)p.sm_count * 8;
  auto capped = [&](long long n) { return (unsigned)(n < cap ? (n > 0 ? n : 1) : cap); };
  if (p.bucket_count == nullptr || gram_dbg != nullptr || n_cand > 65535)
    return launch_chained(k_gram_csc, capped(n_cand), kThreads, 0, s, p, cand, n_cand, gram_dbg, ois, win, 0);
  cudaError_t e;
  if ((e = launch_chained(k_csc_bucket_fill, capped(((long long)n_cand * 32 + kThreads - 1) / kThreads), kThreads, 0, s, p, cand, n_cand, ois, win)) != cudaSuccess)
    return e;
  if ((e = launch_chained(k_csc_bucket_pairs, capped((p.N + kThreads - 1) / kThreads), kThreads, 0, s, p)) != cudaSuccess) return e;
  if ((e = launch_chained(k_csc_pair_bits, p.sm_count * 8, kThreads, 0, s, p, cand)) != cudaSuccess) return e;
  return launch_chained(k_gram_csc, capped(n_cand), kThreads, 0, s, p, cand, n_cand, gram_dbg, ois, win, 1);
}

}  // namespace strads
