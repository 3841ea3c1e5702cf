// SAP step 2, CSC X: conflict bits of all candidate pairs.  x_a^T x_b of two sparse columns is the
// intersection of two ascending row lists.  One CTA owns candidate a and stages its column in shared
// memory; each warp takes 32 consecutive later candidates b (one per lane), every lane merges its own
// column b against the staged column a, and one ballot yields the 32 conflict bits of that mask word.
// Products are accumulated in row order, so the result does not depend on the launch shape.
//
// That all-pairs kernel does one merge per pair, although two sparse columns rarely share a row at all (the
// paper's point about sparse designs: most pairs are exactly uncorrelated).  So the pairs worth a product are found
// first, by rows: every candidate is entered, with its value there, into the bucket of each row it has an entry in.
// One CTA per candidate a then reads the buckets of a's rows: what it finds there are exactly the terms
// x_a[i] x_b[i] of the inner products with the later candidates b that share a row with a.  Sorted by (b, i) and
// added up in that order, they give x_a^T x_b with the products in row order again, so with the same bits as the
// merge, and no second column is ever read.  A bucket holds kBucketSlots candidates and a candidate's terms are
// sorted in shared memory: when a bucket overflows (rows shared by very many columns) or a candidate meets too
// many others, the all-pairs kernel, launched behind, redoes the round's bits, and the buckets are left alone for
// the next 63 rounds of that scheduler.
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

// Buckets, step 1: a warp per candidate a clears its conflict row and enters a, with its value there, into the bucket
// of each of its rows.
__global__ void __launch_bounds__(kThreads) k_csc_bucket_fill(Problem p, const int* __restrict__ cand, int n_cand,
                                                               int only_if_short, int window) {
  chain_begin();
  DeviceState* st = p.st;
  const bool wanted = gram_wanted(p, only_if_short, window);
  const bool use = wanted && !(st->bucket_avoid && ((st->round / (unsigned)p.part_count) & 63ull) != 0);
  if (blockIdx.x == 0 && threadIdx.x == 0) { st->bucket_used = use ? 1 : 0; st->bucket_failed = 0; }
  if (!use) return;
  const int lane = threadIdx.x & 31;
  const int words = (n_cand + 31) >> 5;
  const int n_warps = (int)(gridDim.x * (unsigned)kThreads) >> 5;
  for (int a = (int)((blockIdx.x * (unsigned)kThreads + threadIdx.x) >> 5); a < n_cand; a += n_warps) {
    for (int w = lane; w < words; w += 32) p.conflict[(long long)a * p.mask_words + w] = 0u;
    const int ja = cand[a];
    const long long q0 = p.xptr[ja], q1 = p.xptr[ja + 1];
    if (lane == 0) {
      BucketColumn col;
      col.q0 = q0; col.n = (int)(q1 - q0); col.j = ja; col.n2 = coupling_n2(p, ja);
      p.bucket_cols[a] = col;
    }
    for (long long q = q0 + lane; q < q1; q += 32) {
      const int r = __ldg(p.xrow + q);
      const float v = __ldg(p.xv + q);
      const unsigned int slot = atomicAdd(&p.bucket_count[r], 1u);
      if (slot < (unsigned)kBucketSlots) {
        p.bucket_items[(long long)r * kBucketSlots + slot] = a;
        p.bucket_vals[(long long)r * kBucketSlots + slot] = v;
      }
    }
  }
}

// Step 2: one CTA per candidate a; a thread per entry (row i, value x_a[i]) of column a reads the bucket of row i
// and collects a term (b, i, x_a[i], x_b[i]) for every later candidate b in it.  The CTA ranks its terms by (b, i)
// (each term counts the smaller ones: a few dozen terms, no sorting network needed), and the first term of every b
// adds that b's products up in row order, with the fused multiply-add of sparse_dot, and decides the pair.
// (Earlier forms of this step read column b for every pair found: a thread per pair merging the two sorted lists
// step by step took 40 us for the ~70,000 pairs of a 1,664-candidate window of 50-entry columns, a warp per pair
// looking b's entries up in a table of a's 38 to 48 us, bound by instruction issue.)
constexpr int kMeetThreads = 128;
constexpr int kMaxMeet = 4 * kMeetThreads;      // terms a candidate may collect (more: the round falls back)

__global__ void __launch_bounds__(kMeetThreads) k_csc_bucket_dots(Problem p, int n_cand) {
  chain_begin();
  DeviceState* st = p.st;
  if (!st->bucket_used) return;
  __shared__ unsigned long long key[kMaxMeet];          // b << 32 | position of row i in column a
  __shared__ float fa[kMaxMeet], fb[kMaxMeet];          // x_a[i], x_b[i]
  __shared__ int n_meet;
  const double rho = (double)p.rho;
  const int tid = threadIdx.x;
  // (capped grid: the CTAs take the candidates in turn, the stripes alternately forwards and backwards, since an
  //  early candidate has more later ones to meet)
  for (int base = 0, turn = 0; base < n_cand; base += gridDim.x, ++turn) {
    const int a = base + ((turn & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x);
    if (a >= n_cand) continue;
    const BucketColumn ca = p.bucket_cols[a];
    __syncthreads();                                     // the terms of the last candidate are no longer read
    if (tid == 0) n_meet = 0;
    __syncthreads();
    for (int q = tid; q < ca.n; q += kMeetThreads) {
      const int r = __ldg(p.xrow + ca.q0 + q);
      const float v = __ldg(p.xv + ca.q0 + q);
      const unsigned int cnt = p.bucket_count[r];
      if (cnt > (unsigned)kBucketSlots) { st->bucket_failed = 1; continue; }
      const int* items = p.bucket_items + (long long)r * kBucketSlots;
      const float* vals = p.bucket_vals + (long long)r * kBucketSlots;
      for (unsigned int i = 0; i < cnt; ++i) {
        const int b = items[i];
        if (b <= a) continue;
        const int slot = atomicAdd(&n_meet, 1);
        if (slot < kMaxMeet) {
          key[slot] = ((unsigned long long)(unsigned int)b << 32) | (unsigned int)q;
          fa[slot] = v;
          fb[slot] = vals[i];
        }
      }
    }
    __syncthreads();
    const int np = n_meet;
    if (np > kMaxMeet) {                                 // (the same for all threads of the CTA)
      if (tid == 0) st->bucket_failed = 1;
      continue;
    }
    unsigned long long mk[kMaxMeet / kMeetThreads];
    float ma[kMaxMeet / kMeetThreads], mb[kMaxMeet / kMeetThreads];
    int mr[kMaxMeet / kMeetThreads];
#pragma unroll
    for (int i = 0; i < kMaxMeet / kMeetThreads; ++i) {
      const int t = tid + i * kMeetThreads;
      mr[i] = -1;
      if (t < np) {
        mk[i] = key[t]; ma[i] = fa[t]; mb[i] = fb[t];
        int r = 0;
        for (int s = 0; s < np; ++s) r += key[s] < mk[i] ? 1 : 0;       // (b, i) is unique: the ranks are a permutation
        mr[i] = r;
      }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kMaxMeet / kMeetThreads; ++i)
      if (mr[i] >= 0) { key[mr[i]] = mk[i]; fa[mr[i]] = ma[i]; fb[mr[i]] = mb[i]; }
    __syncthreads();
    for (int t = tid; t < np; t += kMeetThreads) {
      const unsigned int b = (unsigned int)(key[t] >> 32);
      if (t > 0 && (unsigned int)(key[t - 1] >> 32) == b) continue;     // not the first term of its b
      float dot = 0.f;
      for (int s = t; s < np && (unsigned int)(key[s] >> 32) == b; ++s) dot = fmaf(fa[s], fb[s], dot);
      const double den = sqrt(ca.n2 * p.bucket_cols[b].n2);
      if (den > 0.0 && fabs((double)dot) >= rho * den) {
        atomicOr(&p.conflict[(long long)a * p.mask_words + (b >> 5)], 1u << (b & 31));
        list_conflict(p, a, (int)b);
      }
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
    if (used) {                                            // empty this round's buckets: a warp per candidate
      const int n_warps = (int)(gridDim.x * (unsigned)kThreads) >> 5;
      for (int a = (int)((blockIdx.x * (unsigned)kThreads + threadIdx.x) >> 5); a < n_cand; a += n_warps) {
        const int ja = cand[a];
        const long long q1 = p.xptr[ja + 1];
        for (long long q = p.xptr[ja] + (threadIdx.x & 31); q < q1; q += 32) p.bucket_count[__ldg(p.xrow + q)] = 0u;
      }
      if (!failed) return;
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) p.st->edges_off = 1;     // this kernel sets bits without listing the pairs
  __shared__ int arow[kStage];
  __shared__ float aval[kStage];
  // (capped grid: the CTAs take the candidates in turn; candidate a tests only the candidates of its own mask word and
  // after, so the stripes are handed out alternately forwards and backwards to even the CTAs' work out)
  for (int base = 0, turn = 0; base < n_cand; base += gridDim.x, ++turn) {
  const int a = base + ((turn & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x);
  if (turn) __syncthreads();                               // the staged column of the last candidate is no longer read
  if (a >= n_cand) continue;
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
  if ((e = launch_chained(k_csc_bucket_dots, (unsigned)min((long long)n_cand, 2 * cap), kMeetThreads, 0, s, p, n_cand)) != cudaSuccess) return e;
  return launch_chained(k_gram_csc, capped(n_cand), kThreads, 0, s, p, cand, n_cand, gram_dbg, ois, win, 1);
}

}  // namespace strads
