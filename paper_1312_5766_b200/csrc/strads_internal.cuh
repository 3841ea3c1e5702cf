// Internal declarations shared by the kernels of libstrads_b200.so (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "strads.h"

namespace strads {

// ---------------------------------------------------------------------------------------------
// Device-resident state of one handle (lives at the start of the caller's workspace).
// ---------------------------------------------------------------------------------------------
struct SelectState {            // written by the sampler's histogram kernel, read by collect / sort
  unsigned long long prefix;    // boundary value of the top `bits` bits of the 64-bit key
  int bits;                     // how many top bits `prefix` covers
  int n_sure;                   // keys whose top bits are < prefix (all of them are winners)
  int n_boundary;               // keys whose top bits are == prefix
  int pad;
};

struct DeviceState {
  unsigned long long round;     // t, the Philox counter word (of this scheduler's next round: t mod S == its index)
  unsigned long long totals[4]; // rounds, examined, kept, nonzero
  unsigned int status;          // STRADS_STATUS_* bits
  unsigned int hist_ticket;     // "last block done" tickets
  unsigned int sure_count;      // append cursors of the collect kernel
  unsigned int boundary_count;
  int counts[4];                // n_cand, n_examined, n_kept, n_nonzero of the current round
  SelectState sel;
  double objective;             // result slot of the objective reduction
  float x_abs_max;              // max |x_ij| (CSC: bounds the fixed-point residual update)
  int beta0_nonzero;            // set at init when the starting beta has a non-zero entry
  unsigned int amb_count;       // pairs the BF16 screen of the dense Gram left to the exact recheck
  int window_short;             // the filter ran out of its candidate window before P were kept: redo on all P'
  int prefer_walk;              // CSC: the last round needed the whole list, so skip the window attempt for a while
  int bucket_failed;            // ... a bucket or the pair list overflowed this round: the all-pairs kernel redoes the bits
  int bucket_avoid;             // ... it overflowed lately: go straight to the all-pairs kernel for a while
  unsigned long long dmax_bits; // CSC update: bits of max |change| of this round (non-negative doubles order like integers)
  int resid_shift;              // CSC update: this round's fixed-point scale is 2^resid_shift (INT_MIN: nothing moved)
  float t_cut;                  // sampler: cutoff for the next round's first pass (0: none), see k_sample_hist
  int sample_redo;              // sampler: the guided first pass found too few keys; the plain pass behind it runs
  int walk_streak;              // CSC: window attempts in a row that were too short (each doubles the wait for the next)
  int window_hopeless;          // CSC: the last whole-list walk kept fewer than P, or found its P-th member behind the window
  int bucket_used;              // ... this round's Gram went through the buckets (decided once, by the first kernel)
  unsigned int surv_count;      // sampler: keys the guided first pass found below its cutoff and saved (append cursor)
  int surv_valid;               // ... they are all there (no overflow, no repeat): the collect pass reads them, not delta[J]
  unsigned int gram_ticket;     // dense window Gram: CTAs that are done (the last one rechecks and walks)
  int walk_pending;             // ... that CTA could not settle the walk from the pair list: the walk kernel behind it does
  int route;                    // ... which gated copy of the update runs: 0 the one behind the window, 1 the retry branch's
  unsigned int edge_count;      // conflicting pairs listed by the Gram kernels of this round (may exceed the list)
  int edges_off;                // a kernel that sets bits without listing pairs has run: the list is not complete
};

struct WalkControl {            // shared by the CTAs of the cooperative on-demand walk (CSC)
  unsigned int bar_count, bar_gen;   // grid barrier
  int failed;
  int pad;
};

static constexpr int kBucketSlots = 16;   // candidates per row bucket (more: the round falls back to all pairs)
// What the on-demand walk needs of a candidate's column, gathered once per walk (two 16-byte loads instead of a chain
// of three accesses per merge).
struct __align__(16) WalkColumn {
  long long q0;     // first stored entry
  int n;            // entries
  int j;            // the column
  double n2;        // its coupling_n2
  double unused;
};
// What the bucket kernels need of a candidate's column, gathered once per round (one access instead of a chain of three).
struct BucketColumn {
  long long q0;     // first stored entry
  int n;            // entries
  int j;            // the column
  double n2;        // its coupling_n2
};
static constexpr int kHistBits = 12;
static constexpr int kHistBins = 1 << kHistBits;

// Everything a launch needs; filled once at init (host copy in the handle).
struct Problem {
  int layout;
  long long N, J, ld;
  const float* xv;
  const int* xrow;
  const long long* xptr;
  long long nnz;                // CSC: stored entries (the length of xv and xrow)
  const float* y;
  float* beta;
  float* resid;
  float* delta;
  float lambda, eta, rho, c_init;
  int n_cand, n_keep;
  unsigned long long seed;
  unsigned int flags;
  // workspace carve-up
  DeviceState* st;
  double* n2;                   // [J]
  unsigned int* hist;           // [kHistBins]
  unsigned long long* sure;     // [cap_sure]
  unsigned long long* boundary; // [cap_boundary]
  int cap_sure, cap_boundary;
  int* cand;                    // [n_cand]
  int* kept;                    // [n_keep]
  int* kept_pos;                // [n_keep] positions of the kept coefficients in the candidate list
  float* dbeta;                 // [n_keep]
  double* dbeta64;              // [n_keep]
  unsigned int* conflict;       // [n_cand][mask_words]
  int mask_words;
  double* dot_partial;          // [n_keep][dot_parts]
  unsigned int* dot_ticket;     // [n_keep]
  int dot_parts;
  float* margin;                // STRADS_FLAG_LOGISTIC: [N] the margin X beta (shared by all schedulers)
  double* obj_partial;          // [2 * kObjBlocks]
  unsigned int* amb_pairs;      // [cap_amb] (a << 16 | b), positions in the candidate list
  int cap_amb;
  long long ldc;                // N rounded up to a multiple of 4
  unsigned short* xcb;          // dense: the same columns rounded to BF16, [n_cand][ldcb]: operands of the Gram's screen
  long long ldcb;               // N rounded up to a multiple of 8
  // dense, one scheduler: the pack kernel also forms x_c^T r and with it the change every candidate would
  // make if kept (valid while r is untouched between the pack and the update: same stream, same round)
  int proposals;                // 1: the pack kernel fills the two arrays below and the update applies them
  double* cand_dbeta64;         // [n_cand] proposed change of candidate position a
  float* cand_bnew;             // [n_cand] proposed new beta
  const int* cand_cur;          // candidate list of the Gram in flight (set per launch)
  unsigned int* walk_blocked;   // CSC on-demand walk: running mask [mask_words], OR-ed into by the whole grid
  WalkControl* walk_ctl;
  WalkColumn* walk_cols;        // ... [P'] where each candidate's column lies, gathered when the walk starts
  long long* resid_acc;         // CSC: [N] fixed-point accumulators of the residual update (zero between rounds)
  // CSC Gram by row buckets (null / 0 when not provided for)
  unsigned int* bucket_count;   // [N] candidates of this round's list with an entry in row i (zero between rounds)
  int* bucket_items;            // [N][kBucketSlots] their positions in the list
  float* bucket_vals;           // [N][kBucketSlots] their values in row i
  BucketColumn* bucket_cols;    // [P'] where each candidate's column lies, as the bucket kernels need it
  int sm_count;
  // sampling ahead (one scheduler): the draw of round t + 1 is made during round t from the priorities of its start
  // and corrected for the coefficients that round t updates (k_sample_patch)
  const unsigned long long* round_ptr;   // the sampler's round index is *round_ptr + round_ahead
  int round_ahead;
  unsigned long long* keys_out;          // sampler: if set, the winners' keys in rank order go here too
  int* bin_off;                          // sampler: [kHistBins + 1] where the sure keys of a histogram bin start in `sure` (null: appended in any order)
  unsigned int* bin_cur;                 // sampler: [kHistBins] append cursor of every bin
  unsigned long long* survivors;         // sampler: [cap_survivors] keys below the guided first pass's cutoff (null: not kept)
  int cap_survivors;
  float* delta_prev;                     // [n_keep] delta of the kept coefficients before this round's update
  unsigned long long* patch_keys;        // [2][n_keep] their race keys of the NEXT round, before and after the update
  unsigned long long* cand_keys;         // dense, proposals: [2][n_cand] the same for every candidate, by position
  // Conflicts are normally few (a handful per hundred candidates), so the Gram kernels also list the conflicting
  // pairs (a << 16 | b, a < b, positions in the list) and the walk works from that list when it is complete.
  unsigned int* edges;                   // [cap_edges]
  int cap_edges;
  // scheduler threads: this Problem is scheduler part_index of part_count and owns { j : j mod part_count == part_index }
  int part_count, part_index;
  // bounded device-side waits: iteration limit of every spin (0: each kernel's own default), and, for exercising the
  // expiry path, a launch whose operand loads are withheld so that a wait does run out (strads_inject_stall)
  unsigned int wait_limit;
  int stall;
};
static constexpr int kObjBlocks = 296;

// A Gram kernel found candidates a < b (positions in the list) in conflict.
__device__ __forceinline__ void list_conflict(const Problem& p, int a, int b) {
  const unsigned int slot = atomicAdd(&p.st->edge_count, 1u);
  if (slot < (unsigned)p.cap_edges) p.edges[slot] = ((unsigned int)a << 16) | (unsigned int)b;
}

// CSC: whether this round leaves the candidate window out and goes straight to the on-demand walk: after a
// window that was too short, the next attempt comes 64 rounds (of this scheduler) later, and twice as late
// after every further failure (up to 65,536); and not even then while the whole-list walk of the round before shows that
// a window would have been too short again (a failed attempt costs the window's whole Gram: 5 ms on c5, 28 rounds' worth).
__device__ __forceinline__ bool window_skipped(const Problem& p) {
  const DeviceState* st = p.st;
  if (!st->prefer_walk) return false;
  if (st->window_hopeless) return true;                  // (the last round's walk says a window would have been too short again)
  const unsigned long long period = 64ull << min(max(st->walk_streak - 1, 0), 10);
  return ((st->round / (unsigned)p.part_count) & (period - 1ull)) != 0ull;
}


// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) and the FP32 race key.
// The key is a fixed sequence of correctly rounded binary32 operations (explicit _rn intrinsics,
// never contracted), so that any IEEE implementation of the same sequence agrees bit for bit.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const unsigned long long p0 = (unsigned long long)0xD2511F53u * c0, p1 = (unsigned long long)0xCD9E8D57u * c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0, hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

__device__ __forceinline__ float two_atanh_rn(float s) {
  const float z = __fmul_rn(s, s);
  float p = __uint_as_float(0x3d70f0f1u);                       // 1/17
  p = __fmaf_rn(p, z, __uint_as_float(0x3d888889u));            // 1/15
  p = __fmaf_rn(p, z, __uint_as_float(0x3d9d89d9u));            // 1/13
  p = __fmaf_rn(p, z, __uint_as_float(0x3dba2e8cu));            // 1/11
  p = __fmaf_rn(p, z, __uint_as_float(0x3de38e39u));            // 1/9
  p = __fmaf_rn(p, z, __uint_as_float(0x3e124925u));            // 1/7
  p = __fmaf_rn(p, z, __uint_as_float(0x3e4ccccdu));            // 1/5
  p = __fmaf_rn(p, z, __uint_as_float(0x3eaaaaabu));            // 1/3
  const float r = __fmul_rn(z, p);
  const float s2 = __fadd_rn(s, s);
  return __fmaf_rn(s2, r, s2);
}

// Unit exponential E = -ln(1 - v), v = (x + 1/2) / 2^32.
__device__ __forceinline__ float unit_exponential_rn(uint32_t x) {
  const float xf = __uint2float_rn(x);
  float v = __fmaf_rn(xf, __uint_as_float(0x2f800000u), __uint_as_float(0x2f000000u));
  const float vmax = __uint_as_float(0x3f7fffffu);
  if (v > vmax) v = vmax;
  if (v <= 0.5f) {
    const float s = __fdiv_rn(v, __fsub_rn(2.0f, v));
    return two_atanh_rn(s);
  }
  const float q = __fsub_rn(1.0f, v);
  const uint32_t qb = __float_as_uint(q);
  int e = (int)(qb >> 23) - 127;
  float m = __uint_as_float((qb & 0x007fffffu) | 0x3f800000u);
  if (m >= __uint_as_float(0x3fb504f3u)) { m = __fmul_rn(m, 0.5f); e += 1; }
  const float s = __fdiv_rn(__fsub_rn(m, 1.0f), __fadd_rn(m, 1.0f));
  const float a = two_atanh_rn(s);
  const float ef = __int2float_rn(e);
  const float lo = __fmaf_rn(ef, __uint_as_float(0x3805fdf4u), a);
  const float lnq = __fmaf_rn(ef, __uint_as_float(0x3f317000u), lo);
  return -lnq;
}

// 64-bit ranking key of coefficient j: (bits of T_j) << 32 | j, T_j = E_j / (delta_j^2 + eta).
// All keys are distinct; ascending key order = ascending T, ties to the smaller j.
// `mode`: which importance distribution p(j) the flags ask for.
enum WeightMode { kWeightSquare = 0, kWeightAbs = 1, kWeightUniform = 2 };   // delta^2 + eta | |delta| + eta | 1
__host__ __device__ __forceinline__ int weight_mode_of(unsigned int flags) {
  return (flags & STRADS_FLAG_UNIFORM_DRAW) ? kWeightUniform : ((flags & STRADS_FLAG_ABS_WEIGHT) ? kWeightAbs : kWeightSquare);
}
__device__ __forceinline__ float priority_weight(float delta_j, float eta, int mode) {
  return mode == kWeightUniform ? 1.0f : (mode == kWeightAbs ? __fadd_rn(fabsf(delta_j), eta) : __fmaf_rn(delta_j, delta_j, eta));
}
__device__ __forceinline__ unsigned long long race_key_from(float E, float delta_j, float eta, uint32_t j, int mode) {
  const float T = __fdiv_rn(E, priority_weight(delta_j, eta, mode));
  return ((unsigned long long)__float_as_uint(T) << 32) | j;
}
__device__ __forceinline__ unsigned long long race_key64(float delta_j, float eta, uint32_t word, uint32_t j, int mode) {
  return race_key_from(unit_exponential_rn(word), delta_j, eta, j, mode);
}

// The race keys coefficient j has in this scheduler's next round with its priority before (d_old) and after (d_new)
// an update: what k_sample_patch needs to correct a draw made ahead of the update.
// (In two steps, because the unit exponential does not depend on the priorities: it can be had before the update.)
__device__ __forceinline__ float next_round_exponential(const Problem& p, uint32_t j) {
  const unsigned long long t = p.st->round + (unsigned long long)p.part_count;
  uint32_t w[4];
  philox4x32_10(j >> 2, (uint32_t)t, (uint32_t)(t >> 32), 0u, (uint32_t)p.seed, (uint32_t)(p.seed >> 32), w);
  const uint32_t word = (j & 2u) ? ((j & 1u) ? w[3] : w[2]) : ((j & 1u) ? w[1] : w[0]);
  return unit_exponential_rn(word);
}
__device__ __forceinline__ void next_round_keys(const Problem& p, uint32_t j, float d_old, float d_new,
                                                unsigned long long* key_old, unsigned long long* key_new) {
  const int mode = weight_mode_of(p.flags);
  const float E = next_round_exponential(p, j);
  *key_old = race_key_from(E, d_old, p.eta, j, mode);
  *key_new = race_key_from(E, d_new, p.eta, j, mode);
}

// ||x_j||^2 as the dependency check (SAP step 2) sees it.  With STRADS_FLAG_DYNAMIC_DEPS a coefficient that is zero
// and whose last update left it there couples with nobody: it gets 0 here, and every Gram kernel already treats a
// pair with a zero column as free of conflict.
__device__ __forceinline__ double coupling_n2(const Problem& p, int j) {
  if ((p.flags & STRADS_FLAG_DYNAMIC_DEPS) && p.beta[j] == 0.f && p.delta[j] == 0.f) return 0.0;
  return p.n2[j];
}

// The two losses.  Squared loss: resid = y - X beta, the step of Eq. 2.  Logistic loss (STRADS_FLAG_LOGISTIC): resid =
// y - sigma(margin), and the second derivative of the loss along x_j is at most n_j / 4, which scales the step and its
// threshold by 4 (Shotgun's step for this loss).
__device__ __forceinline__ double step_scale(const Problem& p) { return (p.flags & STRADS_FLAG_LOGISTIC) ? 4.0 : 1.0; }
__device__ __forceinline__ double sigmoid64(double m) { return m >= 0.0 ? 1.0 / (1.0 + exp(-m)) : exp(m) / (1.0 + exp(m)); }
// Row i after the kept coefficients have moved the linear predictor x_i^T beta by s.
__device__ __forceinline__ void apply_row(const Problem& p, long long i, double s) {
  if (p.flags & STRADS_FLAG_LOGISTIC) {
    const float m = (float)((double)p.margin[i] + s);
    p.margin[i] = m;
    p.resid[i] = (float)((double)p.y[i] - sigmoid64((double)m));
  } else {
    p.resid[i] = (float)((double)p.resid[i] - s);
  }
}

// x_a^T x_b of two CSC columns (ascending rows): a given as arrays (possibly staged in shared memory), b read
// from X.  Products are added in row order, so every kernel that uses this gets the same bits.
__device__ __forceinline__ float sparse_dot(const int* ar, const float* av, int na, const Problem& p, int jb) {
  long long q = p.xptr[jb];
  const long long qe = p.xptr[jb + 1];
  float dot = 0.f;
  int i = 0;
  if (q < qe && na > 0) {
    int rb = __ldg(p.xrow + q), ra = ar[0];
    while (true) {
      if (ra == rb) {
        dot = fmaf(av[i], __ldg(p.xv + q), dot);
        if (++i >= na || ++q >= qe) break;
        ra = ar[i]; rb = __ldg(p.xrow + q);
      } else if (ra < rb) {
        if (++i >= na) break;
        ra = ar[i];
      } else {
        if (++q >= qe) break;
        rb = __ldg(p.xrow + q);
      }
    }
  }
  return dot;
}

// The same sum with both columns given as arrays (shared or global memory).  Every step loads both heads, adds the
// product if the rows match and advances whichever head is not ahead: no branch depends on the data, so the lanes of a
// warp, each merging a pair of its own, stay together (a three-way branch per step ran the warp through all three
// arms; the in-batch pairs of the on-demand walk took 18 us that way, 4 us this way).
__device__ __forceinline__ float sparse_dot_arrays(const int* ar, const float* av, int na, const int* br, const float* bv,
                                                   int nb) {
  float dot = 0.f;
  int i = 0, k = 0;
  while (i < na && k < nb) {
    const int ra = ar[i], rb = br[k];
    const float pa = av[i], pb = bv[k];
    dot = ra == rb ? fmaf(pa, pb, dot) : dot;
    i += ra <= rb;
    k += rb <= ra;
  }
  return dot;
}

// The same sum for a lane that holds column b (stored at q0, nb entries) in registers: its first kPre rows and values
// are fetched together, and every entry of column a is then compared with all of them.  No memory access and no branch
// depends on the data; the products are still added in row order (a's rows ascend, each matches at most one of b's).
// Entries of b beyond kPre are merged step by step.
template <int kPre>
__device__ __forceinline__ float sparse_dot_fetched(const int* ar, const float* av, int na, const Problem& p, long long q0, int nb) {
  int rb[kPre];
  float vb[kPre];
#pragma unroll
  for (int k = 0; k < kPre; ++k) {
    rb[k] = k < nb ? __ldg(p.xrow + q0 + k) : 0x7fffffff;
    vb[k] = k < nb ? __ldg(p.xv + q0 + k) : 0.f;
  }
  float dot = 0.f;
  if (nb <= kPre) {
    for (int i = 0; i < na; ++i) {
      const int ra = ar[i];
      const float va = av[i];
#pragma unroll
      for (int k = 0; k < kPre; ++k) dot = rb[k] == ra ? fmaf(va, vb[k], dot) : dot;
    }
    return dot;
  }
  return sparse_dot_arrays(ar, av, na, p.xrow + q0, p.xv + q0, nb);      // a long column: plain merge
}

// The same with column b fetched as aligned groups of four entries (16-byte loads; xv and xrow 16-byte aligned): a
// lane that merges a column of its own touches a cache line per load, and it is the number of such loads, not their
// size, that an SM can take per cycle.  The groups start at the aligned entry at or before q0 and cover
// (q0 mod 4) + nb <= 4 kVec entries; those outside the column count as absent.  A group that would reach past the
// last stored entry of the matrix is read entry by entry.
template <int kVec>
__device__ __forceinline__ float sparse_dot_fetched4(const int* ar, const float* av, int na, const Problem& p, long long q0, int nb) {
  const long long e0 = q0 & ~3ll;
  const int head = (int)(q0 - e0), need = head + nb;
  int rb[4 * kVec];
  float vb[4 * kVec];
#pragma unroll
  for (int v = 0; v < kVec; ++v) {
    int4 r = make_int4(0, 0, 0, 0);
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    const long long e = e0 + 4 * v;
    if (4 * v < need) {
      if (e + 4 <= p.nnz) {
        r = __ldg(reinterpret_cast<const int4*>(p.xrow + e));
        x = __ldg(reinterpret_cast<const float4*>(p.xv + e));
      } else {
        if (e < p.nnz) { r.x = __ldg(p.xrow + e); x.x = __ldg(p.xv + e); }
        if (e + 1 < p.nnz) { r.y = __ldg(p.xrow + e + 1); x.y = __ldg(p.xv + e + 1); }
        if (e + 2 < p.nnz) { r.z = __ldg(p.xrow + e + 2); x.z = __ldg(p.xv + e + 2); }
      }
    }
    const int i0 = 4 * v;
    rb[i0] = (i0 >= head && i0 < need) ? r.x : 0x7fffffff;             vb[i0] = x.x;
    rb[i0 + 1] = (i0 + 1 >= head && i0 + 1 < need) ? r.y : 0x7fffffff; vb[i0 + 1] = x.y;
    rb[i0 + 2] = (i0 + 2 >= head && i0 + 2 < need) ? r.z : 0x7fffffff; vb[i0 + 2] = x.z;
    rb[i0 + 3] = (i0 + 3 >= head && i0 + 3 < need) ? r.w : 0x7fffffff; vb[i0 + 3] = x.w;
  }
  float dot = 0.f;
  for (int i = 0; i < na; ++i) {
    const int ra = ar[i];
    const float va = av[i];
#pragma unroll
    for (int k = 0; k < 4 * kVec; ++k) dot = rb[k] == ra ? fmaf(va, vb[k], dot) : dot;
  }
  return dot;
}

// ---------------------------------------------------------------------------------------------
// Chained launches (programmatic dependent launch).  A round is a chain of short kernels, each needing the
// one before it, and the gap between two dependent launches is of the order of the kernels themselves.  A
// kernel launched with launch_chained may be scheduled while the kernel ahead of it in the stream still runs;
// chain_begin() is where it stops until that kernel has finished and its writes are visible, so it is the
// first statement of every kernel launched this way (nothing in global memory is touched before it).  It then
// lets the kernel behind it start in the same manner.  Since every link waits for its predecessor to finish,
// finishing is transitive along the chain.  Launched the ordinary way, chain_begin() does nothing.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void chain_begin() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// The same for a kernel whose CTAs form thread-block clusters of cluster_x consecutive blocks (1: no clusters).
template <typename... KArgs, typename... Args>
cudaError_t launch_chained_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, int cluster_x,
                                   Args&&... args) {
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = (unsigned)cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cfg.attrs = attr; cfg.numAttrs = cluster_x > 1 ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// ---------------------------------------------------------------------------------------------
// Launchers (one per step; all enqueue on `s` and return a cudaError_t).
// ---------------------------------------------------------------------------------------------
cudaError_t launch_init(const Problem& p, cudaStream_t s);
cudaError_t launch_resid_from_beta(const Problem& p, cudaStream_t s);
cudaError_t launch_init_scheduler(const Problem& p, const Problem& first, cudaStream_t s);   // after launch_init of `first`
cudaError_t launch_objective(const Problem& p, cudaStream_t s);
cudaError_t prepare_sample(const Problem& p);
cudaError_t launch_sample(const Problem& p, int* cand_out, cudaStream_t s);
// Candidates of the round at hand from a draw made one round ahead (`ahead`: its keys in rank order, ahead.n_cand of
// them) and the coefficients the last update changed (p.kept, p.delta_prev, p.delta).
// from_cand: before this round's update, from the keys the pack kernel formed for every candidate (p.kept_pos, p.cand_keys);
// gate: 0 always, 1 / 2 only on the branch DeviceState::route names (as launch_update).
cudaError_t launch_sample_patch(const Problem& p, const Problem& ahead, int* cand_out, cudaStream_t s, bool from_cand = false,
                                int gate = 0);
cudaError_t launch_gram_dense_simt(const Problem& p, const int* cand, int n_cand, float* gram_dbg, cudaStream_t s);
cudaError_t prepare_gram_dense_tc();
cudaError_t encode_gram_tensor_map(const Problem& p, void* out_128_bytes);
// `only_if_short`: the launch is the whole-list retry of a windowed round and does nothing unless the
// window's filter set DeviceState::window_short.
cudaError_t launch_gram_dense_tc(const Problem& p, const void* tmap, const int* cand, int n_cand, int n_total, bool only_if_short,
                                 bool fallback_elsewhere, cudaEvent_t after_pack, cudaStream_t s, bool* walked);
cudaError_t launch_gram_csc(const Problem& p, const int* cand, int n_cand, float* gram_dbg, bool only_if_short,
                            bool window, cudaStream_t s);
cudaError_t prepare_filter(const Problem& p);
// Walks cand[0 .. n_cand); n_total >= n_cand is the length of the whole list (n_cand < n_total: a window).
// CSC: greedy walk that forms conflict rows only for the candidates it is about to keep (cooperative kernel).
cudaError_t prepare_walk_csc(const Problem& p, int* grid_out);
cudaError_t launch_walk_csc(const Problem& p, const int* cand, int n_cand, int window, int grid, bool only_if_short, int* kept_out,
                            cudaStream_t s);
// only_if_pending: the launch follows a window Gram whose last CTA walks; it does nothing unless that CTA left the
// walk to it (DeviceState::walk_pending).
cudaError_t launch_filter(const Problem& p, const int* cand, int n_cand, int n_total, bool only_if_short, int* kept_out,
                          cudaStream_t s, bool only_if_pending = false);
cudaError_t launch_update(const Problem& p, const int* kept, int advance, bool after_pack, cudaStream_t s, int gate = 0);
cudaError_t launch_set_counts(const Problem& p, int n_cand, int n_examined, int n_kept, cudaStream_t s);
cudaError_t launch_export(const Problem& p, const int* kept, int* kept_out, float* dbeta_out, int* counts_out,
                          cudaStream_t s);

}  // namespace strads
