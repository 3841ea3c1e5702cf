// SAP step 2, dense X, on the 5th-generation tensor cores: conflict bits of all candidate pairs from
// G = X_C^T X_C, a genuine dense contraction (M = N' = P', K = the N samples).
//
//   k_pack_candidates   writes the P' candidate columns, rounded to BF16, into one contiguous [P'][ldcb]
//                       buffer: the screen's operands.  The candidates are scattered over the whole design
//                       matrix (one 2 MB page each for a 4 GB X); gathering them once makes every later
//                       access TLB- and TMA-friendly (measured: the same GEMM runs 2x slower straight
//                       from scattered columns).  With one scheduler it also forms x_c^T r on the way.
//   k_gram_dense_tc<0>  "screen": one CTA per 128 x 128 tile of the upper triangle of tile pairs; one
//                       thread feeds a 3-stage ring of 64 KB stages with TMA tile loads of the BF16 copy
//                       (128-byte swizzle, zero fill past N and P'), one thread issues tcgen05.mma
//                       kind::f16 into a 128 x 128 FP32 accumulator in tensor memory, four warps read
//                       it back with tcgen05.ld, threshold in FP64 and write mask words.  The kernel is
//                       bound by bringing operands from L2 to shared memory, so half-width operands
//                       halve its main loop; the screen only has to be right about the pairs it calls:
//                       a BF16 correlation is within 2^-8 of the exact one whatever the data, so pairs
//                       further than the band from rho are decided for certain; the few inside the band
//                       go to a list ...
//   k_gram_recheck      ... and are decided exactly (FP64 dot product), so the decisions equal those of
//                       an exact Gram.
//   k_gram_dense_tc<1>  3xTF32 fallback, runs only if that list overflows (or on request): producer
//                       warps copy with cp.async and split every operand into hi + lo TF32 parts,
//                       G ~= lo.hi + hi.lo + hi.hi.
//
// Every wait has an iteration limit; on expiry the CTA raises STRADS_STATUS_WAIT_EXPIRED, stops issuing
// work, and still frees its tensor memory.  No multicast anywhere.
#include <cuda.h>
#include <cuda_bf16.h>

#include "strads_internal.cuh"
#include "walk_pairs.cuh"

namespace strads {
namespace {

constexpr int kTile = 128;                 // rows and columns of the output tile
constexpr int kBlockK = 32;                // floats of K per sub-block = one 128-byte swizzle row
constexpr int kTileBytes = kTile * 128;    // 16 KB: 128 rows x 128 bytes
constexpr int kProducerWarps = 4;          // epilogue warps; also the cp.async producers of the 3xTF32 variant
constexpr int kMmaWarp = 4, kTmaWarp = 5;
constexpr int kThreads = 32 * 6;
constexpr uint32_t kWaitLimit = 1u << 24;
constexpr uint32_t kTmemCols = 128;
constexpr size_t kRingBytes = 192 * 1024;
constexpr size_t kDynSmem = kRingBytes + 1024;
// Half-width of the "too close to call" band of the screen, relative to ||x_a|| ||x_b||.  The screen multiplies
// BF16 roundings of the columns: each operand is off by at most 2^-9 relative (8 significand bits, round to nearest),
// so the sum of products by at most 2^-8 (1 + 2^-10) ||x_a|| ||x_b|| (Cauchy-Schwarz); the FP32 accumulator updates
// add at most 2^-24 each over N / 16 steps.  Doubled for margin.
__device__ __forceinline__ double screen_band(long long N) { return 1.0 / 128.0 + (double)N * (1.0 / 33554432.0); }
constexpr int kScreenK = 64;               // BF16 elements of K per sub-block of the screen = one 128-byte swizzle row

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One TMA tile load: box {64 BF16 elements, 128 rows} at element coordinates (x = k, y = row) -> shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar) : "memory");
}
// Bounded wait for the phase with the given parity; false = gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4)        // start address / 16
         | ((uint64_t)1 << 16)                       // leading byte offset / 16 (unused for swizzled K-major)
         | ((uint64_t)(1024 >> 4) << 32)             // stride byte offset / 16
         | ((uint64_t)1 << 46)                       // descriptor version of this architecture
         | ((uint64_t)2 << 61);                      // 128-byte swizzle
}

// D[tmem] (+)= A[smem] * B[smem]^T, TF32 inputs, FP32 accumulate, M = N = 128, K = 8.
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// The same with BF16 inputs, K = 16.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 16 bytes global -> shared, asynchronously; only the first `bytes` (0, 4, 8, 12 or 16) are read, the rest is zero.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// x = hi + lo with hi the top 11 significand bits of x (what a TF32 MMA reads of x); lo again cut to TF32.
__device__ __forceinline__ float tf32_lo(float x) {
  const float hi = __uint_as_float(__float_as_uint(x) & 0xffffe000u);
  return __uint_as_float(__float_as_uint(x - hi) & 0xffffe000u);
}

// 32 Gram values of row a against columns b0 .. b0 + 31 -> conflict bits.  Screen mode leaves the pairs
// inside the band undecided (bit clear) and appends them to the list k_gram_recheck works through.
template <bool kScreen>
__device__ __forceinline__ uint32_t decide_word(const Problem& p, const uint32_t (&v)[32], int a, int b0, int n_cand,
                                                double norm_a, const double* norm_b, double rho, double band) {
  uint32_t word = 0u;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int b = b0 + j;
    const double den = norm_a * norm_b[j];
    const double g = fabs((double)__uint_as_float(v[j]));
    const bool live = a < n_cand && b < n_cand && a != b && den > 0.0;
    bool hit = live && g >= rho * den;
    if (kScreen && live && b > a && fabs(g - rho * den) <= band * den) {
      hit = false;
      const unsigned int slot = atomicAdd(&p.st->amb_count, 1u);
      if (slot < (unsigned)p.cap_amb) p.amb_pairs[slot] = ((unsigned int)a << 16) | (unsigned int)b;
    }
    if (hit && b > a) list_conflict(p, a, b);
    word |= (uint32_t)hit << j;
  }
  return word;
}

// acc += x * r with acc = hi + lo a pair of floats: the product's rounding error (one fma) and the sum's (two-sum)
// are both exact and collected in lo, so the pair carries about 2^-46 of the summed magnitudes -- FP64-grade
// accumulation on the FP32 pipe, where conversions to double would cost more than the copy they ride on.
// Explicitly rounded operations only: the sequence is the same bits everywhere.
__device__ __forceinline__ void dot_step(float x, float r, float& hi, float& lo) {
  const float pr = __fmul_rn(x, r);
  const float pe = __fmaf_rn(x, r, -pr);
  const float s = __fadd_rn(hi, pr);
  const float bb = __fsub_rn(s, hi);
  const float se = __fadd_rn(__fsub_rn(hi, __fsub_rn(s, bb)), __fsub_rn(pr, bb));
  hi = s;
  lo = __fadd_rn(lo, __fadd_rn(se, pe));
}

// Four consecutive elements of a packed column, rounded to BF16 (nearest even), as one 8-byte store.
__device__ __forceinline__ void store_bf16x4(unsigned short* row, long long g, const float4& v) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 w;
  w.x = *reinterpret_cast<const unsigned int*>(&lo);
  w.y = *reinterpret_cast<const unsigned int*>(&hi);
  reinterpret_cast<uint2*>(row)[g] = w;
}

constexpr int kPackStream = 256;                 // threads that copy (and multiply) the column
constexpr int kPackThreads = kPackStream + 32;   // + one warp with no streaming work, for the next round's keys

// One CTA per candidate at a time: xcb[a][0 .. ldc) = column cand[a] of X rounded to BF16.  With p.proposals the column is
// also multiplied into the residual as it streams by (fixed order: per-thread strided sums, lanes by shuffle
// tree, warps in index order) and the candidate's would-be update follows from it at once (Eq. 2): the update
// step then only has to apply the proposals of the kept candidates.
__device__ __forceinline__ void pack_candidate(const Problem& p, const int* __restrict__ cand, int a) {
  const int j = cand[a];
  const float4* src = reinterpret_cast<const float4*>(p.xv + (long long)j * p.ld);
  const long long n4 = p.ldc >> 2;                      // ldc = N rounded up to 4 <= ld
  unsigned short* dstb = p.xcb + (long long)a * p.ldcb;   // (ldcb >= ldc: every group of four has its place)
  if (!p.proposals) {
    for (long long g = threadIdx.x; g < n4; g += blockDim.x) {
      store_bf16x4(dstb, g, __ldg(src + g));
    }
    return;
  }
  const float4* r4 = reinterpret_cast<const float4*>(p.resid);
  const long long n4_full = p.N >> 2;                   // float4 groups that lie wholly inside the N rows
  double n = 0.0;
  float b_old = 0.f;
  if (threadIdx.x == 0) { n = p.n2[j]; b_old = p.beta[j]; }   // two far gathers, under way while the column streams
  // the candidate's unit exponential of the next round and its key with the present priority, by a thread of the
  // warp that streams nothing (~600 dependent instructions: in a streaming warp they would hold up its loads); the
  // key with the new priority follows from the change, at the end
  __shared__ float s_E;
  if (threadIdx.x == kPackStream && p.patch_keys != nullptr) {
    s_E = next_round_exponential(p, (uint32_t)j);
    p.cand_keys[a] = race_key_from(s_E, p.delta[j], p.eta, (uint32_t)j, weight_mode_of(p.flags));
  }
  float h0 = 0.f, l0 = 0.f, h1 = 0.f, l1 = 0.f;
  constexpr int kU = 4;                                 // column loads in flight per thread
  const long long first = threadIdx.x < kPackStream ? (long long)threadIdx.x : n4;      // (the extra warp: no trips)
  for (long long g0 = first; g0 < n4; g0 += (long long)kU * kPackStream) {
    float4 xv[kU], rv[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const long long g = g0 + (long long)u * kPackStream;
      xv[u] = g < n4 ? __ldg(src + g) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const long long g = g0 + (long long)u * kPackStream;
      if (g < n4_full) {
        rv[u] = r4[g];
      } else if (g < n4) {                              // the last, partial group: rows past N do not exist
        const long long i = g << 2;
        rv[u].x = p.resid[i];
        rv[u].y = i + 1 < p.N ? p.resid[i + 1] : 0.f;
        rv[u].z = i + 2 < p.N ? p.resid[i + 2] : 0.f;
        rv[u].w = 0.f;
      } else {
        rv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const long long g = g0 + (long long)u * kPackStream;
      if (g < n4) store_bf16x4(dstb, g, xv[u]);
      if (g >= n4_full) {                               // padding of the column (and groups past the end) stay out of the sum
        const long long i = g << 2;
        if (i >= p.N) xv[u].x = 0.f;
        if (i + 1 >= p.N) xv[u].y = 0.f;
        if (i + 2 >= p.N) xv[u].z = 0.f;
        xv[u].w = 0.f;
      }
      dot_step(xv[u].x, rv[u].x, h0, l0); dot_step(xv[u].y, rv[u].y, h1, l1);
      dot_step(xv[u].z, rv[u].z, h0, l0); dot_step(xv[u].w, rv[u].w, h1, l1);
    }
  }
  __shared__ double wsum[8];
  double v = ((double)h0 + (double)l0) + ((double)h1 + (double)l1);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0 && threadIdx.x < kPackStream) wsum[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    double g = 0.0;
    for (int w = 0; w < kPackStream / 32; ++w) g += wsum[w];
    float b_new = b_old;
    if (n > 0.0) {
      const double c = step_scale(p);
      const double z = (double)b_old + c * g / n;
      const double m = fabs(z) - c * (double)p.lambda / n;
      b_new = (float)(m <= 0.0 ? 0.0 : (z > 0.0 ? m : -m));
    }
    const double d = isfinite(g) ? (double)b_new - (double)b_old : g - g;      // a non-finite product shows as NaN
    p.cand_bnew[a] = b_new;
    p.cand_dbeta64[a] = d;
    if (p.patch_keys != nullptr)
      p.cand_keys[p.n_cand + a] = race_key_from(s_E, (float)fabs(d), p.eta, (uint32_t)j, weight_mode_of(p.flags));
  }
}

// The CTAs take the candidates in turn (the window's launch has one CTA per candidate; the whole-list retry, which
// normally returns at once, a grid of a few CTAs per SM, so that an idle launch costs little).
__global__ void __launch_bounds__(kPackThreads) k_pack_candidates(Problem p, const int* __restrict__ cand, int n_cand,
                                                         int only_if_short) {
  chain_begin();
  if (only_if_short && !p.st->window_short) return;
  for (int a = blockIdx.x; a < n_cand; a += gridDim.x) {
    pack_candidate(p, cand, a);
    __syncthreads();                                    // (the shared words of one candidate are reused by the next)
  }
}

// Exact decision for one pair the screen could not call, by a whole warp: FP64 dot product of the two columns of X.  Setting a bit is idempotent and order-independent, so the result is deterministic.
__device__ __forceinline__ void recheck_pair(const Problem& p, unsigned int pr, int lane) {
  const long long n4 = (p.N + 3) >> 2;
  const int a = (int)(pr >> 16), b = (int)(pr & 0xffffu);
  const float4* xa = reinterpret_cast<const float4*>(p.xv + (long long)p.cand_cur[a] * p.ld);
  const float4* xb = reinterpret_cast<const float4*>(p.xv + (long long)p.cand_cur[b] * p.ld);
  double acc = 0.0;
  for (long long g = lane; g < n4; g += 32) {
    const float4 u = xa[g], w = xb[g];
    const long long i = g << 2;
    acc += (double)u.x * w.x;
    if (i + 1 < p.N) acc += (double)u.y * w.y;
    if (i + 2 < p.N) acc += (double)u.z * w.z;
    if (i + 3 < p.N) acc += (double)u.w * w.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    const double den = sqrt(coupling_n2(p, p.cand_cur[a])) * sqrt(coupling_n2(p, p.cand_cur[b]));
    if (den > 0.0 && fabs(acc) >= (double)p.rho * den) {
      atomicOr(&p.conflict[(long long)a * p.mask_words + (b >> 5)], 1u << (b & 31));
      list_conflict(p, a, b);
    }
  }
}

// What follows the window's Gram on the round's path, done by the CTA of the Gram kernel that finishes last
// instead of by launches of their own:
//   - the pairs the screen left open, normally a handful or none, are decided exactly.  "Few" is a budget of
//     multiply-adds for this one CTA (2^21, some tens of microseconds at worst): short columns leave many pairs
//     open (their correlations scatter widely around rho) but each is cheap, long columns hardly any.  Beyond the
//     budget the window is handed to the whole-list retry, whose Gram has a recheck kernel of its own;
//   - the greedy first-fit walk is settled from the list of conflicting pairs; if that list is incomplete or the
//     chains of dependent decisions are too long, the walk kernel behind this one does it from the bit rows
//     (walk_pending), otherwise that kernel returns at once.
// DeviceState::route tells the update which of its two gated copies runs: 0 the one behind this kernel, 1 the one
// at the end of the branch that holds the walk kernel and the whole-list retry.
constexpr unsigned int kInlineRecheck = 4096;
constexpr long long kInlineRecheckWork = 1ll << 21;
__device__ void window_tail(const Problem& p, const int* __restrict__ cand, int n_cand, int n_total, unsigned char* sm) {
  __shared__ int s_last, s_kept, s_examined;
  DeviceState* st = p.st;
  const int tid = threadIdx.x;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&st->gram_ticket, 1u) == gridDim.x - 1u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const unsigned int n_amb = __ldcg(&st->amb_count);
  if (n_amb > (unsigned)p.cap_amb || n_amb > kInlineRecheck || (long long)n_amb * p.N > kInlineRecheckWork) {
    if (tid == 0) {                                      // the whole-list retry takes over (it has the 3xTF32 fallback)
      st->gram_ticket = 0u; st->window_short = 1; st->route = 1; st->walk_pending = 0;
      st->amb_count = 0; st->edge_count = 0; st->edges_off = 0;
    }
    return;
  }
  for (unsigned int e = tid >> 5; e < n_amb; e += blockDim.x >> 5) recheck_pair(p, __ldcg(p.amb_pairs + e), tid & 31);
  if (tid == 0) { s_kept = 0; s_examined = n_cand; }
  __syncthreads();
  const unsigned int n_edges = __ldcg(&st->edge_count);
  bool settled = false;
  if (!st->edges_off && n_edges <= (unsigned)p.cap_edges && walk_pairs_smem(n_cand, n_edges) <= kRingBytes)
    settled = walk_from_pair_list<kThreads>(p, cand, n_cand, n_edges, sm, p.kept, &s_kept, &s_examined);
  if (!settled) {
    if (tid == 0) {
      st->gram_ticket = 0u; st->walk_pending = 1; st->route = 1;
    }
    return;
  }
  const int nk = s_kept;
  for (int i = nk + tid; i < p.n_keep; i += blockDim.x) p.kept[i] = -1;
  if (tid == 0) {
    st->gram_ticket = 0u;
    st->counts[1] = s_examined; st->counts[2] = nk; st->counts[3] = 0; st->amb_count = 0;
    st->edge_count = 0; st->edges_off = 0;               // the next Gram starts a new list
    const int short_ = (nk < p.n_keep && n_cand < n_total) ? 1 : 0;
    st->window_short = short_; st->route = short_; st->walk_pending = 0;
  }
}

// n_split > 1: the launch is made of thread-block clusters of n_split CTAs that share one output tile, each taking
// a slice of K (a window of few tiles would otherwise use few SMs); the partial tiles are combined through
// distributed shared memory, in split order.  tail: 0 none; 1 the CTA of the grid that finishes last rechecks the
// pairs the screen left open and settles the greedy walk from the list of conflicting pairs (window_tail).
template <bool k3x>
__global__ void __launch_bounds__(kThreads, 1) k_gram_dense_tc(Problem p, const __grid_constant__ CUtensorMap tmap,
                                                                int n_cand, int n_total, int n_tiles, int n_split, int only_if_short,
                                                                int tail) {
  chain_begin();
  // A stage holds kSub sub-blocks of 32 floats of K for A, the same for B [3xTF32: plus the two lo tiles].
  constexpr int kSub = k3x ? 1 : 2;
  constexpr int kStageBytes = (k3x ? 4 : 2 * kSub) * kTileBytes;       // 64 KB either way
  constexpr int kStages = (int)(kRingBytes / kStageBytes);             // 3
  constexpr int kAhead = kStages - 1;                                  // 3xTF32: stages in flight per producer thread
  constexpr uint32_t kFullCount = k3x ? kProducerWarps : 1;            // arrivals that complete "full"

  extern __shared__ unsigned char dyn_smem[];
  __shared__ __align__(8) unsigned long long bars[2 * kStages + 1];   // full[], empty[], accumulator done
  __shared__ uint32_t s_tmem_base;
  __shared__ volatile int s_abort;
  __shared__ double normA[kTile], normB[kTile];                        // ||x|| of the tile's rows / columns

  if (only_if_short && !p.st->window_short) return;
  // as a fallback the 3xTF32 variant runs only when the screen's list overflowed
  if (k3x && !(p.flags & STRADS_FLAG_GRAM_3XTF32) && p.st->amb_count <= (unsigned)p.cap_amb) return;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t wait_limit = p.wait_limit ? p.wait_limit : kWaitLimit;
  if (k3x && !(p.flags & STRADS_FLAG_GRAM_3XTF32) && blockIdx.x == 0 && tid == 0)
    atomicOr(&p.st->status, STRADS_STATUS_GRAM_FALLBACK);
  // With n_split > 1 the K range of a tile is shared by the n_split CTAs of a cluster (consecutive block indices), one
  // tile per cluster.  Without a split the CTAs take the tiles in turn (a grid of at most one CTA per SM: a launch
  // that has nothing to do -- the whole-list retry of a round whose window sufficed -- then costs one wave of CTAs, not
  // one per tile); the ring's stages and the barriers' phases simply run on from tile to tile.
  const int split = blockIdx.x % n_split;
  const int tile_first = blockIdx.x / n_split, tile_step = gridDim.x / n_split;
  const int tiles_total = n_tiles * (n_tiles + 1) / 2;

  const uint32_t tiles0 = (smem_u32(dyn_smem) + 1023u) & ~1023u;      // swizzle atoms need 1024-byte alignment
  unsigned char* tiles_ptr = dyn_smem + (tiles0 - smem_u32(dyn_smem));
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[kStages]), done_bar = smem_u32(&bars[2 * kStages]);

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8 * s, kFullCount); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(done_bar, 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {                              // the MMA warp owns the tensor-memory allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = s_tmem_base;

  const long long N = p.N;
  constexpr int kBK = k3x ? kBlockK : kScreenK;        // elements of K per sub-block (128 bytes either way)
  const int n_st_all = (int)((N + (long long)kBK * kSub - 1) / ((long long)kBK * kSub));   // stages of K
  const int per_split = (n_st_all + n_split - 1) / n_split;
  const int st_first = min(n_st_all, split * per_split);
  const int n_st = min(n_st_all, st_first + per_split) - st_first;     // this CTA's stages per tile (may be 0)

  int iter = 0;
  for (int tile = tile_first; tile < tiles_total; tile += tile_step, ++iter) {
  const int g0 = iter * n_st;                          // stages this CTA has put through the ring before this tile
  int ti = 0, rem = tile;                              // linear index -> (ti, tj), ti <= tj
  while (rem >= n_tiles - ti) { rem -= n_tiles - ti; ++ti; }
  const int tj = ti + rem;

  if (!k3x && warp == kTmaWarp) {
    // ------------------------------ screen: TMA producer (one lane) ------------------------------
    for (int st = 0; st < n_st; ++st) {
      const int g = g0 + st, s = g % kStages;
      bool got = !s_abort;
      if (got && g >= kStages) got = mbar_wait(empty0 + 8 * s, (uint32_t)(g / kStages - 1) & 1u, wait_limit);
      if (!__all_sync(0xffffffffu, got)) {
        if (lane == 0) { s_abort = 1; atomicOr(&p.st->status, STRADS_STATUS_WAIT_EXPIRED); }
        break;
      }
      if (lane == 0 && !p.stall) {                     // (stall: the loads are withheld and the MMA warp's wait runs out)
        const uint32_t sb = tiles0 + (uint32_t)s * kStageBytes, bar = full0 + 8 * s;
        mbar_arrive_expect_tx(bar, (uint32_t)kStageBytes);
#pragma unroll
        for (int sub = 0; sub < kSub; ++sub) {
          const int k = ((st_first + st) * kSub + sub) * kBK;        // past N the whole box is zero-filled
          tma_load_2d(sb + sub * kTileBytes, &tmap, k, ti * kTile, bar);
          tma_load_2d(sb + (kSub + sub) * kTileBytes, &tmap, k, tj * kTile, bar);
        }
      }
      __syncwarp();
    }
  } else if (k3x && warp < kProducerWarps) {
    // ------------------------------ 3xTF32: cp.async producers that also split hi / lo ------------------------------
    const int chunk = lane & 7;                        // which 16 bytes of the 128-byte row
    const int rsub = lane >> 3;                        // 4 rows per warp-wide copy
    const float* srcA[8];
    const float* srcB[8];
    uint32_t dst_off[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = warp * 32 + i * 4 + rsub;
      const int ga = ti * kTile + row, gb = tj * kTile + row;
      srcA[i] = ga < n_cand ? p.xv + (long long)p.cand_cur[ga] * p.ld : nullptr;   // (straight from X: the fallback is rare)
      srcB[i] = gb < n_cand ? p.xv + (long long)p.cand_cur[gb] * p.ld : nullptr;
      dst_off[i] = (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4));
    }
    auto issue = [&](int st) {                         // all copies of one stage
      const uint32_t sb = tiles0 + (uint32_t)((g0 + st) % kStages) * kStageBytes;
      const long long k = (long long)(st_first + st) * kBlockK + chunk * 4;
      const long long left = N - k;                    // floats of this chunk that exist
      const uint32_t bytes = left >= 4 ? 16u : (left > 0 ? (uint32_t)left * 4u : 0u);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        cp_async16(sb + dst_off[i], srcA[i] ? (const void*)(srcA[i] + (bytes ? k : 0)) : (const void*)p.xv,
                   srcA[i] ? bytes : 0u);
        cp_async16(sb + kTileBytes + dst_off[i], srcB[i] ? (const void*)(srcB[i] + (bytes ? k : 0)) : (const void*)p.xv,
                   srcB[i] ? bytes : 0u);
      }
    };
    for (int st = 0; st < kAhead; ++st) {              // prologue: the ring is empty (the last tile is all done), fill kAhead stages
      if (st < n_st) issue(st);
      cp_async_commit();
    }
    for (int st = 0; st < n_st; ++st) {
      const int s = (g0 + st) % kStages;
      cp_async_wait<kAhead - 1>();                     // this thread's copies of stage st have landed
      unsigned char* sp = tiles_ptr + (size_t)s * kStageBytes;
#pragma unroll
      for (int i = 0; i < 8; ++i) {                    // the raw tile stays as "hi", write the "lo" tiles
        float4 a = *reinterpret_cast<const float4*>(sp + dst_off[i]);
        float4 b = *reinterpret_cast<const float4*>(sp + kTileBytes + dst_off[i]);
        a.x = tf32_lo(a.x); a.y = tf32_lo(a.y); a.z = tf32_lo(a.z); a.w = tf32_lo(a.w);
        b.x = tf32_lo(b.x); b.y = tf32_lo(b.y); b.z = tf32_lo(b.z); b.w = tf32_lo(b.w);
        *reinterpret_cast<float4*>(sp + 2 * kTileBytes + dst_off[i]) = a;
        *reinterpret_cast<float4*>(sp + 3 * kTileBytes + dst_off[i]) = b;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(full0 + 8 * s);      // release: this warp's part of the stage is ready
      const int nxt = st + kAhead;                     // refill the stage that st - 1 used
      if (nxt < n_st) {
        bool got = !s_abort;
        const int gn = g0 + nxt;
        if (got && gn >= kStages) got = mbar_wait(empty0 + 8 * (gn % kStages), (uint32_t)(gn / kStages - 1) & 1u, wait_limit);
        if (!__all_sync(0xffffffffu, got)) {
          if (lane == 0) { s_abort = 1; atomicOr(&p.st->status, STRADS_STATUS_WAIT_EXPIRED); }
          break;
        }
        issue(nxt);
      }
      cp_async_commit();
    }
    cp_async_wait<0>();
  } else if (warp == kMmaWarp) {
    // ------------------------------ MMA issuer (whole warp waits, one lane issues) ------------------------------
    // instruction descriptor: FP32 accumulator; A and B both TF32 (3xTF32) or both BF16 (screen), K-major; N, M
    constexpr uint32_t kFmt = k3x ? 2u : 1u;
    const uint32_t idesc = (1u << 4) | (kFmt << 7) | (kFmt << 10) | ((uint32_t)(kTile >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
    uint32_t acc = 0;
    for (int st = 0; st < n_st; ++st) {
      const int s = (g0 + st) % kStages;
      const uint32_t ph = (uint32_t)((g0 + st) / kStages) & 1u;
      const bool got = !s_abort && mbar_wait(full0 + 8 * s, ph, wait_limit);
      if (!__all_sync(0xffffffffu, got)) {
        if (lane == 0) { s_abort = 1; atomicOr(&p.st->status, STRADS_STATUS_WAIT_EXPIRED); }
        break;
      }
      // 3xTF32 only: its tiles were written through the generic proxy (cp.async, st.shared) by the producers;
      // the acquire above made them visible to this thread, this fence orders them before the MMA's reads.
      // (Fencing here and not in the producers: a producer's fence would also wait for its copies in flight.)
      if (k3x) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (lane == 0) {
        const uint32_t sb = tiles0 + (uint32_t)s * kStageBytes;
#pragma unroll
        for (int k8 = 0; k8 < kSub * kBlockK / 8; ++k8) {   // 32 bytes of K per instruction (8 TF32 / 16 BF16) along the swizzled row
          const int sub = k8 / (kBlockK / 8);
          const uint64_t a_hi = umma_desc(sb + sub * kTileBytes), b_hi = umma_desc(sb + (kSub + sub) * kTileBytes);
          const uint64_t o = (uint64_t)((k8 % (kBlockK / 8)) * 2);
          if (k3x) {
            const uint64_t a_lo = umma_desc(sb + 2 * kTileBytes), b_lo = umma_desc(sb + 3 * kTileBytes);
            umma_tf32(tmem_base, a_lo + o, b_hi + o, idesc, acc);
            umma_tf32(tmem_base, a_hi + o, b_lo + o, idesc, 1u);
            umma_tf32(tmem_base, a_hi + o, b_hi + o, idesc, 1u);
          } else {
            umma_bf16(tmem_base, a_hi + o, b_hi + o, idesc, acc);
          }
          acc = 1;
        }
        umma_commit(empty0 + 8 * s);                   // frees the stage when these MMAs have read it
      }
      __syncwarp();
    }
    if (lane == 0) umma_commit(done_bar);              // accumulator complete
    __syncwarp();
  }

  // ------------------------------ epilogue (warps 0..3: TMEM lanes 32 w .. 32 w + 31) ------------------------------
  if (warp < kProducerWarps) {                           // (screen: while the main loop runs) the norms of the tile
    const int ga = ti * kTile + tid, gb = tj * kTile + tid;
    normA[tid] = ga < n_cand ? sqrt(coupling_n2(p, p.cand_cur[ga])) : 0.0;
    normB[tid] = gb < n_cand ? sqrt(coupling_n2(p, p.cand_cur[gb])) : 0.0;
    asm volatile("bar.sync 1, 128;" ::: "memory");       // the four epilogue warps see all of them
  }
  const double rho = (double)p.rho;
  const double band = screen_band(N);
  if (n_split == 1) {
    if (warp < kProducerWarps) {
      bool ok = !s_abort && mbar_wait(done_bar, (uint32_t)iter & 1u, wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok && lane == 0) { s_abort = 1; atomicOr(&p.st->status, STRADS_STATUS_WAIT_EXPIRED); }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (ok) {
        const int la = warp * 32 + lane;
        const int a = ti * kTile + la;
        const double norm_a = normA[la];
#pragma unroll 1
        for (int c = 0; c < kTile / 32; ++c) {
          uint32_t v[32];
          tmem_load32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c * 32), v);
          const uint32_t word = decide_word<!k3x>(p, v, a, tj * kTile + c * 32, n_cand, norm_a, normB + c * 32, rho, band);
          const int widx = tj * (kTile / 32) + c;
          if (a < n_cand && widx < p.mask_words) p.conflict[(long long)a * p.mask_words + widx] = word;
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
  } else {
    // Split K inside a cluster.  Every CTA parks its partial tile in its own shared memory (the ring is drained:
    // all stages this CTA asked for have been consumed), row r as 32 groups of four columns, group q at slot
    // q ^ (r & 31) so that neither the row-per-thread stores nor the row-per-warp loads meet bank conflicts.
    float* park = reinterpret_cast<float*>(tiles_ptr);
    if (warp < kProducerWarps) {
      bool ok = !s_abort && mbar_wait(done_bar, (uint32_t)iter & 1u, wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok && lane == 0) { s_abort = 1; atomicOr(&p.st->status, STRADS_STATUS_WAIT_EXPIRED); }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int la = warp * 32 + lane;
#pragma unroll 1
      for (int c = 0; c < kTile / 32; ++c) {
        uint32_t v[32];
        if (ok && n_st > 0) {
          tmem_load32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c * 32), v);
        } else {                                         // a split with no K of its own (or one that gave up) adds zero
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int q = c * 8 + j;
          *reinterpret_cast<uint4*>(park + la * kTile + ((q ^ (la & 31)) << 2)) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    // every CTA of the cluster gets here, whatever happened above: the barriers are never left short of an arrival
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
    if (warp < kProducerWarps) {
      // this CTA combines and thresholds its share of the tile's rows: a warp per row, a lane per four columns
      const int row_lo = split * kTile / n_split, row_hi = (split + 1) * kTile / n_split;
      const uint32_t park0 = smem_u32(park);
      for (int la = row_lo + warp; la < row_hi; la += kProducerWarps) {
        const uint32_t local = park0 + (uint32_t)(la * kTile + ((lane ^ (la & 31)) << 2)) * 4u;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sp = 0; sp < n_split; ++sp) {             // in split order
          uint32_t remote;
          asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(sp));
          float4 u;
          asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(u.x), "=f"(u.y), "=f"(u.z), "=f"(u.w) : "r"(remote) : "memory");
          acc.x += u.x; acc.y += u.y; acc.z += u.z; acc.w += u.w;
        }
        const int a = ti * kTile + la;
        const double norm_a = normA[la];
        const float g4[4] = {acc.x, acc.y, acc.z, acc.w};
        unsigned int nib = 0u;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int b = tj * kTile + lane * 4 + k;
          const double den = norm_a * normB[lane * 4 + k];
          const double g = fabs((double)g4[k]);
          const bool live = a < n_cand && b < n_cand && a != b && den > 0.0;
          bool hit = live && g >= rho * den;
          if (live && b > a && fabs(g - rho * den) <= band * den) {
            hit = false;                                   // too close to call: decided exactly by the recheck
            const unsigned int slot = atomicAdd(&p.st->amb_count, 1u);
            if (slot < (unsigned)p.cap_amb) p.amb_pairs[slot] = ((unsigned int)a << 16) | (unsigned int)b;
          }
          if (hit && b > a) list_conflict(p, a, b);
          nib |= (unsigned int)hit << k;
        }
        unsigned int word = nib << ((lane & 7) * 4);       // 8 lanes make one 32-column mask word
        word |= __shfl_xor_sync(0xffffffffu, word, 1);
        word |= __shfl_xor_sync(0xffffffffu, word, 2);
        word |= __shfl_xor_sync(0xffffffffu, word, 4);
        const int widx = tj * (kTile / 32) + (lane >> 3);
        if ((lane & 7) == 0 && a < n_cand && widx < p.mask_words) p.conflict[(long long)a * p.mask_words + widx] = word;
      }
    }
    // nobody leaves (and gives up its shared memory) while a neighbour may still be reading it
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
  }
  __syncthreads();
  if (s_abort) break;                                  // (a wait gave up: nothing more is issued)
  }                                                    // next tile of this CTA
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (tail) window_tail(p, p.cand_cur, n_cand, n_total, tiles_ptr);
}

// All pairs the screen left open: one warp per pair.
__global__ void __launch_bounds__(256) k_gram_recheck(Problem p, int only_if_short) {
  chain_begin();
  if (only_if_short && !p.st->window_short) return;
  const unsigned int n = p.st->amb_count;
  if (n > (unsigned)p.cap_amb) return;                 // overflow: the 3xTF32 kernel redoes every bit instead
  const int lane = threadIdx.x & 31;
  const unsigned int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const unsigned int n_warps = (gridDim.x * blockDim.x) >> 5;
  for (unsigned int e = warp; e < n; e += n_warps) recheck_pair(p, p.amb_pairs[e], lane);
}

}  // namespace

// Clusters of up to kMaxSplit CTAs share a tile; how many clusters of each size the device can hold at once
// (one CTA per SM: the ring takes nearly all of its shared memory) decides the split of a launch.  Eight, the
// portable limit: clusters of 9 to 16 (which the device accepts on request) fill more SMs and shorten the kernel
// when it runs alone (c2's window 22 -> 19 us), but the round as replayed, with the draw of the next round on a stream
// beside it, measured slower with them (c3: 68.4 us per round with clusters of 9, 65.9 with 8; c2 39.1 / 38.2).
constexpr int kMaxSplit = 8;
static int g_max_clusters[kMaxSplit + 1];     // [size]; 0: size not available

cudaError_t prepare_gram_dense_tc() {
  cudaError_t e = cudaFuncSetAttribute(k_gram_dense_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_gram_dense_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem);
  if (e != cudaSuccess) return e;
  for (int size = 2; size <= kMaxSplit; ++size) {
    g_max_clusters[size] = 0;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)size; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)size * 64); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kDynSmem;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k_gram_dense_tc<false>, &cfg) == cudaSuccess) g_max_clusters[size] = n;
    cudaGetLastError();                                  // (a size the device refuses is simply not used)
  }
  return cudaSuccess;
}

// Tensor map over the BF16 copy of the packed candidates: [n_cand rows][N elements], row pitch ldcb, box 64 x 128, 128-byte
// swizzle, zero fill outside.  `out` is 128 bytes, 64-byte aligned (a CUtensorMap).
cudaError_t encode_gram_tensor_map(const Problem& p, void* out) {
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
  using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  const cuuint64_t dims[2] = {(cuuint64_t)p.N, (cuuint64_t)p.n_cand};
  const cuuint64_t strides[1] = {(cuuint64_t)p.ldcb * sizeof(unsigned short)};
  const cuuint32_t box[2] = {(cuuint32_t)kScreenK, (cuuint32_t)kTile};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeFn>(fn)(static_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.xcb,
                                                    dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// pack -> screen (K split inside clusters when the tiles are few) -> exact recheck of the borderline pairs -> (only
// if their list overflowed) 3xTF32 over everything.
// `fallback_elsewhere`: the launch covers a window (n_cand of n_total candidates) and a whole-list retry follows; an
// overflow of the borderline list is then handled by that retry, not by a 3xTF32 launch here, and the last CTA of
// the screen rechecks and walks (*walked = true: the caller's walk kernel need only run if walk_pending is raised).
cudaError_t launch_gram_dense_tc(const Problem& p, const void* tmap, const int* cand, int n_cand, int n_total, bool only_if_short,
                                 bool fallback_elsewhere, cudaEvent_t after_pack, cudaStream_t s, bool* walked) {
  if (walked != nullptr) *walked = false;
  const int n_tiles = (n_cand + kTile - 1) / kTile;
  const int tiles = n_tiles * (n_tiles + 1) / 2;
  const int ois = only_if_short ? 1 : 0;
  // few tiles (a candidate window): share each tile's K range among the CTAs of a cluster so that all SMs work; the
  // largest cluster size of which the device holds `tiles` at once (one wave), and at least two stages of K each
  int n_split = 1;
  if (tiles * 2 <= p.sm_count) {
    const int n_st = (int)((p.N + 2 * kScreenK - 1) / (2 * kScreenK));
    for (int size = kMaxSplit; size >= 2; --size)
      if (g_max_clusters[size] >= tiles && size * 2 <= n_st) { n_split = size; break; }
  }
  Problem q = p;
  q.cand_cur = cand;
  const CUtensorMap& tm = *static_cast<const CUtensorMap*>(tmap);
  cudaError_t e;
  const int pack_ctas = only_if_short ? (n_cand < 4 * p.sm_count ? n_cand : 4 * p.sm_count) : n_cand;
  if ((e = launch_chained(k_pack_candidates, pack_ctas, kPackThreads, 0, s, q, cand, n_cand, ois)) != cudaSuccess) return e;
  if (after_pack != nullptr && (e = cudaEventRecord(after_pack, s)) != cudaSuccess) return e;   // optional step timing
  if (!(p.flags & STRADS_FLAG_GRAM_3XTF32)) {
    const int tail = (fallback_elsewhere && !only_if_short) ? 1 : 0;
    const int ctas = n_split > 1 ? tiles * n_split : (tiles < p.sm_count ? tiles : p.sm_count);
    if ((e = launch_chained_cluster(k_gram_dense_tc<false>, ctas, kThreads, kDynSmem, s, n_split, q, tm, n_cand, n_total,
                                    n_tiles, n_split, ois, tail)) != cudaSuccess)
      return e;
    if (tail && walked != nullptr) *walked = true;
    if (!tail && (e = launch_chained(k_gram_recheck, p.sm_count * 2, 256, 0, s, q, ois)) != cudaSuccess) return e;
  }
  if (!fallback_elsewhere || (p.flags & STRADS_FLAG_GRAM_3XTF32))
    return launch_chained(k_gram_dense_tc<true>, tiles < p.sm_count ? tiles : p.sm_count, kThreads, kDynSmem, s, q, tm, n_cand, n_total,
                          n_tiles, 1, ois, 0);
  return cudaSuccess;
}

}  // namespace strads
