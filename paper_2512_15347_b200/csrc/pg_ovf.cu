// Optimal Variance Filtering (Eq. "ovf"), survivor index compaction, group-relative advantages
// (Eq. "advK"), clustering diagnostics and the uniform-subsampling baseline.
//
// Selection: one warp (or half a warp) per group; the scores become order-preserving 32-bit keys, are sorted in
// registers, the running sums from both ends give the k+1 candidate variances "j lowest + (k-j)
// highest" in fp64 with explicitly rounded operations, membership follows from the keys at the
// two cuts (from ranks in the total order (score, slot) when keys tie there), and the kept slots
// are written in ascending slot order through ballots and popcounts.
#include "pg_common.cuh"
#include <float.h>

namespace pg {

constexpr int kOvfThreads = 256;

struct OvfParams {
  const float* scores;      // [G, n]
  int32_t* keep_idx;        // [G, k]
  int32_t* src_rows;        // [G, k] or null
  float* sel_var;           // [G] or null
  float* kept_scores;       // [G, k] or null
  float* adv;               // [G, k] or null
  const int32_t* traj_in;   // [G, n] or null
  int32_t* traj_out;        // [G, k] or null
  int32_t* status;          // device word or null
  int n, k;
  float adv_eps;
  int bulk_ok;              // scores base is 16-byte aligned: rows may be staged with a bulk copy
};

// Monotone map fp32 -> uint32: a < b (as floats, -0 == +0, NaN highest) <=> key(a) < key(b).
__device__ __forceinline__ uint32_t order_key(float s) {
  if (s != s) return 0xFFFFFFFFu;
  uint32_t b = __float_as_uint(s);
  if (b == 0x80000000u) b = 0u;                       // -0 -> +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Value that enters the variance arithmetic: non-finite scores clamp to +-FLT_MAX.
__device__ __forceinline__ double arithmetic_value(float s) {
  if (s != s) return (double)FLT_MAX;
  if (s > FLT_MAX) return (double)FLT_MAX;
  if (s < -FLT_MAX) return -(double)FLT_MAX;
  return (double)s;
}

// ---------------------------------------------------------------- selection kernel
//
// A group of n scores is handled by the W lanes of a warp (W = 32 in every instantiation the
// launcher uses), E scores per lane, n <= W * E <= 1024.  The kernel is written for W = 16 as
// well - two groups per warp, one per half, so that the phases which use few lanes per group
// (serial running sums, candidate argmax, prefix counts, advantage statistics) serve two groups
// at once - but on the 4096 x 256 -> 32 shape that variant was no faster (each lane then sorts
// twice as many keys and half as many warps are left to hide latencies), so it is not dispatched.
// The warps of a CTA only meet once, for the staging of their rows.
//  0. The CTA's score rows are staged in shared memory by one bulk asynchronous copy
//     (cp.async.bulk, completion on an mbarrier, bounded wait) when source and size are
//     16-byte aligned, else read with ordinary loads.  Lane l takes slots l, l + W, l + 2W, ...
//     (consecutive lanes read consecutive words: no bank conflicts, coalesced global loads).
//  1. The 32-bit order keys alone are sorted with a bitonic network held in registers (one
//     integer min and one max per compare-exchange; shuffles for distances of E and more).
//     Slots >= n hold an all-ones key and sort to the end.  Sorted position q sits in register
//     q % E of lane q / E and is kept in shared memory at word (q % E) * W + q / E, again so that
//     consecutive lanes store consecutive words.
//  2. Running sums from both ends: the centred values and their squares are formed by all lanes
//     in parallel, then lanes 0..3 accumulate one sequence each serially, in order, in fp64 with
//     explicitly rounded operations - the same operations in the same order as a plain serial loop.
//  3. k+1 candidates, argmax with the "largest j" tie rule.
//  4. Membership: by comparison with the two keys at the cuts of the order; only when a key just
//     inside a cut equals the one just outside it (rare for real scores) is the rank of every
//     element in the total order (score, slot) worked out, by a binary search in the sorted keys
//     plus a direct count of equal keys in lower slots.  Ascending slot order of the kept slots
//     follows from one ballot per register index (slots r * W + lane are ascending in r, then lane).
//  5. Kept scores go through shared memory so that their stores, the advantage statistics and
//     the single division are spread over the lanes.
constexpr int kOvfMaxWarps = 4;                 // warps per CTA, fewer when the groups' shared memory is large
constexpr size_t kOvfSmemBudget = 47 * 1024;    // dynamic shared memory a CTA may use without opting in

__device__ __forceinline__ float key_to_score(uint32_t key) {
  const uint32_t b = (key & 0x80000000u) ? (key ^ 0x80000000u) : ~key;
  return __uint_as_float(b);      // all-ones key -> 0x7FFFFFFF, a NaN, as it went in
}

template <int W>
__device__ __forceinline__ double lanes_sum(double v) {      // sum over the W lanes of a group
#pragma unroll
  for (int o = W / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// bytes of shared memory per group: four running-sum arrays of k + 1 doubles, sorted keys and
// slot-order keys of W * E words each (the staged row comes on top: W * E floats)
__host__ __device__ inline size_t ovf_group_bytes(int k, int N) {
  return (size_t)(k + 1) * 4 * sizeof(double) + (size_t)N * 2 * sizeof(uint32_t);
}

template <int E, int W>
__global__ void __launch_bounds__(kOvfMaxWarps * 32)
ovf_warp_kernel(const __grid_constant__ OvfParams p, int n_groups) {
  constexpr int N = W * E;
  constexpr int kPerWarp = 32 / W;                       // groups per warp
  constexpr unsigned int kFull = 0xFFFFFFFFu;
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ __align__(8) unsigned long long stage_bar;
  const int n = p.n, k = p.k;
  const int groups_per_cta = (blockDim.x >> 5) * kPerWarp;
  const int warp = threadIdx.x >> 5, wlane = threadIdx.x & 31;
  const int lane = wlane & (W - 1), sub = wlane / W;     // lane within the group, group within the warp
  const int slot = warp * kPerWarp + sub;                // group within the CTA
  const int g0 = blockIdx.x * groups_per_cta;
  const int g = g0 + slot;
  const bool active = g < n_groups;                      // a warp's second half may have no group

  // 0. stage the score rows of this CTA's groups (contiguous in memory) in shared memory with
  //    one bulk asynchronous copy, completion signalled on an mbarrier.  Needs a 16-byte
  //    aligned source and size; otherwise the rows are read with ordinary loads.  The wait is
  //    bounded: if the copy has not landed in time, status bit 1 is set, the wait is repeated
  //    once, and if any thread still has not seen the copy land the whole CTA gives up together.
  float* stage = reinterpret_cast<float*>(smem);                 // [groups_per_cta * N]
  const int groups_here = min(groups_per_cta, n_groups - g0);
  const unsigned int stage_bytes = (unsigned int)groups_here * (unsigned int)n * 4u;
  const bool bulk = p.bulk_ok && (stage_bytes & 15u) == 0 && ((((size_t)g0 * n * 4) & 15) == 0);
  if (bulk) {                                                    // uniform over the CTA
    const unsigned int bar = (unsigned int)__cvta_generic_to_shared(&stage_bar);
    const unsigned int dst = (unsigned int)__cvta_generic_to_shared(stage);
    if (threadIdx.x == 0) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      const float* src = p.scores + (size_t)g0 * n;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(stage_bytes)
                   : "memory");
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
          "l"(src), "r"(stage_bytes), "r"(bar)
          : "memory");
    }
    bool done = false;
    for (int round = 0; round < 2 && !done; ++round) {
      done = mbarrier_wait_bounded(bar, 0u, kBulkWaitLimit);
      if (!done && round == 0 && threadIdx.x == 0 && p.status) atomicOr(p.status, 2);
    }
    // one verdict for the CTA: threads whose last attempt succeeded must not run ahead into the
    // warp-wide shuffles while others of their warp leave
    if (!__syncthreads_and(done ? 1 : 0)) {
      if (threadIdx.x == 0 && p.status) atomicOr(p.status, 2);
      return;
    }
  }
  if (g0 + warp * kPerWarp >= n_groups) return;                  // the whole warp has no group
  const size_t per_group = ovf_group_bytes(k, N);
  unsigned char* base = smem + (size_t)groups_per_cta * N * sizeof(float) + (size_t)slot * per_group;
  double* L1 = reinterpret_cast<double*>(base);
  double* L2 = L1 + (k + 1);
  double* H1 = L2 + (k + 1);
  double* H2 = H1 + (k + 1);
  uint32_t* skey = reinterpret_cast<uint32_t*>(H2 + (k + 1));   // [N] sorted keys, position q at (q % E) * W + q / E
  uint32_t* okey = skey + N;                                    // [N] keys in slot order
  auto sorted_key = [&](int q) -> uint32_t { return skey[(q & (E - 1)) * W + (q / E)]; };

  const float* sc = p.scores + (size_t)(active ? g : 0) * n;
  float orig[E];
  uint32_t mine[E], key[E];
  bool bad = false;
#pragma unroll
  for (int r = 0; r < E; ++r) {
    const int i = r * W + lane;                                  // slot within the group
    if (active && i < n) {
      orig[r] = bulk ? stage[slot * n + i] : sc[i];
      bad |= !(fabsf(orig[r]) <= FLT_MAX);
      mine[r] = order_key(orig[r]);
    } else {
      orig[r] = 0.f;
      mine[r] = 0xFFFFFFFFu;
    }
    key[r] = mine[r];
  }
  if (bad && p.status) atomicOr(p.status, 1);

  // 1. bitonic sort, ascending over position lane * E + r; every compare-exchange points the same
  //    way: a merge first pairs a position with its mirror q ^ (size - 1), then halves the distance.
  //    (Which slot starts in which register does not matter to a sort.)
#pragma unroll
  for (int size = 2; size <= N; size <<= 1) {
    if (size <= E) {
#pragma unroll
      for (int r = 0; r < E; ++r) {
        const int q = r ^ (size - 1);
        if (r < q) {
          const uint32_t a = key[r], b = key[q];
          key[r] = min(a, b);
          key[q] = max(a, b);
        }
      }
    } else {
      const int lane_mask = size / E - 1;
      const bool lower = (lane & (size / E / 2)) == 0;
      uint32_t other[E];
#pragma unroll
      for (int r = 0; r < E; ++r) other[r] = __shfl_xor_sync(kFull, key[r ^ (E - 1)], lane_mask);
      // (a compare combined with the lane's side plus one select instead of min, max and select
      // measured slower: 15.1 instead of 13.8 us on 4096 groups of 256)
#pragma unroll
      for (int r = 0; r < E; ++r) key[r] = lower ? min(key[r], other[r]) : max(key[r], other[r]);
    }
#pragma unroll
    for (int j = size >> 2; j > 0; j >>= 1) {
      if (j < E) {
#pragma unroll
        for (int r = 0; r < E; ++r) {
          if ((r & j) == 0) {
            const uint32_t a = key[r], b = key[r | j];
            key[r] = min(a, b);
            key[r | j] = max(a, b);
          }
        }
      } else {
        const int lane_mask = j / E;
        const bool lower = (lane & lane_mask) == 0;
#pragma unroll
        for (int r = 0; r < E; ++r) {
          const uint32_t other = __shfl_xor_sync(kFull, key[r], lane_mask);
          key[r] = lower ? min(key[r], other) : max(key[r], other);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < E; ++r) skey[r * W + lane] = key[r];
  __syncwarp();

  // 2. centred values and squares in parallel, then the serial running sums
  const double pivot = arithmetic_value(key_to_score(sorted_key(n / 2)));
  for (int j = lane; j < k; j += W) {
    const double cl = __dsub_rn(arithmetic_value(key_to_score(sorted_key(j))), pivot);
    const double ch = __dsub_rn(arithmetic_value(key_to_score(sorted_key(n - 1 - j))), pivot);
    L1[j + 1] = cl;
    L2[j + 1] = __dmul_rn(cl, cl);
    H1[j + 1] = ch;
    H2[j + 1] = __dmul_rn(ch, ch);
  }
  __syncwarp();
  if (lane < 4) {                       // L1, L2, H1, H2 are contiguous: one serial chain per lane
    double* S = L1 + (size_t)lane * (k + 1);
    double a = 0.0;
    S[0] = 0.0;
#pragma unroll 4
    for (int j = 1; j <= k; ++j) {
      a = __dadd_rn(a, S[j]);
      S[j] = a;
    }
  }
  __syncwarp();

  // 3. candidates
  double best_m = -1.0;
  int best_j = -1;
  for (int j = lane; j <= k; j += W) {
    const double S = __dadd_rn(L1[j], H1[k - j]);
    const double Q = __dadd_rn(L2[j], H2[k - j]);
    const double M = __dsub_rn(__dmul_rn((double)k, Q), __dmul_rn(S, S));
    if (best_j < 0 || M >= best_m) { best_m = M; best_j = j; }
  }
#pragma unroll
  for (int o = W / 2; o > 0; o >>= 1) {
    const double om = __shfl_xor_sync(kFull, best_m, o);
    const int oj = __shfl_xor_sync(kFull, best_j, o);
    if (oj >= 0 && (best_j < 0 || om > best_m || (om == best_m && oj > best_j))) {
      best_m = om; best_j = oj;
    }
  }
  const int jstar = best_j;
  const int high_from = n - (k - jstar);
  if (lane == 0 && active && p.sel_var) p.sel_var[g] = (float)(best_m / ((double)k * (double)k));

  // 4. membership.  With distinct keys at both cuts of the order an element is kept exactly when
  //    its key is at most the j*-th lowest or at least the (k - j*)-th highest key.  Only when the
  //    key just inside a cut equals the key just outside it does the slot decide: then every
  //    element finds its rank in the total order (score, slot) by a binary search for its key in
  //    the sorted list, advanced by the number of equal keys in lower slots.
  const int n_high = k - jstar;
  const uint32_t lowkey = jstar > 0 ? sorted_key(jstar - 1) : 0u;
  const uint32_t highkey = n_high > 0 ? sorted_key(high_from) : 0xFFFFFFFFu;
  const bool cut_tie = (jstar > 0 && jstar < n && sorted_key(jstar) == lowkey) ||
                       (n_high > 0 && high_from > 0 && sorted_key(high_from - 1) == highkey);
  if (__any_sync(kFull, cut_tie)) {                 // uniform over the warp: both groups publish their keys
#pragma unroll
    for (int r = 0; r < E; ++r) okey[r * W + lane] = mine[r];
    __syncwarp();
  }
  unsigned int bits = 0u;
  if (!cut_tie) {                                   // uniform over the group; no warp-wide operation inside
#pragma unroll
    for (int r = 0; r < E; ++r) {
      const bool in_low = jstar > 0 && mine[r] <= lowkey;
      const bool in_high = n_high > 0 && mine[r] >= highkey;
      if (r * W + lane < n && (in_low || in_high)) bits |= 1u << r;
    }
  } else {
#pragma unroll
    for (int r = 0; r < E; ++r) {
      const int i = r * W + lane;
      int rank = 0;
#pragma unroll
      for (int step = N / 2; step > 0; step >>= 1)
        if (sorted_key(rank + step - 1) < mine[r]) rank += step;    // first position whose key is >= mine
      if (i < n && rank + 1 < N && sorted_key(rank + 1) == mine[r]) {  // equal keys exist
        int lower_slots = 0;
        for (int j = 0; j < i; ++j) lower_slots += (okey[j] == mine[r]) ? 1 : 0;
        rank += lower_slots;
      }
      if (i < n && (rank < jstar || rank >= high_from)) bits |= 1u << r;
    }
  }

  // 5. output in ascending slot order: slots r * W + lane ascend with r first, then with the lane
  const bool want_scores = p.kept_scores || p.adv;
  float* kept_s = reinterpret_cast<float*>(L1);     // [k], reuses the running sums' space
  __syncwarp();                                     // every lane is done with the running sums
  constexpr unsigned int kGroupMask = (W == 32) ? 0xFFFFFFFFu : ((1u << (W & 31)) - 1u);
  int before = 0;                                   // kept slots of this group below the current r
#pragma unroll
  for (int r = 0; r < E; ++r) {
    const bool kept = (bits >> r) & 1u;
    const unsigned int group_votes = (__ballot_sync(kFull, kept) >> (sub * W)) & kGroupMask;
    if (kept && active) {
      const int i = r * W + lane;
      const int pos = before + __popc(group_votes & ((1u << lane) - 1u));
      const size_t o = (size_t)g * k + pos;
      p.keep_idx[o] = i;
      if (p.src_rows) p.src_rows[o] = g * n + i;
      if (p.traj_out) p.traj_out[o] = p.traj_in[(size_t)g * n + i];
      if (want_scores) kept_s[pos] = orig[r];
    }
    before += __popc(group_votes);
  }
  if (want_scores) {
    // kept scores in slot order, now spread over the lanes: coalesced stores, one division
    __syncwarp();
    double sum_kept = 0.0;
    for (int j = lane; j < k; j += W) {
      const float v = kept_s[j];
      if (p.kept_scores && active) p.kept_scores[(size_t)g * k + j] = v;
      sum_kept += (double)v;
    }
    if (p.adv) {
      const double mu = lanes_sum<W>(sum_kept) / (double)k;
      double sq = 0.0;
      for (int j = lane; j < k; j += W) {
        const double dlt = (double)kept_s[j] - mu;
        sq += dlt * dlt;
      }
      const double inv = 1.0 / (sqrt(lanes_sum<W>(sq) / (double)k) + (double)p.adv_eps);
      if (active)
        for (int j = lane; j < k; j += W)
          p.adv[(size_t)g * k + j] = (float)(((double)kept_s[j] - mu) * inv);
    }
  }
}

template <int E, int W>
static void launch_ovf_warp(const OvfParams& p, int n_groups, cudaStream_t stream) {
  constexpr int N = W * E, kPerWarp = 32 / W;
  const size_t per_group = ovf_group_bytes(p.k, N) + (size_t)N * sizeof(float);   // + the staged row
  int warps = kOvfMaxWarps;
  while (warps > 1 && (size_t)warps * kPerWarp * per_group > kOvfSmemBudget) warps >>= 1;
  const int groups_per_cta = warps * kPerWarp;
  const int ctas = (n_groups + groups_per_cta - 1) / groups_per_cta;
  ovf_warp_kernel<E, W><<<ctas, warps * 32, (size_t)groups_per_cta * per_group, stream>>>(p, n_groups);
}

int launch_ovf(int n_groups, int n, int k, const float* scores, int32_t* keep_idx,
               int32_t* src_rows, float* sel_var, float* kept_scores, float* adv, float adv_eps,
               const int32_t* traj_in, int32_t* traj_out, int32_t* status, cudaStream_t stream) {
  if (n_groups == 0) return PG_OK;
  OvfParams p;
  p.scores = scores;
  p.keep_idx = keep_idx;
  p.src_rows = src_rows;
  p.sel_var = sel_var;
  p.kept_scores = kept_scores;
  p.adv = adv;
  p.traj_in = traj_in;
  p.traj_out = traj_out;
  p.status = status;
  p.n = n;
  p.k = k;
  p.adv_eps = adv_eps;
  p.bulk_ok = (((uintptr_t)scores) & 15) == 0;
  if (n <= 32)       launch_ovf_warp<1, 32>(p, n_groups, stream);
  else if (n <= 64)  launch_ovf_warp<2, 32>(p, n_groups, stream);
  else if (n <= 128) launch_ovf_warp<4, 32>(p, n_groups, stream);
  else if (n <= 256) launch_ovf_warp<8, 32>(p, n_groups, stream);
  else if (n <= 512) launch_ovf_warp<16, 32>(p, n_groups, stream);
  else               launch_ovf_warp<32, 32>(p, n_groups, stream);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- advantages

// One warp per group: mean, population standard deviation, (R - mu) / (sigma + eps).
__global__ void __launch_bounds__(128)
advantages_kernel(int n_groups, int K, const float* rewards, float eps, float* adv, float* mean,
                  float* std_out) {
  const int g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (g >= n_groups) return;
  const float* r = rewards + (size_t)g * K;
  double s = 0.0;
  for (int i = lane; i < K; i += 32) s += (double)r[i];
  const double mu = warp_sum(s) / (double)K;
  double q = 0.0;
  for (int i = lane; i < K; i += 32) {
    const double dlt = (double)r[i] - mu;
    q += dlt * dlt;
  }
  const double sigma = sqrt(warp_sum(q) / (double)K);
  const double denom = sigma + (double)eps;
  for (int i = lane; i < K; i += 32) adv[(size_t)g * K + i] = (float)(((double)r[i] - mu) / denom);
  if (lane == 0) {
    if (mean) mean[g] = (float)mu;
    if (std_out) std_out[g] = (float)sigma;
  }
}

int launch_advantages(int n_groups, int K, const float* rewards, float eps, float* adv,
                      float* mean, float* std_out, cudaStream_t stream) {
  if (n_groups == 0) return PG_OK;
  const int warps = 4;
  advantages_kernel<<<(n_groups + warps - 1) / warps, warps * 32, 0, stream>>>(
      n_groups, K, rewards, eps, adv, mean, std_out);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- diagnostics / uniform baseline

// One warp per group: mean, population standard deviation and the fraction of scores inside
// the clustered region |R - mu| <= delta * sigma (Eq. "near-mean").
__global__ void __launch_bounds__(128)
group_stats_kernel(int n_groups, int n, const float* scores, double delta, float* mean, float* std_out,
                   float* clustered) {
  const int g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (g >= n_groups) return;
  const float* r = scores + (size_t)g * n;
  double s = 0.0;
  for (int i = lane; i < n; i += 32) s += (double)r[i];
  const double mu = warp_sum(s) / (double)n;
  double q = 0.0;
  for (int i = lane; i < n; i += 32) {
    const double dlt = (double)r[i] - mu;
    q += dlt * dlt;
  }
  const double sigma = sqrt(warp_sum(q) / (double)n);
  int inside = 0;
  for (int i = lane; i < n; i += 32) inside += (fabs((double)r[i] - mu) <= delta * sigma) ? 1 : 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) inside += __shfl_xor_sync(0xFFFFFFFFu, inside, o);
  if (lane == 0) {
    if (mean) mean[g] = (float)mu;
    if (std_out) std_out[g] = (float)sigma;
    if (clustered) clustered[g] = (float)((double)inside / (double)n);
  }
}

int launch_group_stats(int n_groups, int n, const float* scores, double delta, float* mean,
                       float* std_out, float* clustered, cudaStream_t stream) {
  if (n_groups == 0) return PG_OK;
  group_stats_kernel<<<(n_groups + 3) / 4, 128, 0, stream>>>(n_groups, n, scores, delta, mean, std_out,
                                                            clustered);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// Uniform k-of-n subsampling per group: slot i draws the first Philox word of counter
// (i, stage, group, stream 4); the k smallest (word, slot) pairs are kept, ascending slot order.
__global__ void __launch_bounds__(kOvfThreads)
uniform_select_kernel(const __grid_constant__ PhiloxKeys rk, int n, int k, uint32_t stage,
                      uint32_t group_offset, int32_t* keep_idx, int32_t* src_rows,
                      const int32_t* traj_in, int32_t* traj_out) {
  __shared__ unsigned long long keys[PG_MAX_GROUP];
  __shared__ int warp_cnt[kOvfThreads / 32];
  const int g = blockIdx.x, tid = threadIdx.x;
  for (int i = tid; i < n; i += kOvfThreads) {
    const uint4 r = philox4x32_10((uint32_t)i, stage, group_offset + (uint32_t)g, 4u, rk);
    keys[i] = ((unsigned long long)r.x << 32) | (unsigned int)i;
  }
  __syncthreads();
  int running = 0;
  for (int base = 0; base < n; base += kOvfThreads) {
    const int i = base + tid;
    bool keep = false;
    if (i < n) {
      const unsigned long long mine = keys[i];
      int smaller = 0;
      for (int j = 0; j < n; ++j) smaller += (keys[j] < mine) ? 1 : 0;
      keep = smaller < k;
    }
    const unsigned int bal = __ballot_sync(0xFFFFFFFFu, keep);
    if ((tid & 31) == 0) warp_cnt[tid >> 5] = __popc(bal);
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kOvfThreads / 32; ++w) {
      const int c = warp_cnt[w];
      if (w < (tid >> 5)) before += c;
      total += c;
    }
    if (keep) {
      const size_t o = (size_t)g * k + running + before + __popc(bal & ((1u << (tid & 31)) - 1u));
      keep_idx[o] = i;
      if (src_rows) src_rows[o] = g * n + i;
      if (traj_out) traj_out[o] = traj_in[(size_t)g * n + i];
    }
    running += total;
    __syncthreads();
  }
}

int launch_uniform_select(int n_groups, int n, int k, uint64_t seed, uint32_t stage,
                          uint32_t group_offset, int32_t* keep_idx, int32_t* src_rows,
                          const int32_t* traj_in, int32_t* traj_out, cudaStream_t stream) {
  if (n_groups == 0) return PG_OK;
  uniform_select_kernel<<<n_groups, kOvfThreads, 0, stream>>>(make_philox_keys(seed), n, k, stage,
                                                              group_offset, keep_idx, src_rows, traj_in,
                                                              traj_out);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- bounded-wait self-test

// One CTA waits, exactly as the selection kernel waits for its staged rows, on an mbarrier whose
// phase nothing will ever complete (no copy is issued, nobody arrives).  Both rounds of attempts
// run out, status bit 1 is set after the first, and the kernel returns normally: the path a lost
// copy would take, exercised without losing one.
__global__ void __launch_bounds__(32) wait_selftest_kernel(int32_t* status) {
  __shared__ __align__(8) unsigned long long bar_mem;
  const unsigned int bar = (unsigned int)__cvta_generic_to_shared(&bar_mem);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  bool done = false;
  for (int round = 0; round < 2 && !done; ++round) {
    done = mbarrier_wait_bounded(bar, 0u, kBulkWaitLimit);
    if (!done && round == 0 && threadIdx.x == 0 && status) atomicOr(status, 2);
  }
  if (!__syncthreads_and(done ? 1 : 0)) return;      // the same CTA-wide verdict as in the selection kernel
}

int launch_wait_selftest(int32_t* status, cudaStream_t stream) {
  wait_selftest_kernel<<<1, 32, 0, stream>>>(status);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

// ---------------------------------------------------------------- trajectory ids

__global__ void iota_kernel(int32_t* dst, int n, int32_t base) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = base + i;
}

int launch_iota(int32_t* dst, int n, int32_t base, cudaStream_t stream) {
  if (n == 0) return PG_OK;
  iota_kernel<<<(n + 255) / 256, 256, 0, stream>>>(dst, n, base);
  PG_LAUNCH_CHECK();
  return PG_OK;
}

}  // namespace pg
