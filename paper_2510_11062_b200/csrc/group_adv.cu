// Agent- and turn-wise grouped advantage (Eq. 1 over the groups of Algorithm 1).
//
// Three pipelines, all on the caller's stream with no host synchronisation.
//
// (A) Advantages only (no bucketing output requested): a sort-free group aggregate in three
//     passes over the candidates plus one over the groups.  Everything that is accumulated with
//     atomics is an integer, so the result does not depend on the order of arrival:
//       minmax  : g, per-group count, min and max reward (order-preserving integer encoding)
//       moments : x = round((r - min)/(max - min) * 2^25); sum of x and of x^2 in 64-bit integers
//                 (2^30 and a second word for x^2 in groups of 4096 members or more)
//       finalize: exact integer K*sum(x^2) - sum(x)^2 (128-bit) -> mean, 1/(std + eps) per group
//       apply   : adv = (r - mean) * 1/(std + eps)
//     Quantising to 2^-25 of the group's range moves mean and std by < 3e-8 of the range; a group
//     with max == min gets exact zeros.  Random access touches only the per-group table, two
//     16-byte entries per group.
//
// (B) Bucketing requested (group_offsets / group_perm): counting sort + ordered statistics:
//   key_count  : g = (e*n_role + i)*n_turn + t, per-group histogram; the atomic's return value is
//                the candidate's (arbitrary) arrival slot inside its group
//   scan       : exclusive scan of the histogram -> group_offsets        (two launches)
//   scatter    : unordered bucket fill, perm_u[offsets[g] + slot] = c
//   stats      : one thread per group sorts its few members by candidate index (which makes the
//                permutation stable and the fp64 sums order-fixed), then mean / std / advantage.
//
// (C) Adjacent groups (params.candidates_grouped): the caller promises that the members of every
//     group are adjacent, which is the order Algorithm 1 appends them in (the K samples of one
//     (environment, agent, turn) together).  One streaming pass: a block stages a tile of
//     candidates in shared memory and marks where runs of equal keys begin; one thread per run
//     fetches the run's members once into registers, sums them in ascending order (fp32 on values
//     shifted by the run's first reward for runs of up to 16 members, fp64 otherwise) and
//     writes the advantages back over the staged rewards, and the tile leaves with coalesced
//     stores; longer runs loop over shared memory, are summed by a warp, or (beyond the staged
//     window) by the whole block.  One integer atomic per RUN checks the promise (a key that
//     starts two runs raises ATGRPO_ERR_LAYOUT).
//
// Groups of the paper hold K = 4 .. 16 candidates, far fewer than a warp, so a thread per group
// with block-cooperative coalesced staging keeps every lane busy; blocks that meet a large group
// switch to a block-per-group path (shared-memory bitonic sort or an ordered rescan) with a
// shuffle/shared-memory tree reduction.
#include "internal.h"

namespace atgrpo {
namespace {

constexpr int kThreads = 256;
constexpr int kScanItems = 4;                        // counts per thread in the scan kernels
constexpr int kScanBlock = kThreads * kScanItems;    // 1024 groups per scan block
constexpr int kCap = 4096;                           // staged members per stats block
constexpr int kSerialMaxK = 64;                      // largest group a single thread sorts

__device__ __forceinline__ int group_of(int e, int i, int t, int n_env, int n_role, int n_turn) {
  const bool ok = (unsigned)e < (unsigned)n_env && (unsigned)i < (unsigned)n_role &&
                  (unsigned)t < (unsigned)n_turn;
  return ok ? (e * n_role + i) * n_turn + t : -1;
}

// kPacked (here and in k_hash_minmax): `env` holds ready-made group ids in [0, n_env) and the
// role / turn arrays are not read (n_role = n_turn = 1).
template <bool kVec, bool kPacked>
__global__ void __launch_bounds__(kThreads)
k_key_count(const int32_t* __restrict__ env, const int32_t* __restrict__ role,
            const int32_t* __restrict__ turn, int n, int n_env, int n_role, int n_turn,
            int32_t* __restrict__ count, int32_t* __restrict__ slot, int32_t* __restrict__ gid,
            float* __restrict__ adv, int32_t* status) {
  const int stride = gridDim.x * blockDim.x;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x;
  if (kVec) {
    const int n4 = n >> 2;
    for (int q = tid; q < n4; q += stride) {
      const int4 e = reinterpret_cast<const int4*>(env)[q];
      const int4 zero = make_int4(0, 0, 0, 0);
      const int4 r = kPacked ? zero : reinterpret_cast<const int4*>(role)[q];
      const int4 t = kPacked ? zero : reinterpret_cast<const int4*>(turn)[q];
      int4 g, s;
      g.x = group_of(e.x, r.x, t.x, n_env, n_role, n_turn);
      g.y = group_of(e.y, r.y, t.y, n_env, n_role, n_turn);
      g.z = group_of(e.z, r.z, t.z, n_env, n_role, n_turn);
      g.w = group_of(e.w, r.w, t.w, n_env, n_role, n_turn);
      s.x = g.x >= 0 ? atomicAdd(&count[g.x], 1) : 0;
      s.y = g.y >= 0 ? atomicAdd(&count[g.y], 1) : 0;
      s.z = g.z >= 0 ? atomicAdd(&count[g.z], 1) : 0;
      s.w = g.w >= 0 ? atomicAdd(&count[g.w], 1) : 0;
      reinterpret_cast<int4*>(gid)[q] = g;
      reinterpret_cast<int4*>(slot)[q] = s;
      if ((g.x | g.y | g.z | g.w) < 0) {
        raise_status(status, ATGRPO_ERR_BAD_INDEX);
        if (g.x < 0) adv[4 * q + 0] = 0.f;
        if (g.y < 0) adv[4 * q + 1] = 0.f;
        if (g.z < 0) adv[4 * q + 2] = 0.f;
        if (g.w < 0) adv[4 * q + 3] = 0.f;
      }
    }
  }
  const int first = kVec ? (n & ~3) : 0;
  for (int c = first + tid; c < n; c += stride) {
    const int g = group_of(env[c], kPacked ? 0 : role[c], kPacked ? 0 : turn[c], n_env, n_role, n_turn);
    gid[c] = g;
    if (g >= 0) {
      slot[c] = atomicAdd(&count[g], 1);
    } else {
      slot[c] = 0;
      adv[c] = 0.f;
      raise_status(status, ATGRPO_ERR_BAD_INDEX);
    }
  }
}

// Inclusive scan of one int per thread across the block (shuffle inside warps, shared across).
__device__ __forceinline__ int block_inclusive_scan(int v, int* warp_tot /* [kThreads/32] */) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += u;
  }
  if (lane == 31) warp_tot[w] = v;
  __syncthreads();
  int add = 0;
  for (int i = 0; i < w; ++i) add += warp_tot[i];
  __syncthreads();
  return v + add;
}

__global__ void __launch_bounds__(kThreads)
k_block_sums(const int32_t* __restrict__ count, int G, int32_t* __restrict__ block_sum) {
  __shared__ int warp_tot[kThreads / 32];
  const int base = blockIdx.x * kScanBlock + threadIdx.x * kScanItems;
  int v = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i)
    if (base + i < G) v += count[base + i];
  const int incl = block_inclusive_scan(v, warp_tot);
  if (threadIdx.x == kThreads - 1) block_sum[blockIdx.x] = incl;
}

__global__ void __launch_bounds__(kThreads)
k_scan_offsets(const int32_t* __restrict__ count, int G, const int32_t* __restrict__ block_sum,
               int32_t* __restrict__ offsets) {
  __shared__ int warp_tot[kThreads / 32];
  __shared__ int red[kThreads];
  // prefix of the blocks before this one, fixed-order tree
  int pre = 0;
  for (int b = threadIdx.x; b < (int)blockIdx.x; b += kThreads) pre += block_sum[b];
  red[threadIdx.x] = pre;
  __syncthreads();
  for (int s = kThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  const int block_pre = red[0];
  const int base = blockIdx.x * kScanBlock + threadIdx.x * kScanItems;
  int c[kScanItems];
  int v = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    c[i] = (base + i < G) ? count[base + i] : 0;
    v += c[i];
  }
  const int incl = block_inclusive_scan(v, warp_tot);
  int run = block_pre + incl - v;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    if (base + i < G) offsets[base + i] = run;
    run += c[i];
    if (base + i == G - 1) offsets[G] = run;
  }
}

__global__ void __launch_bounds__(kThreads)
k_scatter(const int32_t* __restrict__ gid, const int32_t* __restrict__ slot,
          const int32_t* __restrict__ offsets, int n, int32_t* __restrict__ perm_u) {
  const int stride = gridDim.x * blockDim.x;
  for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < n; c += stride) {
    const int g = gid[c];
    if (g >= 0) perm_u[offsets[g] + slot[c]] = c;
  }
}


// ------------------------------------------------------------------ (A) sort-free aggregate
constexpr double kQuantSmall = 33554432.0;     // 2^25 steps across a group's reward range (< 4096 members)
constexpr double kQuantBig = 1073741824.0;     // 2^30 steps for larger groups (x^2 sum split in two words)
constexpr unsigned kBigGroup = 4096;           // 4096 * (2^25)^2 = 2^62 still fits one 64-bit sum

// Order-preserving map float -> uint32 (and back), so integer atomicMax orders rewards.
__device__ __forceinline__ uint32_t enc_ordered(float f) {
  const uint32_t b = __float_as_uint(f);
  return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float dec_ordered(uint32_t e) {
  return __uint_as_float((e & 0x80000000u) ? (e ^ 0x80000000u) : ~e);
}

// Two 16-byte entries per group slot, in separate arrays: the first pass and the last touch one
// array each, so a table larger than L2 costs them half the traffic.  One memset zeroes both.
struct alignas(16) GroupHead {
  uint32_t cnt;                // members
  uint32_t nmin;               // ~enc(min): atomicMax from 0 tracks the minimum
  uint32_t emax;               // enc(max)
  uint32_t pad;
};
struct alignas(16) GroupMoments {
  unsigned long long sum;      // sum of x;   after finalize: mean as double
  unsigned long long sq;       // sum of x^2 (low 32-bit parts for big groups); after finalize: 1/(std+eps)
};

struct GroupTable {
  GroupHead* h;
  GroupMoments* m;
  unsigned long long* sqhi;    // sum of x^2 >> 32, touched by groups of kBigGroup members or more only
  unsigned long long* best;    // optional: max of (enc(reward) << 32 | ~candidate): argmax, ties to the lowest index
};

__device__ __forceinline__ void minmax_one(int g, float r, int c, const GroupTable& t) {
  const uint32_t e = enc_ordered(r);
  GroupHead* ge = t.h + g;
  atomicAdd(&ge->cnt, 1u);
  atomicMax(&ge->nmin, ~e);
  atomicMax(&ge->emax, e);
  if (t.best) atomicMax(&t.best[g], ((unsigned long long)e << 32) | (0xFFFFFFFFu - (uint32_t)c));
}

template <bool kVec, bool kPacked>
__global__ void __launch_bounds__(kThreads)
k_hash_minmax(const int32_t* __restrict__ env, const int32_t* __restrict__ role,
              const int32_t* __restrict__ turn, const float* __restrict__ rewards, int n, int n_env,
              int n_role, int n_turn, GroupTable t, int32_t* __restrict__ gid,
              float* __restrict__ adv, int32_t* status) {
  const int stride = gridDim.x * blockDim.x;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x;
  if (kVec) {
    const int n4 = n >> 2;
    for (int q = tid; q < n4; q += stride) {
      const int4 e = reinterpret_cast<const int4*>(env)[q];
      const int4 zero = make_int4(0, 0, 0, 0);
      const int4 r = kPacked ? zero : reinterpret_cast<const int4*>(role)[q];
      const int4 u = kPacked ? zero : reinterpret_cast<const int4*>(turn)[q];
      const float4 w = reinterpret_cast<const float4*>(rewards)[q];
      int4 g;
      g.x = group_of(e.x, r.x, u.x, n_env, n_role, n_turn);
      g.y = group_of(e.y, r.y, u.y, n_env, n_role, n_turn);
      g.z = group_of(e.z, r.z, u.z, n_env, n_role, n_turn);
      g.w = group_of(e.w, r.w, u.w, n_env, n_role, n_turn);
      reinterpret_cast<int4*>(gid)[q] = g;
      if (g.x >= 0) minmax_one(g.x, w.x, 4 * q + 0, t);
      if (g.y >= 0) minmax_one(g.y, w.y, 4 * q + 1, t);
      if (g.z >= 0) minmax_one(g.z, w.z, 4 * q + 2, t);
      if (g.w >= 0) minmax_one(g.w, w.w, 4 * q + 3, t);
      if ((g.x | g.y | g.z | g.w) < 0) {
        raise_status(status, ATGRPO_ERR_BAD_INDEX);
        if (g.x < 0) adv[4 * q + 0] = 0.f;
        if (g.y < 0) adv[4 * q + 1] = 0.f;
        if (g.z < 0) adv[4 * q + 2] = 0.f;
        if (g.w < 0) adv[4 * q + 3] = 0.f;
      }
    }
  }
  const int first = kVec ? (n & ~3) : 0;
  for (int c = first + tid; c < n; c += stride) {
    const int g = group_of(env[c], kPacked ? 0 : role[c], kPacked ? 0 : turn[c], n_env, n_role, n_turn);
    gid[c] = g;
    if (g >= 0) {
      minmax_one(g, rewards[c], c, t);
    } else {
      adv[c] = 0.f;
      raise_status(status, ATGRPO_ERR_BAD_INDEX);
    }
  }
}

__device__ __forceinline__ void moments_one(int g, float r, const GroupTable& t) {
  GroupMoments* ge = t.m + g;
  const uint4 head = *reinterpret_cast<const uint4*>(t.h + g);     // cnt, nmin, emax in one 16-byte load
  const double lo = (double)dec_ordered(~head.y);
  const double range = (double)dec_ordered(head.z) - lo;
  if (!(range > 0.0)) return;                       // single member or all equal: nothing to add
  const bool big = head.x >= kBigGroup;
  const unsigned long long x = (unsigned long long)__double2ll_rn(
      ((double)r - lo) * ((big ? kQuantBig : kQuantSmall) / range));
  const unsigned long long x2 = x * x;
  atomicAdd(&ge->sum, x);
  if (big) {
    atomicAdd(&ge->sq, x2 & 0xFFFFFFFFull);
    atomicAdd(&t.sqhi[g], x2 >> 32);
  } else {
    atomicAdd(&ge->sq, x2);
  }
}

template <bool kVec>
__global__ void __launch_bounds__(kThreads)
k_hash_moments(const int32_t* __restrict__ gid, const float* __restrict__ rewards, int n,
               GroupTable t) {
  const int stride = gridDim.x * blockDim.x;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x;
  if (kVec) {
    const int n4 = n >> 2;
    for (int q = tid; q < n4; q += stride) {
      const int4 g = reinterpret_cast<const int4*>(gid)[q];
      const float4 w = reinterpret_cast<const float4*>(rewards)[q];
      if (g.x >= 0) moments_one(g.x, w.x, t);
      if (g.y >= 0) moments_one(g.y, w.y, t);
      if (g.z >= 0) moments_one(g.z, w.z, t);
      if (g.w >= 0) moments_one(g.w, w.w, t);
    }
  }
  const int first = kVec ? (n & ~3) : 0;
  for (int c = first + tid; c < n; c += stride) {
    const int g = gid[c];
    if (g >= 0) moments_one(g, rewards[c], t);
  }
}

__global__ void __launch_bounds__(kThreads)
k_hash_finalize(GroupTable t, int G, float std_eps, int ddof, float* __restrict__ group_mean,
                float* __restrict__ group_std, int32_t* __restrict__ group_best) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= G) return;
  GroupMoments* ge = t.m + g;
  const GroupHead hd = t.h[g];
  const unsigned K = hd.cnt;
  double mu = 0.0, sd = 0.0, inv = 0.0;
  if (K > 0) {
    const double lo = (double)dec_ordered(~hd.nmin);
    const double range = (double)dec_ordered(hd.emax) - lo;
    mu = lo;
    if (range > 0.0) {
      const bool big = K >= kBigGroup;
      const unsigned long long sx = ge->sum;
      const unsigned __int128 sxx =
          big ? (((unsigned __int128)t.sqhi[g] << 32) + ge->sq) : (unsigned __int128)ge->sq;
      const unsigned __int128 num = (unsigned __int128)K * sxx - (unsigned __int128)sx * sx;   // exact, >= 0
      const double step = range / (big ? kQuantBig : kQuantSmall);
      mu = lo + ((double)sx / (double)K) * step;
      const int dof = (int)K - ddof;
      if (dof > 0) {
        const double num_d = (double)(unsigned long long)(num >> 64) * 18446744073709551616.0 +
                             (double)(unsigned long long)num;
        sd = sqrt(num_d / ((double)K * (double)dof)) * step;
      }
    }
    if (K > 1) inv = 1.0 / (sd + (double)std_eps);
  }
  ge->sum = (unsigned long long)__double_as_longlong(mu);
  ge->sq = (unsigned long long)__double_as_longlong(inv);
  if (group_mean) group_mean[g] = (float)mu;
  if (group_std) group_std[g] = (float)sd;
  if (group_best) group_best[g] = K > 0 ? (int32_t)(0xFFFFFFFFu - (uint32_t)(t.best[g] & 0xFFFFFFFFull)) : -1;
}

// Eq. 3: reward = alpha * team + local, one fused multiply-add per candidate (correctly rounded).
__global__ void __launch_bounds__(kThreads)
k_mix_rewards(const float* __restrict__ team, const float* __restrict__ loc, float alpha, int n,
              float* __restrict__ out) {
  const int stride = gridDim.x * blockDim.x;
  for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < n; c += stride) out[c] = fmaf(alpha, team[c], loc[c]);
}

__device__ __forceinline__ float apply_one(int g, float r, const GroupTable& t) {
  const double2 mi = *reinterpret_cast<const double2*>(t.m + g);      // mean, 1/(std+eps): one 16-byte load
  return (float)(((double)r - mi.x) * mi.y);
}

template <bool kVec>
__global__ void __launch_bounds__(kThreads)
k_hash_apply(const int32_t* __restrict__ gid, const float* __restrict__ rewards, int n,
             GroupTable t, float* __restrict__ adv) {
  const int stride = gridDim.x * blockDim.x;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x;
  if (kVec) {
    const int n4 = n >> 2;
    for (int q = tid; q < n4; q += stride) {
      const int4 g = reinterpret_cast<const int4*>(gid)[q];
      const float4 w = reinterpret_cast<const float4*>(rewards)[q];
      float4 a;
      a.x = g.x >= 0 ? apply_one(g.x, w.x, t) : 0.f;
      a.y = g.y >= 0 ? apply_one(g.y, w.y, t) : 0.f;
      a.z = g.z >= 0 ? apply_one(g.z, w.z, t) : 0.f;
      a.w = g.w >= 0 ? apply_one(g.w, w.w, t) : 0.f;
      reinterpret_cast<float4*>(adv)[q] = a;
    }
  }
  const int first = kVec ? (n & ~3) : 0;
  for (int c = first + tid; c < n; c += stride) {
    const int g = gid[c];
    adv[c] = g >= 0 ? apply_one(g, rewards[c], t) : 0.f;
  }
}

// ------------------------------------------------------------------ (B) ordered statistics
struct StatsArgs {
  const float* rewards;
  const int32_t* offsets;
  const int32_t* gid;
  int32_t* perm;          // in: unordered buckets, out: ordered
  float* adv;
  float* group_mean;
  float* group_std;
  int G, n;
  float std_eps;
  int ddof;
};

// Fixed-order block sum of one double per thread.
__device__ __forceinline__ double block_sum_fixed(double v, double* red) {
  red[threadIdx.x] = v;
  __syncthreads();
  for (int s = kThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  const double r = red[0];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kThreads) k_group_stats(StatsArgs a) {
  __shared__ int idx_s[kCap];
  __shared__ __align__(16) float val_s[kCap];
  __shared__ int warp_tot[kThreads / 32];
  __shared__ int s_max;
  __shared__ int s_tot;
  double* red = reinterpret_cast<double*>(val_s);     // reused by the block-per-group path

  const int g0 = blockIdx.x * kThreads;
  const int g1 = min(g0 + kThreads, a.G);
  const int g = g0 + threadIdx.x;
  const int beg_blk = a.offsets[g0];
  const int n_blk = a.offsets[g1] - beg_blk;
  int beg = 0, K = 0;
  if (g < a.G) {
    beg = a.offsets[g];
    K = a.offsets[g + 1] - beg;
  }
  if (threadIdx.x == 0) s_max = 0;
  __syncthreads();
  atomicMax(&s_max, K);
  __syncthreads();
  const int max_k = s_max;

  if (n_blk <= kCap && max_k <= kSerialMaxK) {
    // ---------------- thread-per-group path ----------------
    for (int i = threadIdx.x; i < n_blk; i += kThreads) idx_s[i] = a.perm[beg_blk + i];
    __syncthreads();
    int* mine = idx_s + (beg - beg_blk);
    for (int i = 1; i < K; ++i) {                       // insertion sort, ascending candidate index
      const int x = mine[i];
      int j = i - 1;
      while (j >= 0 && mine[j] > x) {
        mine[j + 1] = mine[j];
        --j;
      }
      mine[j + 1] = x;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n_blk; i += kThreads) {
      const int c = idx_s[i];
      a.perm[beg_blk + i] = c;
      val_s[i] = a.rewards[c];
    }
    __syncthreads();
    if (g < a.G) {
      float* r = val_s + (beg - beg_blk);
      double mu = 0.0, sd = 0.0;
      if (K > 0) {
        double sum = 0.0;
        for (int i = 0; i < K; ++i) sum += (double)r[i];
        mu = sum / (double)K;
        double ss = 0.0;
        for (int i = 0; i < K; ++i) {
          const double dlt = (double)r[i] - mu;
          ss += dlt * dlt;
        }
        const int dof = K - a.ddof;
        sd = dof > 0 ? sqrt(ss / (double)dof) : 0.0;
        const double den = sd + (double)a.std_eps;
        for (int i = 0; i < K; ++i) r[i] = K > 1 ? (float)(((double)r[i] - mu) / den) : 0.f;
      }
      if (a.group_mean) a.group_mean[g] = (float)mu;
      if (a.group_std) a.group_std[g] = (float)sd;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n_blk; i += kThreads) a.adv[idx_s[i]] = val_s[i];
    return;
  }

  // ---------------- block-per-group path (a large group is present) ----------------
  for (int gg = g0; gg < g1; ++gg) {
    const int b = a.offsets[gg];
    const int Kg = a.offsets[gg + 1] - b;
    double mu = 0.0, sd = 0.0;
    if (Kg > 0) {
      int* p = a.perm + b;
      if (Kg <= kCap) {
        int n2 = 1;
        while (n2 < Kg) n2 <<= 1;
        for (int i = threadIdx.x; i < n2; i += kThreads) idx_s[i] = i < Kg ? p[i] : 0x7fffffff;
        __syncthreads();
        for (int k = 2; k <= n2; k <<= 1) {
          for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < n2; i += kThreads) {
              const int ixj = i ^ j;
              if (ixj > i) {
                const int x = idx_s[i], y = idx_s[ixj];
                const bool up = (i & k) == 0;
                if ((x > y) == up) {
                  idx_s[i] = y;
                  idx_s[ixj] = x;
                }
              }
            }
            __syncthreads();
          }
        }
        for (int i = threadIdx.x; i < Kg; i += kThreads) p[i] = idx_s[i];
        __syncthreads();
      } else {
        // ordered rescan of all candidates: members appear in ascending index by construction
        int run = 0;
        for (int base = 0; base < a.n; base += kThreads) {
          const int c = base + threadIdx.x;
          const int f = (c < a.n && a.gid[c] == gg) ? 1 : 0;
          const int incl = block_inclusive_scan(f, warp_tot);
          if (f) p[run + incl - 1] = c;
          if (threadIdx.x == kThreads - 1) s_tot = incl;
          __syncthreads();
          run += s_tot;
          __syncthreads();
        }
      }
      __threadfence_block();
      __syncthreads();
      // statistics: strided partial sums in a fixed order, fixed tree across threads
      double part = 0.0;
      for (int i = threadIdx.x; i < Kg; i += kThreads) part += (double)a.rewards[p[i]];
      mu = block_sum_fixed(part, red) / (double)Kg;
      part = 0.0;
      for (int i = threadIdx.x; i < Kg; i += kThreads) {
        const double dlt = (double)a.rewards[p[i]] - mu;
        part += dlt * dlt;
      }
      const double ss = block_sum_fixed(part, red);
      const int dof = Kg - a.ddof;
      sd = dof > 0 ? sqrt(ss / (double)dof) : 0.0;
      const double den = sd + (double)a.std_eps;
      for (int i = threadIdx.x; i < Kg; i += kThreads) {
        const int c = p[i];
        a.adv[c] = Kg > 1 ? (float)(((double)a.rewards[c] - mu) / den) : 0.f;
      }
    }
    if (threadIdx.x == 0) {
      if (a.group_mean) a.group_mean[gg] = (float)mu;
      if (a.group_std) a.group_std[gg] = (float)sd;
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------ (C) adjacent groups
// 4096 candidates a block owns per step, 16 per thread: measured against 2048 (8 % slower: the five
// block barriers, the run-list scan and the look-ahead are paid per tile), 6144 with three blocks per SM
// and 8192 with 512-thread blocks (both 10 % slower than 4096: fewer or larger blocks wait longer at
// the barriers)
constexpr int kRunTile = 4096;
constexpr int kRunHalo = 256;                        // look-ahead for runs that cross the end of a tile
constexpr int kRunWin = kRunTile + kRunHalo;

struct RunArgs {
  const float* rewards;
  const int32_t* env;
  const int32_t* role;
  const int32_t* turn;
  int n, n_env, n_role, n_turn;
  float* adv;
  int32_t* gid_out;        // optional
  int32_t* seen;           // [G], zeroed: runs started per group
  float* group_mean;       // optional, zeroed
  float* group_std;        // optional, zeroed
  float std_eps;
  int ddof;
  int32_t* status;
};

// `earlier` = runs of group g seen before this one (the value the atomic on seen[g] returned).
__device__ __forceinline__ void run_publish(const RunArgs& a, int g, int earlier, double mu, double sd) {
  if (earlier != 0) raise_status(a.status, ATGRPO_ERR_LAYOUT);
  if (a.group_mean) a.group_mean[g] = (float)mu;
  if (a.group_std) a.group_std[g] = (float)sd;
}

constexpr int kRunWarpK = 64;                        // runs longer than this are summed by a whole warp
constexpr int kRunRegK = 16;                         // runs up to this size are held in registers by their thread
constexpr int kRunPad = 4;                           // g_s[kRunPad + i] = key of staged candidate i (16-byte aligned quads)

// 1/k (correctly rounded by the compiler) for the divisions by a run's size in the thread-per-run
// path (k <= kRunWarpK = 64).
__constant__ double c_inv_k[kRunWarpK + 1] = {
    0.0, 1.0 / 1, 1.0 / 2, 1.0 / 3, 1.0 / 4, 1.0 / 5, 1.0 / 6, 1.0 / 7,
    1.0 / 8, 1.0 / 9, 1.0 / 10, 1.0 / 11, 1.0 / 12, 1.0 / 13, 1.0 / 14, 1.0 / 15,
    1.0 / 16, 1.0 / 17, 1.0 / 18, 1.0 / 19, 1.0 / 20, 1.0 / 21, 1.0 / 22, 1.0 / 23,
    1.0 / 24, 1.0 / 25, 1.0 / 26, 1.0 / 27, 1.0 / 28, 1.0 / 29, 1.0 / 30, 1.0 / 31,
    1.0 / 32, 1.0 / 33, 1.0 / 34, 1.0 / 35, 1.0 / 36, 1.0 / 37, 1.0 / 38, 1.0 / 39,
    1.0 / 40, 1.0 / 41, 1.0 / 42, 1.0 / 43, 1.0 / 44, 1.0 / 45, 1.0 / 46, 1.0 / 47,
    1.0 / 48, 1.0 / 49, 1.0 / 50, 1.0 / 51, 1.0 / 52, 1.0 / 53, 1.0 / 54, 1.0 / 55,
    1.0 / 56, 1.0 / 57, 1.0 / 58, 1.0 / 59, 1.0 / 60, 1.0 / 61, 1.0 / 62, 1.0 / 63,
    1.0 / 64,
};

// Std and 1/(std + eps) of one run of K members from its sum of squared deviations.
__device__ __forceinline__ void run_stats(double ss, int K, int ddof, float std_eps, double& sd, double& inv) {
  const int dof = K - ddof;
  sd = dof > 0 ? sqrt(K <= kRunWarpK ? ss * c_inv_k[dof] : ss / (double)dof) : 0.0;
  inv = K > 1 ? 1.0 / (sd + (double)std_eps) : 0.0;
}

// First set bit at index >= pos in a bit array that is known to have one (the sentinel).
__device__ __forceinline__ int next_boundary(const unsigned* bnd, int pos) {
  int w = pos >> 5;
  unsigned m = bnd[w] >> (pos & 31);
  if (m) return pos + __ffs(m) - 1;
  do m = bnd[++w];
  while (m == 0);
  return (w << 5) + __ffs(m) - 1;
}

constexpr int kRunBndWords = (kRunWin + 32) / 32 + 1;

// kVec: all five arrays are 16-byte aligned.  kPacked: a.env holds ready-made group ids in
// [0, n_env) and the role / turn arrays are not read (n_role = n_turn = 1).
template <bool kVec, bool kPacked>
__global__ void __launch_bounds__(kThreads, 4) k_run_advantages(RunArgs a) {
  __shared__ __align__(16) int g_s[kRunPad + kRunWin];     // g_s[kRunPad - 1] = key of the candidate before the tile
  __shared__ __align__(16) float r_s[kRunWin];             // rewards in; candidate i's advantage replaces its reward
  __shared__ unsigned bnd_s[kRunBndWords];                 // bit i: staged candidate i does not continue the run of i-1
  __shared__ unsigned short head_s[kRunTile];              // first members of the runs that start in the tile
  __shared__ unsigned short big_s[kRunTile / kRunWarpK + 1];   // those with more than kRunWarpK members
  __shared__ double red[kThreads];
  __shared__ int s_heads, s_big, s_lead, s_cross, s_long, s_end;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_tiles = (a.n + kRunTile - 1) / kRunTile;
  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int t0 = tile * kRunTile;
    const int own = min(kRunTile, a.n - t0);          // candidates whose runs this block owns
    const int cnt = min(kRunWin, a.n - t0);           // candidates staged
    // ---- stage keys and rewards
    const int n_quads = kVec ? cnt >> 2 : 0;
    if (kVec) {
#pragma unroll
      for (int e = 0; e < (kRunWin / 4 + kThreads - 1) / kThreads; ++e) {
        const int q = e * kThreads + threadIdx.x;
        if (q < n_quads) {
          const int c4 = (t0 >> 2) + q;
          const int4 ev = reinterpret_cast<const int4*>(a.env)[c4];
          const int4 zero = make_int4(0, 0, 0, 0);
          const int4 rv = kPacked ? zero : reinterpret_cast<const int4*>(a.role)[c4];
          const int4 tv = kPacked ? zero : reinterpret_cast<const int4*>(a.turn)[c4];
          const float4 w = reinterpret_cast<const float4*>(a.rewards)[c4];
          int4 g;
          g.x = group_of(ev.x, rv.x, tv.x, a.n_env, a.n_role, a.n_turn);
          g.y = group_of(ev.y, rv.y, tv.y, a.n_env, a.n_role, a.n_turn);
          g.z = group_of(ev.z, rv.z, tv.z, a.n_env, a.n_role, a.n_turn);
          g.w = group_of(ev.w, rv.w, tv.w, a.n_env, a.n_role, a.n_turn);
          *reinterpret_cast<int4*>(&g_s[kRunPad + 4 * q]) = g;
          *reinterpret_cast<float4*>(&r_s[4 * q]) = w;
          if (a.gid_out && 4 * q < own) *reinterpret_cast<int4*>(&a.gid_out[t0 + 4 * q]) = g;   // own % 4 == 0 here or the tail below
        }
      }
    }
    for (int i = 4 * n_quads + threadIdx.x; i < cnt; i += kThreads) {
      const int c = t0 + i;
      const int g = group_of(a.env[c], kPacked ? 0 : a.role[c], kPacked ? 0 : a.turn[c], a.n_env, a.n_role, a.n_turn);
      g_s[kRunPad + i] = g;
      r_s[i] = a.rewards[c];
      if (a.gid_out && i < own) a.gid_out[c] = g;
    }
    if (threadIdx.x < kRunBndWords) bnd_s[threadIdx.x] = 0u;
    if (threadIdx.x == 0) {
      g_s[kRunPad - 1] = t0 > 0 ? group_of(a.env[t0 - 1], kPacked ? 0 : a.role[t0 - 1], kPacked ? 0 : a.turn[t0 - 1],
                                           a.n_env, a.n_role, a.n_turn)
                                : -1;
      s_long = -1, s_heads = 0, s_big = 0;
    }
    __syncthreads();
    const int* gk = g_s + kRunPad;                    // gk[i] = key of staged candidate i, gk[-1] = the one before
    if (kVec && threadIdx.x < 4 && !(kPacked && (threadIdx.x == 1 || threadIdx.x == 2))) {
      // Blocks that start together stay in step (every tile costs the same), so without help all of
      // them load, then all of them compute.  Ask L2 for this block's next tile now: HBM then works
      // during the compute phases and the next staging loop finds its data in L2.
      const int nt = tile + gridDim.x;
      if (nt < n_tiles) {
        const int nb = nt * kRunTile;
        const int bytes = (min(kRunWin, a.n - nb) & ~3) * 4;
        const void* src = threadIdx.x == 0 ? (const void*)(a.env + nb)
                          : threadIdx.x == 1 ? (const void*)(a.role + nb)
                          : threadIdx.x == 2 ? (const void*)(a.turn + nb) : (const void*)(a.rewards + nb);
        if (bytes > 0)
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
      }
    }

    // ---- mark where runs begin (whole window) and list the runs that start inside the tile
    unsigned head_bits = 0;                           // bit 4*e + j: candidate 4*(e*kThreads + threadIdx.x) + j starts a run
#pragma unroll
    for (int e = 0; e < (kRunWin / 4 + kThreads - 1) / kThreads; ++e) {
      const int i0 = 4 * (e * kThreads + threadIdx.x);
      if (i0 < cnt) {
        const int4 g = *reinterpret_cast<const int4*>(&gk[i0]);
        const int prev = gk[i0 - 1];
        const int gg[5] = {prev, g.x, g.y, g.z, g.w};
        unsigned nib = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (i0 + j < cnt) {
            const bool bad = gg[j + 1] < 0;
            if (bad || gg[j + 1] != gg[j]) nib |= 1u << j;
            if (i0 + j < own) {
              if (bad) {
                r_s[i0 + j] = 0.f;
                raise_status(a.status, ATGRPO_ERR_BAD_INDEX);
              } else if (gg[j + 1] != gg[j]) {
                head_bits |= 1u << (4 * e + j);
              }
            }
          }
        }
        if (nib) atomicOr(&bnd_s[i0 >> 5], nib << (i0 & 31));
      }
    }
    if (threadIdx.x == 0) atomicOr(&bnd_s[cnt >> 5], 1u << (cnt & 31));   // sentinel: the window ends a run
    {
      // one shared-memory atomic per warp reserves the warp's slots in the run list
      const int mine = __popc(head_bits);
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += u;
      }
      int base = 0;
      if (lane == 31) base = atomicAdd(&s_heads, incl);
      base = __shfl_sync(0xffffffffu, base, 31);
      int pos = base + incl - mine;
      while (head_bits) {
        const int bit = __ffs(head_bits) - 1;
        head_bits &= head_bits - 1;
        head_s[pos++] = (unsigned short)(4 * ((bit >> 2) * kThreads + threadIdx.x) + (bit & 3));
      }
    }
    __syncthreads();

    // Thread 0: how many leading candidates continue a run the previous tile owns, and where the
    // run that crosses the end of this tile stops.
    if (threadIdx.x == 0) {
      s_lead = (bnd_s[0] & 1u) ? 0 : next_boundary(bnd_s, 1);
      s_cross = own < cnt ? next_boundary(bnd_s, own) : own;
    }
    // ---- one thread per run (the list is dense, so every lane works): sums in ascending order
    const int n_heads = s_heads;
    for (int h = threadIdx.x; h < n_heads; h += kThreads) {
      const int i = head_s[h];
      const int K = next_boundary(bnd_s, i + 1) - i;
      if (i + K == cnt && t0 + cnt < a.n) {           // may go on beyond the staged window
        s_long = i;
        continue;
      }
      if (K > kRunWarpK) {
        big_s[atomicAdd(&s_big, 1)] = (unsigned short)i;
        continue;
      }
      const int g = gk[i];
      const int earlier = atomicAdd(&a.seen[g], 1);   // issued early: its round trip overlaps the arithmetic
      // Shared memory is read at 32 unrelated offsets per warp (bank conflicts), so the members are
      // fetched ONCE into registers; everything after that is register arithmetic.
      float* p = r_s + i;
      double mu, sd = 0.0;
      bool done = false;
      if (K <= kRunRegK) {
        // Runs of up to 16 members, the common case: everything in fp32 on SHIFTED values
        // x = r - c, c = the run's first reward (exact for close values, 2^-24 relative otherwise;
        // identical rewards give x = 0 throughout, hence exact zeros).  Two passes: the mean of at
        // most 16 values of the run's own scale, then squared deviations, which cannot cancel.
        const float c = p[0];
        float x[kRunRegK];
#pragma unroll
        for (int k = 0; k < kRunRegK; ++k) x[k] = k < K ? p[k] - c : 0.f;
        float sum = 0.f, amax = 0.f;
#pragma unroll
        for (int k = 0; k < kRunRegK; ++k) {
          sum += x[k];                                // ascending order; the padding adds exact zeros
          amax = fmaxf(amax, fabsf(x[k]));
        }
        const float kf = (float)K;
        const float mean_x = __fdividef(sum, kf);
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < kRunRegK; ++k) {
          const float dlt = k < K ? x[k] - mean_x : 0.f;
          x[k] = dlt;
          ss = fmaf(dlt, dlt, ss);
        }
        // fp32 is trusted while the squares sit well inside its normal range (and for identical
        // rewards, whose deviations are exactly zero); otherwise the fp64 route below
        if (amax == 0.f || (ss > 1e-25f && ss < 1e30f)) {
          const int dof = K - a.ddof;
          const float var = dof > 0 ? __fdividef(ss, (float)dof) : 0.f;
          const float sdf = sqrtf(var);
          const float invf = amax != 0.f ? 1.0f / (sdf + a.std_eps) : 0.f;   // identical rewards (K = 1 too): exact zeros
#pragma unroll
          for (int k = 0; k < kRunRegK; ++k)
            if (k < K) p[k] = x[k] * invf;
          mu = (double)c + (double)mean_x;
          sd = (double)sdf;
          done = true;
        }
      }
      if (done) {
        // finished above
      } else if (K <= kRunRegK) {
        double v[kRunRegK];
#pragma unroll
        for (int k = 0; k < kRunRegK; ++k) v[k] = k < K ? (double)p[k] : 0.0;
        const double first = v[0];
        double sum = 0.0;
        bool all_eq = true;
#pragma unroll
        for (int k = 0; k < kRunRegK; ++k) {
          sum += v[k];                                // ascending order; the padding adds exact zeros
          all_eq = all_eq && (k >= K || v[k] == first);
        }
        mu = first;
        if (all_eq) {                                 // identical rewards: exact zeros, no rounding of the mean
#pragma unroll
          for (int k = 0; k < kRunRegK; ++k)
            if (k < K) p[k] = 0.f;
        } else {
          mu = sum * c_inv_k[K];
          double ss = 0.0;
#pragma unroll
          for (int k = 0; k < kRunRegK; ++k) {
            const double dlt = k < K ? v[k] - mu : 0.0;
            ss = fma(dlt, dlt, ss);
          }
          // only runs whose squares leave the comfortable fp32 range get here: fp64 throughout
          double inv;
          run_stats(ss, K, a.ddof, a.std_eps, sd, inv);
#pragma unroll
          for (int k = 0; k < kRunRegK; ++k)
            if (k < K) p[k] = (float)((v[k] - mu) * inv);
        }
      } else {
        const double first = (double)p[0];
        double sum = 0.0;
        bool all_eq = true;
        for (int k = 0; k < K; ++k) {
          const double v = (double)p[k];
          sum += v;
          all_eq = all_eq && (v == first);
        }
        mu = first;
        if (all_eq) {
          for (int k = 0; k < K; ++k) p[k] = 0.f;
        } else {
          mu = sum * c_inv_k[K];
          double ss = 0.0;
          for (int k = 0; k < K; ++k) {
            const double dlt = (double)p[k] - mu;
            ss = fma(dlt, dlt, ss);
          }
          double inv;
          run_stats(ss, K, a.ddof, a.std_eps, sd, inv);
          for (int k = 0; k < K; ++k) p[k] = (float)(((double)p[k] - mu) * inv);
        }
      }
      run_publish(a, g, earlier, mu, sd);
    }
    __syncthreads();

    // ---- runs of more than kRunWarpK members inside the window: one warp each, lane-strided
    // partial sums in ascending order and a fixed shuffle tree
    const int n_big = s_big;
    for (int b = warp; b < n_big; b += kThreads / 32) {
      const int i = big_s[b];
      const int g = gk[i];
      const int K = next_boundary(bnd_s, i + 1) - i;
      double part = 0.0;
      for (int k = lane; k < K; k += 32) part += (double)r_s[i + k];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      const double mu = part / (double)K;
      part = 0.0;
      for (int k = lane; k < K; k += 32) {
        const double dlt = (double)r_s[i + k] - mu;
        part += dlt * dlt;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      double sd, inv;
      run_stats(part, K, a.ddof, a.std_eps, sd, inv);
      for (int k = lane; k < K; k += 32) r_s[i + k] = (float)(((double)r_s[i + k] - mu) * inv);
      if (lane == 0) run_publish(a, g, atomicAdd(&a.seen[g], 1), mu, sd);
    }
    if (n_big > 0) __syncthreads();                   // n_big is the same in every thread: no barrier for the usual tile

    // ---- the tile leaves with coalesced stores
    const int lh = s_long;
    const int lo = s_lead, hi = lh >= 0 ? lh : s_cross;   // the long run is written by the block path below
    if (kVec) {
      const int q_lo = (lo + 3) >> 2, q_hi = hi >> 2;      // whole quads inside [lo, hi)
      for (int q = q_lo + threadIdx.x; q < q_hi; q += kThreads)
        reinterpret_cast<float4*>(a.adv + t0)[q] = *reinterpret_cast<const float4*>(&r_s[4 * q]);
      if (q_lo < q_hi) {
        if ((int)threadIdx.x < 4 * q_lo - lo) a.adv[t0 + lo + threadIdx.x] = r_s[lo + threadIdx.x];
        if ((int)threadIdx.x < hi - 4 * q_hi) a.adv[t0 + 4 * q_hi + threadIdx.x] = r_s[4 * q_hi + threadIdx.x];
      } else {
        for (int i = lo + threadIdx.x; i < hi; i += kThreads) a.adv[t0 + i] = r_s[i];
      }
    } else {
      for (int i = lo + threadIdx.x; i < hi; i += kThreads) a.adv[t0 + i] = r_s[i];
    }

    if (lh >= 0) {
      // ---- a run that outgrew the window: the whole block reduces it from global memory
      const int g = gk[lh];
      const int beg = t0 + lh;
      int end = t0 + cnt;                             // equal up to here
      for (;;) {
        const int c = end + threadIdx.x;
        const bool same = c < a.n && group_of(a.env[c], kPacked ? 0 : a.role[c], kPacked ? 0 : a.turn[c], a.n_env,
                                              a.n_role, a.n_turn) == g;
        const int n_same = __syncthreads_count(same);
        if (n_same == kThreads) {
          end += kThreads;
          continue;
        }
        // first mismatch inside this chunk: members are the threads before it
        if (threadIdx.x == 0) s_end = a.n;
        __syncthreads();
        if (!same) atomicMin(&s_end, c);
        __syncthreads();
        end = min(s_end, a.n);
        break;
      }
      const int K = end - beg;                        // > kRunHalo
      double part = 0.0;
      for (int c = beg + threadIdx.x; c < end; c += kThreads) part += (double)a.rewards[c];
      const double mu = block_sum_fixed(part, red) / (double)K;
      part = 0.0;
      for (int c = beg + threadIdx.x; c < end; c += kThreads) {
        const double dlt = (double)a.rewards[c] - mu;
        part += dlt * dlt;
      }
      const double ss = block_sum_fixed(part, red);
      double sd, inv;
      run_stats(ss, K, a.ddof, a.std_eps, sd, inv);
      for (int c = beg + threadIdx.x; c < end; c += kThreads)
        a.adv[c] = (float)(((double)a.rewards[c] - mu) * inv);
      if (threadIdx.x == 0) run_publish(a, g, atomicAdd(&a.seen[g], 1), mu, sd);
    }
    __syncthreads();                                  // the tile's shared memory is reused
  }
}

struct Plan {
  size_t count, slot, gid, offsets, perm, block_sum;   // pipeline (B)
  size_t h_gid, h_table;                               // pipeline (A): gid[n], then 40 bytes per slot
  size_t total;
};
Plan make_plan(int64_t n, int64_t G) {
  Plan p;
  Carver c(nullptr);
  p.count = c.off; c.take<int32_t>((size_t)G);
  p.slot = c.off; c.take<int32_t>((size_t)n);
  p.gid = c.off; c.take<int32_t>((size_t)n);
  p.offsets = c.off; c.take<int32_t>((size_t)G + 1);
  p.perm = c.off; c.take<int32_t>((size_t)n);
  p.block_sum = c.off; c.take<int32_t>((size_t)((G + kScanBlock - 1) / kScanBlock) + 1);
  Carver h(nullptr);                                   // the two pipelines never run together:
  p.h_gid = h.off; h.take<int32_t>((size_t)n);         // they share the same bytes
  p.h_table = h.off; h.take<unsigned long long>((size_t)G * 5 + 8);   // two 16-byte entries + one overflow word per slot
  p.total = c.off > h.off ? c.off : h.off;
  return p;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

size_t group_select_workspace_bytes(int64_t n_cand, int64_t n_groups) {
  const int64_t n = n_cand < 0 ? 0 : n_cand, G = n_groups < 0 ? 0 : n_groups;
  Carver x(nullptr);
  x.take<float>((size_t)n + 1);
  x.take<unsigned long long>((size_t)G + 1);
  return make_plan(n, G).total + x.off;
}

size_t group_adv_workspace_bytes(int64_t n_cand, int64_t n_groups) {
  return make_plan(n_cand < 0 ? 0 : n_cand, n_groups < 0 ? 0 : n_groups).total;
}

int group_adv_launch(const float* rewards, const int32_t* env_id, const int32_t* role_id,
                     const int32_t* turn_id, int64_t n_cand, int32_t n_env, int32_t n_role,
                     int32_t n_turn, const atgrpo_params& prm, float* adv, int32_t* group_of_cand,
                     int32_t* group_offsets, int32_t* group_perm, float* group_mean,
                     float* group_std, int32_t* device_status, void* workspace, cudaStream_t st,
                     const GroupExtras* ex, bool packed) {
  // packed: env_id holds ready-made group ids in [0, n_env); role_id / turn_id are not read
  if (packed) n_role = 1, n_turn = 1;
  const int64_t G = (int64_t)n_env * n_role * n_turn;
  const int n = (int)n_cand;
  const Plan pl = make_plan(n_cand, G);
  char* ws = static_cast<char*>(workspace);
  // Optional Eq. 3 mix and greedy argmax: their scratch follows the regular plan.
  unsigned long long* best = nullptr;
  int32_t* group_best = nullptr;
  if (ex != nullptr) {
    Carver x(ws + pl.total);
    float* mixed = x.take<float>((size_t)n + 1);
    best = x.take<unsigned long long>((size_t)G + 1);
    group_best = ex->group_best;
    if (ex->r_team != nullptr && n > 0) {
      float* dst = ex->rewards_out ? ex->rewards_out : mixed;
      int64_t mg = ((int64_t)n + kThreads - 1) / kThreads;
      if (mg > 148 * 16) mg = 148 * 16;
      k_mix_rewards<<<(int)mg, kThreads, 0, st>>>(ex->r_team, ex->r_loc, ex->alpha, n, dst);
      rewards = dst;
    }
    if (group_best == nullptr) best = nullptr;
    else if (n == 0) ATGRPO_CUDA_OK(cudaMemsetAsync(group_best, 0xFF, (size_t)G * sizeof(int32_t), st));
    else ATGRPO_CUDA_OK(cudaMemsetAsync(best, 0, (size_t)G * sizeof(unsigned long long), st));
  }
  int32_t* count = reinterpret_cast<int32_t*>(ws + pl.count);
  int32_t* slot = reinterpret_cast<int32_t*>(ws + pl.slot);
  int32_t* gid = group_of_cand ? group_of_cand : reinterpret_cast<int32_t*>(ws + pl.gid);
  int32_t* offsets = group_offsets ? group_offsets : reinterpret_cast<int32_t*>(ws + pl.offsets);
  int32_t* perm = group_perm ? group_perm : reinterpret_cast<int32_t*>(ws + pl.perm);
  int32_t* block_sum = reinterpret_cast<int32_t*>(ws + pl.block_sum);

  if (n > 0 && group_offsets == nullptr && group_perm == nullptr && ex == nullptr && prm.candidates_grouped) {
    // (C) adjacent groups: one streaming pass
    ATGRPO_CUDA_OK(cudaMemsetAsync(count, 0, (size_t)G * sizeof(int32_t), st));
    if (group_mean) ATGRPO_CUDA_OK(cudaMemsetAsync(group_mean, 0, (size_t)G * sizeof(float), st));
    if (group_std) ATGRPO_CUDA_OK(cudaMemsetAsync(group_std, 0, (size_t)G * sizeof(float), st));
    RunArgs a{rewards, env_id, role_id, turn_id, n, n_env, n_role, n_turn, adv, group_of_cand, count,
              group_mean, group_std, prm.std_eps, prm.ddof, device_status};
    const int n_tiles = (n + kRunTile - 1) / kRunTile;
    const bool vec = aligned16(env_id) && (packed || (aligned16(role_id) && aligned16(turn_id))) &&
                     aligned16(rewards) && aligned16(adv) && (group_of_cand == nullptr || aligned16(group_of_cand));
    // one resident wave of blocks; each walks its tiles with a grid stride
    int dev = 0, n_sm = 148, per_sm = 0;
    ATGRPO_CUDA_OK(cudaGetDevice(&dev));
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm <= 0) n_sm = 148;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_run_advantages<true, false>, kThreads, 0) !=
            cudaSuccess || per_sm <= 0)
      per_sm = 4;
    const int grid = n_tiles < per_sm * n_sm ? n_tiles : per_sm * n_sm;
    if (packed) {
      if (vec) k_run_advantages<true, true><<<grid, kThreads, 0, st>>>(a);
      else k_run_advantages<false, true><<<grid, kThreads, 0, st>>>(a);
    } else {
      if (vec) k_run_advantages<true, false><<<grid, kThreads, 0, st>>>(a);
      else k_run_advantages<false, false><<<grid, kThreads, 0, st>>>(a);
    }
    return launch_ok();
  }
  if (n > 0 && group_offsets == nullptr && group_perm == nullptr) {
    // (A) advantages only
    int32_t* hgid = group_of_cand ? group_of_cand : reinterpret_cast<int32_t*>(ws + pl.h_gid);
    char* tb = ws + pl.h_table;
    GroupTable t;
    t.h = reinterpret_cast<GroupHead*>(tb);
    t.m = reinterpret_cast<GroupMoments*>(tb + (size_t)G * 16);
    t.sqhi = reinterpret_cast<unsigned long long*>(tb + (size_t)G * 32);
    t.best = best;
    ATGRPO_CUDA_OK(cudaMemsetAsync(tb, 0, (size_t)G * 40, st));
    const bool v1 = aligned16(env_id) && (packed || (aligned16(role_id) && aligned16(turn_id))) &&
                    aligned16(rewards) && aligned16(hgid);
    const bool v2 = aligned16(rewards) && aligned16(hgid);
    const bool v3 = v2 && aligned16(adv);
    auto grid_of = [&](bool v) {
      int64_t b = ((v ? (n + 3) / 4 : n) + kThreads - 1) / kThreads;
      return (int)(b > 148 * 16 ? 148 * 16 : b);
    };
#define ATGRPO_MINMAX(V, P)                                                                                 \
  k_hash_minmax<V, P><<<grid_of(V), kThreads, 0, st>>>(env_id, role_id, turn_id, rewards, n, n_env, n_role, \
                                                       n_turn, t, hgid, adv, device_status)
    if (packed) {
      if (v1) ATGRPO_MINMAX(true, true);
      else ATGRPO_MINMAX(false, true);
    } else {
      if (v1) ATGRPO_MINMAX(true, false);
      else ATGRPO_MINMAX(false, false);
    }
#undef ATGRPO_MINMAX
    if (v2) k_hash_moments<true><<<grid_of(true), kThreads, 0, st>>>(hgid, rewards, n, t);
    else k_hash_moments<false><<<grid_of(false), kThreads, 0, st>>>(hgid, rewards, n, t);
    k_hash_finalize<<<(int)((G + kThreads - 1) / kThreads), kThreads, 0, st>>>(t, (int)G, prm.std_eps, prm.ddof,
                                                                               group_mean, group_std, group_best);
    if (v3) k_hash_apply<true><<<grid_of(true), kThreads, 0, st>>>(hgid, rewards, n, t, adv);
    else k_hash_apply<false><<<grid_of(false), kThreads, 0, st>>>(hgid, rewards, n, t, adv);
    return launch_ok();
  }

  ATGRPO_CUDA_OK(cudaMemsetAsync(count, 0, (size_t)G * sizeof(int32_t), st));
  if (n == 0) {
    ATGRPO_CUDA_OK(cudaMemsetAsync(offsets, 0, ((size_t)G + 1) * sizeof(int32_t), st));
    if (group_mean) ATGRPO_CUDA_OK(cudaMemsetAsync(group_mean, 0, (size_t)G * sizeof(float), st));
    if (group_std) ATGRPO_CUDA_OK(cudaMemsetAsync(group_std, 0, (size_t)G * sizeof(float), st));
    return ATGRPO_OK;
  }
  const bool vec = aligned16(env_id) && (packed || (aligned16(role_id) && aligned16(turn_id))) &&
                   aligned16(gid) && aligned16(slot);
  const int work = vec ? (n + 3) / 4 : n;
  const int grid_c = (int)((work + kThreads - 1) / kThreads);
#define ATGRPO_KEYCOUNT(V, P)                                                                          \
  k_key_count<V, P><<<grid_c, kThreads, 0, st>>>(env_id, role_id, turn_id, n, n_env, n_role, n_turn, count, \
                                                 slot, gid, adv, device_status)
  if (packed) {
    if (vec) ATGRPO_KEYCOUNT(true, true);
    else ATGRPO_KEYCOUNT(false, true);
  } else {
    if (vec) ATGRPO_KEYCOUNT(true, false);
    else ATGRPO_KEYCOUNT(false, false);
  }
#undef ATGRPO_KEYCOUNT
  const int nb = (int)((G + kScanBlock - 1) / kScanBlock);
  k_block_sums<<<nb, kThreads, 0, st>>>(count, (int)G, block_sum);
  k_scan_offsets<<<nb, kThreads, 0, st>>>(count, (int)G, block_sum, offsets);
  k_scatter<<<(n + kThreads - 1) / kThreads, kThreads, 0, st>>>(gid, slot, offsets, n, perm);
  StatsArgs a{rewards, offsets, gid, perm, adv, group_mean, group_std, (int)G, n, prm.std_eps,
              prm.ddof};
  k_group_stats<<<(int)((G + kThreads - 1) / kThreads), kThreads, 0, st>>>(a);
  return launch_ok();
}

}  // namespace atgrpo
