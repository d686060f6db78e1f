// Agent- and turn-wise grouped advantage (Eq. 1 over the groups of Algorithm 1).
//
// Two pipelines, both on the caller's stream with no host synchronisation.
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

template <bool kVec>
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
      const int4 r = reinterpret_cast<const int4*>(role)[q];
      const int4 t = reinterpret_cast<const int4*>(turn)[q];
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
    const int g = group_of(env[c], role[c], turn[c], n_env, n_role, n_turn);
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

template <bool kVec>
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
      const int4 r = reinterpret_cast<const int4*>(role)[q];
      const int4 u = reinterpret_cast<const int4*>(turn)[q];
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
    const int g = group_of(env[c], role[c], turn[c], n_env, n_role, n_turn);
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
                     const GroupExtras* ex) {
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
    const bool v1 = aligned16(env_id) && aligned16(role_id) && aligned16(turn_id) &&
                    aligned16(rewards) && aligned16(hgid);
    const bool v2 = aligned16(rewards) && aligned16(hgid);
    const bool v3 = v2 && aligned16(adv);
    auto grid_of = [&](bool v) {
      int64_t b = ((v ? (n + 3) / 4 : n) + kThreads - 1) / kThreads;
      return (int)(b > 148 * 16 ? 148 * 16 : b);
    };
    if (v1)
      k_hash_minmax<true><<<grid_of(true), kThreads, 0, st>>>(env_id, role_id, turn_id, rewards, n, n_env,
                                                              n_role, n_turn, t, hgid, adv, device_status);
    else
      k_hash_minmax<false><<<grid_of(false), kThreads, 0, st>>>(env_id, role_id, turn_id, rewards, n, n_env,
                                                                n_role, n_turn, t, hgid, adv, device_status);
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
  const bool vec = aligned16(env_id) && aligned16(role_id) && aligned16(turn_id) &&
                   aligned16(gid) && aligned16(slot);
  const int work = vec ? (n + 3) / 4 : n;
  const int grid_c = (int)((work + kThreads - 1) / kThreads);
  if (vec)
    k_key_count<true><<<grid_c, kThreads, 0, st>>>(env_id, role_id, turn_id, n, n_env, n_role,
                                                   n_turn, count, slot, gid, adv, device_status);
  else
    k_key_count<false><<<grid_c, kThreads, 0, st>>>(env_id, role_id, turn_id, n, n_env, n_role,
                                                    n_turn, count, slot, gid, adv, device_status);
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
