// Eq. 2 reduction over response tokens, token routing to policies (B_m of Sec. 3), and the row
// gather that lays the hidden states out policy by policy in 128-row tiles.
#include "internal.h"

namespace atgrpo {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 1184;     // 148 SMs x 8 resident blocks of 256 threads

struct LossArgs {
  const float* logp;
  const float* old_logp;
  const int32_t* resp;
  const float* adv;
  int64_t n_resp;
  const int32_t* role;
  const int32_t* head_of_role;
  int n_role, M;
  int64_t T;
  float lo, hi;                // 1 - eps_low, 1 + eps_high
  float* loss;
  float* coef;                 // optional, single-policy only
  int64_t* clip_counts;        // optional [M,2]
  int32_t* status;
  double* part_sum;            // [grid, M]
  int64_t* part_cnt;           // [grid, M, 3] tokens, clipped-low, clipped-high
  unsigned* done;
  int vec;                     // logp, old_logp, resp (and coef) are 16-byte aligned
  int64_t* head_cnt;           // optional [M]: items counted per head (sequence mode keeps it for backward)
  const float* seg_term;       // sequence mode: per-response term, stored at the response's first token
  const int32_t* seg_flags;    // sequence mode: bit 0 ratio below 1-eps_low, bit 1 above 1+eps_high,
                               // bit 2 first response seen of its group, bit 3 response left out (bad group id)
  const int32_t* group_of_resp;   // group-mean mode: group of every response
  const int32_t* group_cnt;       // group-mean mode: K_g, responses with tokens per group
};

// Per-token term of Eq. 2.  Returns l_j; `active` tells whether the unclipped branch carries the
// gradient (ties pass it, A = 0 does not).
__device__ __forceinline__ float clipped_term(float logp, float old_logp, float A, float lo,
                                              float hi, float& rho, bool& active) {
  rho = expf(logp - old_logp);
  const float rc = fminf(fmaxf(rho, lo), hi);
  const float u = rho * A, c = rc * A;
  active = (u <= c) && (A != 0.f);
  return -fminf(u, c);
}

struct TokenAcc {
  double sum;
  int cnt, clo, chi;
};

template <int kHeads>
__device__ __forceinline__ void loss_token(const LossArgs& a, int64_t j, float logp, float old_logp,
                                           int rs, float inv_T, TokenAcc* acc) {
  int head = 0;
  if (kHeads != 1) {
    const int r = a.role[j];
    head = (unsigned)r < (unsigned)a.n_role ? a.head_of_role[r] : -1;
    if ((unsigned)head >= (unsigned)a.M) {
      raise_status(a.status, ATGRPO_ERR_BAD_INDEX);
      return;
    }
  }
  float A = 0.f;
  if ((unsigned)rs < (unsigned)a.n_resp) A = a.adv[rs];
  else raise_status(a.status, ATGRPO_ERR_BAD_INDEX);
  float rho;
  bool active;
  const float l = clipped_term(logp, old_logp, A, a.lo, a.hi, rho, active);
  if (kHeads == 1 && a.coef) a.coef[j] = active ? A * rho * inv_T : 0.f;
#pragma unroll
  for (int m = 0; m < (kHeads == 1 ? 1 : ATGRPO_MAX_HEADS); ++m) {
    if (m == head) {
      acc[m].sum += (double)l;
      acc[m].cnt += 1;
      acc[m].clo += rho < a.lo;
      acc[m].chi += rho > a.hi;
    }
  }
}

// Fixed-order reduction of the per-thread accumulators: shuffle tree inside each warp, one thread
// per head across the warps, per-block partials, and the block that finishes last adds the
// partials (fixed strided subsets, fixed tree), so the result never depends on block timing.
template <int kHeads>
__device__ __forceinline__ void reduce_and_finish(TokenAcc* acc, const LossArgs& a) {
  constexpr int H = kHeads == 1 ? 1 : ATGRPO_MAX_HEADS;
  __shared__ double s_sum[kThreads / 32][H];
  __shared__ int s_cnt[kThreads / 32][H][3];
  __shared__ bool s_last;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int M = kHeads == 1 ? 1 : a.M;
#pragma unroll
  for (int m = 0; m < H; ++m) {
    if (m < M) {
      double v = acc[m].sum;
      int c0 = acc[m].cnt, c1 = acc[m].clo, c2 = acc[m].chi;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        v += __shfl_down_sync(0xffffffffu, v, o);
        c0 += __shfl_down_sync(0xffffffffu, c0, o);
        c1 += __shfl_down_sync(0xffffffffu, c1, o);
        c2 += __shfl_down_sync(0xffffffffu, c2, o);
      }
      if (lane == 0) {
        s_sum[w][m] = v;
        s_cnt[w][m][0] = c0, s_cnt[w][m][1] = c1, s_cnt[w][m][2] = c2;
      }
    }
  }
  __syncthreads();
  if ((int)threadIdx.x < M) {
    const int m = threadIdx.x;
    double v = 0.0;
    int64_t c0 = 0, c1 = 0, c2 = 0;
    for (int i = 0; i < kThreads / 32; ++i) {
      v += s_sum[i][m];
      c0 += s_cnt[i][m][0], c1 += s_cnt[i][m][1], c2 += s_cnt[i][m][2];
    }
    a.part_sum[(size_t)blockIdx.x * M + m] = v;
    int64_t* pc = a.part_cnt + ((size_t)blockIdx.x * M + m) * 3;
    pc[0] = c0, pc[1] = c1, pc[2] = c2;
  }
  // the block that finishes last adds the per-block partials: each thread a fixed strided
  // subset, then a fixed tree, so the order never depends on which block came last
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(a.done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  __shared__ double r_sum[kThreads];
  __shared__ long long r_cnt[kThreads][3];
  for (int m = 0; m < M; ++m) {
    double v = 0.0;
    long long c0 = 0, c1 = 0, c2 = 0;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += kThreads) {
      v += a.part_sum[(size_t)b * M + m];
      const int64_t* pc = a.part_cnt + ((size_t)b * M + m) * 3;
      c0 += pc[0], c1 += pc[1], c2 += pc[2];
    }
    r_sum[threadIdx.x] = v;
    r_cnt[threadIdx.x][0] = c0, r_cnt[threadIdx.x][1] = c1, r_cnt[threadIdx.x][2] = c2;
    __syncthreads();
    for (int s2 = kThreads / 2; s2 > 0; s2 >>= 1) {
      if ((int)threadIdx.x < s2) {
        r_sum[threadIdx.x] += r_sum[threadIdx.x + s2];
        r_cnt[threadIdx.x][0] += r_cnt[threadIdx.x + s2][0];
        r_cnt[threadIdx.x][1] += r_cnt[threadIdx.x + s2][1];
        r_cnt[threadIdx.x][2] += r_cnt[threadIdx.x + s2][2];
      }
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      if (a.head_cnt) a.head_cnt[m] = r_cnt[0][0];
      if (a.loss) a.loss[m] = r_cnt[0][0] > 0 ? (float)(r_sum[0] / (double)r_cnt[0][0]) : 0.f;
      if (a.clip_counts) a.clip_counts[2 * m] = r_cnt[0][1], a.clip_counts[2 * m + 1] = r_cnt[0][2];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) *a.done = 0;
}

template <int kHeads>   // 1: single policy, no routing arrays; 0: generic (a.M heads)
__global__ void __launch_bounds__(kThreads) k_clipped_loss(LossArgs a) {
  constexpr int H = kHeads == 1 ? 1 : ATGRPO_MAX_HEADS;
  TokenAcc acc[H];
#pragma unroll
  for (int m = 0; m < H; ++m) acc[m].sum = 0.0, acc[m].cnt = 0, acc[m].clo = 0, acc[m].chi = 0;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const float inv_T = a.T > 0 ? 1.f / (float)a.T : 0.f;
  // Four consecutive tokens per thread and iteration (16-byte loads) when the arrays allow it.  The
  // loads of the next iteration are issued before the current one is worked on, so a warp's
  // streaming loads overlap its advantage gathers and arithmetic (all warps start in step, and
  // without this every round of loads waited for the previous round's arithmetic).
  const int64_t n4 = a.vec ? a.T >> 2 : 0;
  int64_t q = tid;
  float4 lp = make_float4(0.f, 0.f, 0.f, 0.f), lo = lp;
  int4 rs = make_int4(0, 0, 0, 0);
  if (q < n4) {
    lp = reinterpret_cast<const float4*>(a.logp)[q];
    lo = reinterpret_cast<const float4*>(a.old_logp)[q];
    rs = reinterpret_cast<const int4*>(a.resp)[q];
  }
  while (q < n4) {
    const int64_t qn = q + stride;
    float4 lp_n = lp, lo_n = lo;
    int4 rs_n = rs;
    if (qn < n4) {
      lp_n = reinterpret_cast<const float4*>(a.logp)[qn];
      lo_n = reinterpret_cast<const float4*>(a.old_logp)[qn];
      rs_n = reinterpret_cast<const int4*>(a.resp)[qn];
    }
    loss_token<kHeads>(a, 4 * q + 0, lp.x, lo.x, rs.x, inv_T, acc);
    loss_token<kHeads>(a, 4 * q + 1, lp.y, lo.y, rs.y, inv_T, acc);
    loss_token<kHeads>(a, 4 * q + 2, lp.z, lo.z, rs.z, inv_T, acc);
    loss_token<kHeads>(a, 4 * q + 3, lp.w, lo.w, rs.w, inv_T, acc);
    q = qn, lp = lp_n, lo = lo_n, rs = rs_n;
  }
  for (int64_t j = 4 * n4 + tid; j < a.T; j += stride)
    loss_token<kHeads>(a, j, a.logp[j], a.old_logp[j], a.resp[j], inv_T, acc);

  reduce_and_finish<kHeads>(acc, a);
}

// ------------------------------------------------------------------ sequence-level Eq. 2
// Eq. 2 as printed: one ratio per response, r_c = exp(sum_j logp_j - sum_j old_logp_j), and the
// mean over the responses of the policy's batch.  Tokens are packed response by response
// (resp_of_token non-decreasing), so a response is a segment found by binary search; one warp per
// response sums its tokens in a fixed order.  Per-response results are parked at the response's
// first token, which keeps the scratch proportional to T.
// Group-mean mode (the expectation of Eq. 2 as printed): the response pass also counts K_g, the
// responses with tokens of every group (integer atomics: order-free), and marks the response that
// found its group's counter at zero, so the reduction can count the groups G_m; the reduction then
// adds term_c / K_g and divides by G_m.
__device__ __forceinline__ int64_t lower_bound_resp(const int32_t* resp, int64_t T, int c) {
  int64_t lo = 0, hi = T;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (resp[mid] < c) lo = mid + 1;
    else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(kThreads)
k_seq_resp(const float* __restrict__ logp, const float* __restrict__ old_logp,
           const int32_t* __restrict__ resp, const float* __restrict__ adv, int64_t n_resp, int64_t T,
           float lo, float hi, float* __restrict__ seg_term, int32_t* __restrict__ seg_flags,
           float* __restrict__ coef_un, const int32_t* __restrict__ group_of_resp,
           int32_t* __restrict__ group_cnt, int n_groups, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
  for (int64_t c = (int64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); c < n_resp; c += warps) {
    const int64_t beg = lower_bound_resp(resp, T, (int)c);
    const int64_t end = lower_bound_resp(resp, T, (int)c + 1);
    if (beg >= end) continue;                                  // a response without tokens
    double part = 0.0;
    for (int64_t j = beg + lane; j < end; j += 32) part += (double)logp[j] - (double)old_logp[j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    const double A = (double)adv[c];
    const double rho = exp(part);
    const double rc = fmin(fmax(rho, (double)lo), (double)hi);
    const double u = rho * A, cl = rc * A;
    const bool active = (u <= cl) && (A != 0.0);
    int gflag = 0;
    if (group_cnt != nullptr) {
      if (lane == 0) {
        const int g = group_of_resp[c];
        if ((unsigned)g < (unsigned)n_groups) {
          gflag = atomicAdd(&group_cnt[g], 1) == 0 ? 4 : 0;
        } else {
          gflag = 8;
          raise_status(status, ATGRPO_ERR_BAD_INDEX);
        }
      }
      gflag = __shfl_sync(0xffffffffu, gflag, 0);
    }
    if (lane == 0) {
      seg_term[beg] = (float)(-fmin(u, cl));
      seg_flags[beg] = (rho < (double)lo ? 1 : 0) | (rho > (double)hi ? 2 : 0) | gflag;
    }
    if (coef_un) {
      const float cu = (active && !(gflag & 8)) ? (float)(A * rho) : 0.f;
      for (int64_t j = beg + lane; j < end; j += 32) coef_un[j] = cu;
    }
  }
}

template <int kHeads>
__global__ void __launch_bounds__(kThreads) k_seq_reduce(LossArgs a) {
  constexpr int H = kHeads == 1 ? 1 : ATGRPO_MAX_HEADS;
  TokenAcc acc[H];
#pragma unroll
  for (int m = 0; m < H; ++m) acc[m].sum = 0.0, acc[m].cnt = 0, acc[m].clo = 0, acc[m].chi = 0;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < a.T; j += stride) {
    const int rs = a.resp[j];
    const int prev = j > 0 ? a.resp[j - 1] : -1;
    if (rs < prev || (unsigned)rs >= (unsigned)a.n_resp) raise_status(a.status, ATGRPO_ERR_BAD_INDEX);
    if (rs == prev || (unsigned)rs >= (unsigned)a.n_resp) continue;        // not the first token of a response
    int head = 0;
    if (kHeads != 1) {
      const int r = a.role[j];
      head = (unsigned)r < (unsigned)a.n_role ? a.head_of_role[r] : -1;
      if ((unsigned)head >= (unsigned)a.M) {
        raise_status(a.status, ATGRPO_ERR_BAD_INDEX);
        continue;
      }
    }
    const int fl = a.seg_flags[j];
    if (fl & 8) continue;                                                    // left out: bad group id
    double term = (double)a.seg_term[j];
    int item = 1;
    if (a.group_cnt != nullptr) {
      term /= (double)a.group_cnt[a.group_of_resp[rs]];                      // K_g >= 1: this response counted itself
      item = (fl >> 2) & 1;                                                  // one response per group counts the group
    }
#pragma unroll
    for (int m = 0; m < H; ++m) {
      if (m == head) {
        acc[m].sum += term;
        acc[m].cnt += item;
        acc[m].clo += fl & 1;
        acc[m].chi += (fl >> 1) & 1;
      }
    }
  }
  reduce_and_finish<kHeads>(acc, a);
}

// coef[j] (holding A*rho*[active] of the token's response) *= grad_loss[m] / R_m, or
// grad_loss[m] / (K_g * G_m) in group-mean mode (head_cnt then holds G_m).
__global__ void __launch_bounds__(kThreads)
k_seq_scale(float* __restrict__ coef, const int32_t* __restrict__ role,
            const int32_t* __restrict__ head_of_role, int n_role, int M, int64_t T,
            const float* __restrict__ grad_loss, const int64_t* __restrict__ head_cnt,
            const int32_t* __restrict__ resp, int64_t n_resp, const int32_t* __restrict__ group_of_resp,
            const int32_t* __restrict__ group_cnt, int n_groups) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < T; j += stride) {
    int head = 0;
    if (M > 1) {
      const int r = role[j];
      head = (unsigned)r < (unsigned)n_role ? head_of_role[r] : -1;
    }
    float s = 0.f;
    if ((unsigned)head < (unsigned)M && head_cnt[head] > 0)
      s = (grad_loss ? grad_loss[head] : 1.f) / (float)head_cnt[head];
    if (group_cnt != nullptr) {
      const int rs = resp[j];
      const int g = (unsigned)rs < (unsigned)n_resp ? group_of_resp[rs] : -1;
      const int K = (unsigned)g < (unsigned)n_groups ? group_cnt[g] : 0;
      s = K > 0 ? s / (float)K : 0.f;
    }
    coef[j] *= s;
  }
}

__global__ void __launch_bounds__(kThreads)
k_coef(const float* logp, const float* old_logp, const int32_t* resp, const float* adv,
       int64_t n_resp, const int32_t* role, const int32_t* head_of_role, int n_role, int M,
       int64_t T, float lo, float hi, const float* grad_loss, const Schedule* sched, float* coef,
       int32_t* status) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < T; j += stride) {
    int head = 0;
    if (M > 1) {
      const int r = role[j];
      head = (unsigned)r < (unsigned)n_role ? head_of_role[r] : -1;
      if ((unsigned)head >= (unsigned)M) {
        coef[j] = 0.f;
        continue;
      }
    }
    const int rs = resp[j];
    float A = 0.f;
    if ((unsigned)rs < (unsigned)n_resp) A = adv[rs];
    else raise_status(status, ATGRPO_ERR_BAD_INDEX);
    float rho;
    bool active;
    (void)clipped_term(logp[j], old_logp[j], A, lo, hi, rho, active);
    const float gm = grad_loss ? grad_loss[head] : 1.f;
    const int Tm = sched->rows[head];
    coef[j] = (active && Tm > 0) ? gm * A * rho / (float)Tm : 0.f;
  }
}

int loss_grid(int64_t T) {
  int64_t g = (T + kThreads * 4 - 1) / (kThreads * 4);
  if (g < 1) g = 1;
  if (g > kMaxBlocks) g = kMaxBlocks;
  return (int)g;
}

// ------------------------------------------------------------------------------- routing
constexpr int kRouteThreads = 1024;

// Head of token j, or -1 if it is routed nowhere.  `keep` (optional) drops tokens whose entry is
// zero: the backward pass routes only the tokens that carry a gradient.
__device__ __forceinline__ int head_of_token(const int32_t* role, const int32_t* head_of_role,
                                             int n_role, int M, int64_t j, const float* keep,
                                             int32_t* status) {
  if (keep != nullptr && keep[j] == 0.f) return -1;
  if (role == nullptr) return 0;                       // single policy
  const int r = role[j];
  const int h = (unsigned)r < (unsigned)n_role ? head_of_role[r] : -1;
  if ((unsigned)h >= (unsigned)M) {
    raise_status(status, ATGRPO_ERR_BAD_INDEX);
    return -1;
  }
  return h;
}

__global__ void __launch_bounds__(kRouteThreads)
k_route_hist(const int32_t* role, const int32_t* head_of_role, int n_role, int M, int64_t T,
             int nb, const float* keep, int32_t* blk_cnt, int32_t* status) {
  __shared__ int s_cnt[ATGRPO_MAX_HEADS];
  if (threadIdx.x < ATGRPO_MAX_HEADS) s_cnt[threadIdx.x] = 0;
  __syncthreads();
  const int64_t j = (int64_t)blockIdx.x * kRouteThreads + threadIdx.x;
  const int h = j < T ? head_of_token(role, head_of_role, n_role, M, j, keep, status) : -1;
  for (int m = 0; m < M; ++m) {
    const unsigned b = __ballot_sync(0xffffffffu, h == m);
    if ((threadIdx.x & 31) == 0 && b) atomicAdd(&s_cnt[m], __popc(b));   // integer: order-free
  }
  __syncthreads();
  if ((int)threadIdx.x < M) blk_cnt[threadIdx.x * nb + blockIdx.x] = s_cnt[threadIdx.x];
}

__global__ void __launch_bounds__(kRouteThreads)
k_route_scan(int M, int nb, const int32_t* blk_cnt, int32_t* blk_off, Schedule* sched,
             int32_t* role_offsets_out) {
  __shared__ int warp_tot[kRouteThreads / 32];
  __shared__ int s_carry;
  __shared__ int s_head_begin[ATGRPO_MAX_HEADS + 1];
  if (threadIdx.x == 0) s_carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int total = M * nb;                   // head-major: all blocks of head 0, then head 1 ...
  for (int base = 0; base < total; base += kRouteThreads) {
    const int i = base + threadIdx.x;
    const int c = i < total ? blk_cnt[i] : 0;
    int v = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    if (lane == 31) warp_tot[w] = v;
    __syncthreads();
    int add = s_carry;
    for (int k = 0; k < w; ++k) add += warp_tot[k];
    const int excl = add + v - c;
    if (i < total) {
      blk_off[i] = excl;
      if (i % nb == 0) s_head_begin[i / nb] = excl;
    }
    __syncthreads();
    if (threadIdx.x == kRouteThreads - 1) s_carry = add + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    s_head_begin[M] = s_carry;
    sched->n_heads = M;
    int tile = 0;
    for (int m = 0; m < M; ++m) {
      const int rows = s_head_begin[m + 1] - s_head_begin[m];
      sched->tile_begin[m] = tile;
      sched->rows[m] = rows;
      sched->role_offsets[m] = s_head_begin[m];
      if (role_offsets_out) role_offsets_out[m] = s_head_begin[m];
      tile += ((rows + 127) / 128 + 1) & ~1;      // whole 256-row pair tiles per head
    }
    sched->tile_begin[M] = tile;
    sched->role_offsets[M] = s_head_begin[M];
    if (role_offsets_out) role_offsets_out[M] = s_head_begin[M];
    for (int m = M + 1; m <= ATGRPO_MAX_HEADS; ++m) sched->tile_begin[m] = tile;
  }
}

__global__ void __launch_bounds__(kRouteThreads)
k_route_scatter(const int32_t* role, const int32_t* head_of_role, int n_role, int M, int64_t T,
                int nb, const float* keep, const int32_t* blk_off, const Schedule* sched, int32_t* row_of_token,
                int32_t* tok_of_row, int32_t* role_perm) {
  __shared__ int s_warp[ATGRPO_MAX_HEADS][kRouteThreads / 32];
  const int64_t j = (int64_t)blockIdx.x * kRouteThreads + threadIdx.x;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int h = j < T ? head_of_token(role, head_of_role, n_role, M, j, keep, nullptr) : -1;
  int rank_in_warp = 0;
  for (int m = 0; m < M; ++m) {
    const unsigned b = __ballot_sync(0xffffffffu, h == m);
    if (h == m) rank_in_warp = __popc(b & ((1u << lane) - 1u));
    if (lane == 0) s_warp[m][w] = __popc(b);
  }
  __syncthreads();
  if (h >= 0) {
    int before = 0;
    for (int k = 0; k < w; ++k) before += s_warp[h][k];
    const int pos = blk_off[h * nb + blockIdx.x] + before + rank_in_warp;   // stable position
    const int row = sched->tile_begin[h] * 128 + (pos - sched->role_offsets[h]);
    if (role_perm) role_perm[pos] = (int)j;
    row_of_token[j] = row;
    tok_of_row[row] = (int)j;
  } else if (j < T) {
    row_of_token[j] = -1;
  }
}

__global__ void k_route_single(int64_t T, int64_t T_pad, Schedule* sched, int32_t* tok_of_row,
                               int32_t* row_of_token, int32_t* role_offsets_out,
                               int32_t* role_perm) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < T_pad; p += stride) {
    tok_of_row[p] = p < T ? (int)p : -1;
    if (p < T) {
      row_of_token[p] = (int)p;
      if (role_perm) role_perm[p] = (int)p;
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    sched->n_heads = 1;
    sched->tile_begin[0] = 0;
    for (int m = 1; m <= ATGRPO_MAX_HEADS; ++m) sched->tile_begin[m] = (int)((T + 255) / 256) * 2;
    sched->rows[0] = (int)T;
    sched->role_offsets[0] = 0;
    sched->role_offsets[1] = (int)T;
    if (role_offsets_out) role_offsets_out[0] = 0, role_offsets_out[1] = (int)T;
  }
}

__global__ void __launch_bounds__(256)
k_gather_rows(const uint4* __restrict__ H, int64_t ldH16, const int32_t* __restrict__ tok_of_row,
              int64_t T_pad, int d16, uint4* __restrict__ Hs) {
  const int64_t total = T_pad * d16;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t row = i / d16;
    const int c = (int)(i - row * d16);
    const int tok = tok_of_row[row];
    Hs[i] = tok >= 0 ? H[(int64_t)tok * ldH16 + c] : make_uint4(0, 0, 0, 0);
  }
}

}  // namespace

size_t loss_reduce_workspace_bytes(int64_t T) {
  Carver c(nullptr);
  const int g = loss_grid(T < 0 ? 0 : T);
  c.take<double>((size_t)g * ATGRPO_MAX_HEADS);
  c.take<int64_t>((size_t)g * ATGRPO_MAX_HEADS * 3);
  c.take<unsigned>(1);
  c.take<int64_t>(ATGRPO_MAX_HEADS);                 // sequence mode: responses per head
  c.take<float>((size_t)(T < 0 ? 0 : T) + 1);        // sequence mode: per-response term
  c.take<int32_t>((size_t)(T < 0 ? 0 : T) + 1);      // sequence mode: per-response clip flags
  return c.off;
}

int loss_reduce_launch(const float* logp, const float* old_logp, const int32_t* resp_of_token,
                       const float* adv, int64_t n_resp, const int32_t* role_of_token,
                       const int32_t* head_of_role, int32_t n_role, int32_t M, int64_t T,
                       const atgrpo_params& prm, const float* grad_loss, float* loss, float* coef,
                       int64_t* clip_counts, int32_t* device_status, void* workspace, cudaStream_t st) {
  Carver c(workspace);
  const int g = loss_grid(T);
  LossArgs a;
  a.logp = logp, a.old_logp = old_logp, a.resp = resp_of_token, a.adv = adv, a.n_resp = n_resp;
  a.role = role_of_token, a.head_of_role = head_of_role, a.n_role = n_role, a.M = M, a.T = T;
  a.lo = 1.f - prm.clip_eps_low, a.hi = 1.f + prm.clip_eps_high;
  a.loss = loss, a.coef = coef, a.clip_counts = clip_counts, a.status = device_status;
  a.part_sum = c.take<double>((size_t)g * ATGRPO_MAX_HEADS);
  a.part_cnt = c.take<int64_t>((size_t)g * ATGRPO_MAX_HEADS * 3);
  a.done = c.take<unsigned>(1);
  int64_t* head_cnt = c.take<int64_t>(ATGRPO_MAX_HEADS);
  float* seg_term = c.take<float>((size_t)T + 1);
  int32_t* seg_flags = c.take<int32_t>((size_t)T + 1);
  a.head_cnt = nullptr, a.seg_term = nullptr, a.seg_flags = nullptr;
  a.group_of_resp = nullptr, a.group_cnt = nullptr;
  auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
  a.vec = al16(logp) && al16(old_logp) && al16(resp_of_token);
  ATGRPO_CUDA_OK(cudaMemsetAsync(a.done, 0, sizeof(unsigned), st));
  if (prm.reduction != ATGRPO_REDUCE_TOKEN_MEAN) {
    // per-response ratios, then the mean over responses (or over groups of the per-group mean);
    // coef (if asked for) is scaled afterwards
    const bool by_group = prm.reduction == ATGRPO_REDUCE_GROUP_MEAN;
    int32_t* group_cnt = by_group ? prm.group_scratch : nullptr;
    if (by_group) ATGRPO_CUDA_OK(cudaMemsetAsync(group_cnt, 0, (size_t)prm.n_groups * sizeof(int32_t), st));
    int64_t rg = (n_resp + kThreads / 32 - 1) / (kThreads / 32);
    if (rg > kMaxBlocks) rg = kMaxBlocks;
    if (rg < 1) rg = 1;
    k_seq_resp<<<(int)rg, kThreads, 0, st>>>(logp, old_logp, resp_of_token, adv, n_resp, T, a.lo, a.hi,
                                             seg_term, seg_flags, coef, prm.group_of_resp, group_cnt,
                                             prm.n_groups, device_status);
    a.head_cnt = head_cnt, a.seg_term = seg_term, a.seg_flags = seg_flags;
    if (by_group) a.group_of_resp = prm.group_of_resp, a.group_cnt = group_cnt;
    a.coef = nullptr;
    if (M == 1) k_seq_reduce<1><<<g, kThreads, 0, st>>>(a);
    else k_seq_reduce<0><<<g, kThreads, 0, st>>>(a);
    if (coef)
      k_seq_scale<<<g, kThreads, 0, st>>>(coef, role_of_token, head_of_role, n_role, M, T, grad_loss, head_cnt,
                                          resp_of_token, n_resp, prm.group_of_resp, group_cnt, prm.n_groups);
    return launch_ok();
  }
  // one resident wave: the grid-stride loop then keeps every thread's next loads in flight
  // (a second wave of blocks would start cold behind the first)
  int n_sm = 148, cc = 0, per_sm = 0, grid = g;
  if (device_sm_count(&n_sm, &cc) != ATGRPO_OK || n_sm <= 0) n_sm = 148;
  const cudaError_t oe = M == 1
      ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_clipped_loss<1>, kThreads, 0)
      : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_clipped_loss<0>, kThreads, 0);
  if (oe == cudaSuccess && per_sm > 0 && grid > per_sm * n_sm) grid = per_sm * n_sm;
  if (M == 1) k_clipped_loss<1><<<grid, kThreads, 0, st>>>(a);
  else k_clipped_loss<0><<<grid, kThreads, 0, st>>>(a);
  return launch_ok();
}

int coef_launch(const float* logp, const float* old_logp, const int32_t* resp_of_token,
                const float* adv, int64_t n_resp, const int32_t* role_of_token,
                const int32_t* head_of_role, int32_t n_role, int32_t M, int64_t T,
                const atgrpo_params& prm, const float* grad_loss, const Schedule* sched,
                float* coef, int32_t* device_status, cudaStream_t st) {
  k_coef<<<loss_grid(T), kThreads, 0, st>>>(logp, old_logp, resp_of_token, adv, n_resp,
                                            role_of_token, head_of_role, n_role, M, T,
                                            1.f - prm.clip_eps_low, 1.f + prm.clip_eps_high,
                                            grad_loss, sched, coef, device_status);
  return launch_ok();
}

size_t routing_workspace_bytes(int64_t T, int32_t M) {
  Carver c(nullptr);
  const size_t nb = (size_t)((T + kRouteThreads - 1) / kRouteThreads) + 1;
  c.take<int32_t>(nb * M);
  c.take<int32_t>(nb * M);
  return c.off;
}

int routing_launch(const int32_t* role_of_token, const int32_t* head_of_role, int32_t n_role,
                   int32_t M, int64_t T, int64_t T_pad, Schedule* sched, int32_t* row_of_token,
                   int32_t* tok_of_row, int32_t* role_offsets, int32_t* role_perm,
                   int32_t* device_status, void* workspace, cudaStream_t st, const float* keep) {
  if (M == 1 && keep == nullptr) {
    const int grid = (int)((T_pad + 255) / 256 > 0 ? (T_pad + 255) / 256 : 1);
    k_route_single<<<grid, 256, 0, st>>>(T, T_pad, sched, tok_of_row, row_of_token, role_offsets,
                                         role_perm);
    return launch_ok();
  }
  Carver c(workspace);
  const int nb = (int)((T + kRouteThreads - 1) / kRouteThreads);
  int32_t* blk_cnt = c.take<int32_t>((size_t)(nb + 1) * M);
  int32_t* blk_off = c.take<int32_t>((size_t)(nb + 1) * M);
  ATGRPO_CUDA_OK(cudaMemsetAsync(tok_of_row, 0xFF, (size_t)T_pad * sizeof(int32_t), st));
  if (nb > 0)
    k_route_hist<<<nb, kRouteThreads, 0, st>>>(M == 1 ? nullptr : role_of_token, head_of_role, n_role, M, T, nb,
                                               keep, blk_cnt, device_status);
  k_route_scan<<<1, kRouteThreads, 0, st>>>(M, nb, blk_cnt, blk_off, sched, role_offsets);
  if (nb > 0)
    k_route_scatter<<<nb, kRouteThreads, 0, st>>>(M == 1 ? nullptr : role_of_token, head_of_role, n_role, M, T, nb,
                                                  keep, blk_off, sched, row_of_token, tok_of_row,
                                                  role_perm);
  return launch_ok();
}

int gather_rows_launch(const void* H, int64_t ldH, const int32_t* tok_of_row, int64_t T_pad,
                       int32_t d, void* Hs, cudaStream_t st) {
  const int64_t total = T_pad * (d / 8);
  if (total == 0) return ATGRPO_OK;
  int64_t grid = (total + 255) / 256;
  if (grid > 148 * 16) grid = 148 * 16;
  k_gather_rows<<<(int)grid, 256, 0, st>>>(static_cast<const uint4*>(H), ldH / 8, tok_of_row,
                                           T_pad, d / 8, static_cast<uint4*>(Hs));
  return launch_ok();
}

}  // namespace atgrpo
