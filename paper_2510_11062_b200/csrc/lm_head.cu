// LM-head contractions of the policy loss (pi_theta of Eq. 2 and the gradient of Eq. 2) on the
// sm_100a tensor cores.  One warp-specialised persistent kernel template serves four modes:
//
//   kFwd : z = H W_m^T tile by tile, streaming logsumexp and target-logit gather in the epilogue;
//          the logits only ever exist in tensor memory.
//   kDz  : the same contraction for one vocabulary chunk; the epilogue turns the logits into
//          dZ = coef*(softmax - onehot) and writes them as bf16 into the chunk buffer.
//   kDh  : dH_rows += dZ_chunk * W_m[chunk, :]          (A K-major, B MN-major)
//   kDw  : dW_m[chunk, :] = dZ_chunk^T * H_rows          (A and B MN-major)
//
// The kernel runs on CTA pairs (clusters of two, cta_group::2): a pair owns a 256 x 256 output
// tile, each CTA stages its own 128 rows of A and half of B (32 KiB per k-step of 64) through TMA
// into a 6-deep ring of 128-byte-swizzled shared-memory tiles, the pair's leader issues
// tcgen05.mma (M = 256, N = 256, K = 16) over both CTAs' shared memory, and each CTA's 128
// accumulator rows live in its own tensor memory, double buffered in the 512 TMEM columns so the
// epilogue of tile i overlaps the MMAs of tile i+1.
// CTA layout (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer (leader only) and TMEM
// owner, warps 2-9 = epilogue (two warps per TMEM lane quarter, each taking half of the columns).
// Rows are addressed in the "padded row space": the tokens of policy m occupy whole 256-row pair
// tiles starting at tile_begin[m], so no tile mixes two heads (grouped GEMM).
#include <cuda_bf16.h>
#include <cstring>
#include "internal.h"
#include "sm100.cuh"

namespace atgrpo {
namespace {
using namespace sm100;

constexpr int BM = 128, BN = 256, BK = 64;          // BM rows per CTA: a CTA pair owns 2*BM = 256 rows
constexpr int kPairRows = 2 * BM;
constexpr int kStages = 6;
constexpr int kABytes = BM * BK * 2;               // 16 KiB: this CTA's 128 rows of A
constexpr int kBBytes = (BN / 2) * BK * 2;         // 16 KiB: this CTA's half of B
constexpr int kStageBytes = kABytes + kBBytes;     // 32 KiB per CTA and k-step
constexpr int kBoxBytes = 64 * 64 * 2;             // one 64 x 64 MN-major box, 8 KiB
constexpr int kGemmThreads = 320;               // producer warp, MMA warp, 8 epilogue warps
constexpr int kEpilogueThreads = 256;
constexpr int kTmemCols = 512;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

enum Mode { kFwd = 0, kDz = 1, kDh = 2, kDw = 3 };

struct Maps {
  CUtensorMap a;
  CUtensorMap b[ATGRPO_MAX_HEADS];
};

struct GemmArgs {
  const Schedule* sched;
  const int32_t* tok_of_row;
  const int32_t* target;
  int32_t* status;
  int V, d, M;
  int64_t T_pad;
  // kFwd / kDz: vocabulary tiling
  int v_begin;            // first vocabulary row of this launch (0 for kFwd)
  int n_vtiles;           // 256-wide vocabulary tiles in this launch
  int tiles_per_chunk;    // kFwd: tiles one work item sweeps (1 for kDz)
  int n_chunks;
  int m_block;            // kFwd / kDz: row tiles swept together so their rows of H stay in L2
  float* part_m;          // kFwd out: running max (log2 domain) [2*n_chunks, T_pad]
  float* part_s;          // kFwd out: sum of 2^(t - max)        [2*n_chunks, T_pad]
  float* zt;              // kFwd out: target logit              [T_pad]
  const float* lse;       // kDz in, token order
  const float* coef;      // kDz in, token order
  __nv_bfloat16* dz;      // kDz out / kDh, kDw in: [T_pad, vc]
  int vc;                 // chunk buffer width (multiple of 256)
  int vc_valid;           // vocabulary rows of this chunk that exist (<= vc)
  // kDh
  float* dh_acc;          // [T_pad, d] fp32
  int first_chunk;
  // kDw
  void* dW[ATGRPO_MAX_HEADS];
  int dw_bf16, dw_accumulate;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 256-bit global store (sm_100): p must be 32-byte aligned.
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v[0]), "r"(v[1]),
               "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}

__device__ __forceinline__ void ld_global_v8(const void* p, uint32_t* v) {
  asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "l"(p)
               : "memory");
}

struct Tile {
  int head;
  int row0;        // first padded row (kFwd/kDz/kDh) or first K row (kDw)
  int rows_valid;  // valid token rows of this tile (kFwd/kDz/kDh)
  int n0;          // first vocabulary row (kFwd/kDz, absolute) or first d column (kDh/kDw)
  int v0;          // kDw: first vocabulary row of the tile inside the chunk buffer
  int k_steps;
  int chunk;       // kFwd: work-item chunk index
  int nt_begin, nt_end;   // kFwd: tiles of the item
};

__device__ __forceinline__ int head_of_tile(const Schedule* s, int M, int mt) {
  int h = 0;
  for (int m = 1; m < M; ++m)
    if (mt >= s->tile_begin[m]) h = m;
  return h;
}

// Work items are tiles of a CTA pair: 256 rows x 256 columns.  `rank` selects this CTA's half.
template <int kMode>
__device__ __forceinline__ int total_items(const GemmArgs& g, const Schedule* sched) {
  const int n_pt = sched->tile_begin[g.M] / 2;          // heads start on even 128-row tiles
  const int n_dt = (g.d + BN - 1) / BN;
  if (kMode == kFwd || kMode == kDz) return n_pt * g.n_chunks;
  if (kMode == kDh) return n_pt * n_dt;
  return g.M * ((g.vc_valid + kPairRows - 1) / kPairRows) * n_dt;
}

template <int kMode>
__device__ __forceinline__ Tile decode_item(const GemmArgs& g, const Schedule* s, int it, int rank) {
  Tile t;
  const int n_dt = (g.d + BN - 1) / BN;
  t.v0 = 0, t.chunk = 0, t.nt_begin = 0, t.nt_end = 1;
  if (kMode == kFwd || kMode == kDz) {
    // Row tiles come in blocks of m_block pairs; inside a block the row tile runs fastest, then
    // the vocabulary chunk: co-resident pairs share W tiles, and a block's rows of H stay in L2.
    const int n_pt = s->tile_begin[g.M] / 2;
    const int per_block = g.m_block * g.n_chunks;
    const int blk = it / per_block, rem = it - blk * per_block;
    const int gm = min(g.m_block, n_pt - blk * g.m_block);
    const int c = rem / gm, pt = blk * g.m_block + (rem - c * gm);
    const int mt = 2 * pt + rank;
    t.head = head_of_tile(s, g.M, 2 * pt);
    t.row0 = mt * BM;
    t.rows_valid = min(BM, s->rows[t.head] - (mt - s->tile_begin[t.head]) * BM);
    t.chunk = c;
    t.nt_begin = c * g.tiles_per_chunk;
    t.nt_end = min(t.nt_begin + g.tiles_per_chunk, g.n_vtiles);
    t.n0 = g.v_begin + t.nt_begin * BN;
    t.k_steps = (g.d + BK - 1) / BK;
  } else if (kMode == kDh) {
    const int pt = it / n_dt, dt = it - pt * n_dt;     // d tiles fastest: they share the dZ tile
    const int mt = 2 * pt + rank;
    t.head = head_of_tile(s, g.M, 2 * pt);
    t.row0 = mt * BM;
    t.rows_valid = min(BM, s->rows[t.head] - (mt - s->tile_begin[t.head]) * BM);
    t.n0 = dt * BN;
    t.k_steps = (g.vc_valid + BK - 1) / BK;
  } else {
    const int n_vt = (g.vc_valid + kPairRows - 1) / kPairRows;
    const int dt = it % n_dt, rest = it / n_dt;
    const int vt = rest % n_vt;
    t.head = rest / n_vt;
    t.row0 = s->tile_begin[t.head] * BM;
    t.rows_valid = 0;
    t.n0 = dt * BN;
    t.v0 = vt * kPairRows + rank * BM;
    t.k_steps = (s->tile_begin[t.head + 1] - s->tile_begin[t.head]) * (BM / BK);
  }
  return t;
}

template <int kMode>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_lm_head(const __grid_constant__ Maps maps, const GemmArgs g) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  uint8_t* smem_aligned = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(
      smem_aligned + kStages * kStageBytes + 8 * (2 * kStages + 4));
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();           // 0 = leader of the pair (issues the MMAs)
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  // the tile schedule is read once per CTA: every role decodes its tiles from shared memory
  __shared__ Schedule s_sched;
  if (threadIdx.x >= 64 && threadIdx.x < 64 + sizeof(Schedule) / 4)
    reinterpret_cast<int32_t*>(&s_sched)[threadIdx.x - 64] =
        reinterpret_cast<const int32_t*>(g.sched)[threadIdx.x - 64];
  const Schedule* sched = &s_sched;

  // Barrier protocol of a pair.  full[s] lives in the leader: its producer announces the bytes of
  // both CTAs (2 x 32 KiB) and the TMA loads of both CTAs report there.  empty[s] and tfull[a] exist in both CTAs and are
  // signalled by the leader's multicast tcgen05.commit.  tempty[a] lives in the leader: the
  // epilogue threads of both CTAs arrive on it.
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 2 * kEpilogueThreads);
    }
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tmap(&maps.a);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(s_tmem)), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                 // peer barriers initialised, TMEM allocated
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int n_items = total_items<kMode>(g, sched);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t keep = l2_policy_evict_last();
      for (int it = pair; ok && it < n_items; it += n_pairs) {
        const Tile t = decode_item<kMode>(g, sched, it, rank);
        for (int nt = t.nt_begin; ok && nt < t.nt_end; ++nt) {
          const int n0 = t.n0 + (nt - t.nt_begin) * BN + rank * (BN / 2);   // this CTA's half of B
          for (int ks = 0; ks < t.k_steps; ++ks) {
            if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, s_abort, g.status))) break;
            const uint32_t sa = smem_base + stage * kStageBytes, sb = sa + kABytes;
            const uint32_t fb = mapa_shared(full_bar(stage), 0);             // the leader's barrier
            if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * kStageBytes);
            if (kMode == kFwd || kMode == kDz) {
              tma_load_2d_pair_hint(sa, &maps.a, ks * BK, t.row0, fb, keep);          // rows of H: re-read per W tile
              tma_load_2d_pair(sb, &maps.b[t.head], ks * BK, n0, fb);
            } else if (kMode == kDh) {
              tma_load_2d_pair(sa, &maps.a, ks * BK, t.row0, fb);                      // dZ: shared by the d tiles
#pragma unroll
              for (int b = 0; b < 2; ++b)                                             // W chunk: re-read per wave
                tma_load_2d_pair_hint(sb + b * kBoxBytes, &maps.b[t.head], n0 + 64 * b, g.v_begin + ks * BK, fb, keep);
            } else {
#pragma unroll
              for (int b = 0; b < 2; ++b)
                tma_load_2d_pair(sa + b * kBoxBytes, &maps.a, t.v0 + 64 * b, t.row0 + ks * BK, fb);
#pragma unroll
              for (int b = 0; b < 2; ++b)                                             // H: re-read per wave
                tma_load_2d_pair_hint(sb + b * kBoxBytes, &maps.b[0], n0 + 64 * b, t.row0 + ks * BK, fb, keep);
            }
            if (++stage == kStages) stage = 0, phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr bool a_mn = (kMode == kDw), b_mn = (kMode == kDh || kMode == kDw);
      constexpr uint32_t idesc = idesc_bf16(kPairRows, BN, a_mn, b_mn);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int it = pair; ok && it < n_items; it += n_pairs) {
        const Tile t = decode_item<kMode>(g, sched, it, rank);
        if (t.k_steps == 0) continue;
        for (int nt = t.nt_begin; ok && nt < t.nt_end; ++nt) {
          if (!(ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, s_abort, g.status))) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * BN;
          for (int ks = 0; ks < t.k_steps; ++ks) {
            if (!(ok = mbar_wait(full_bar(stage), phase, s_abort, g.status))) break;
            tc_fence_after();
            const uint32_t sa = smem_base + stage * kStageBytes, sb = sa + kABytes;
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
              const uint64_t ad = a_mn ? smem_desc(sa + kk * 2048, kBoxBytes, 1024)
                                       : smem_desc(sa + kk * 32, 16, 1024);
              const uint64_t bd = b_mn ? smem_desc(sb + kk * 2048, kBoxBytes, 1024)
                                       : smem_desc(sb + kk * 32, 16, 1024);
              umma_bf16_pair(d_tmem, ad, bd, idesc, (ks | kk) != 0 ? 1u : 0u);
            }
            umma_commit_pair(empty_bar(stage), 3);   // frees the stage in both CTAs
            if (++stage == kStages) stage = 0, phase ^= 1u;
          }
          if (!ok) break;
          umma_commit_pair(tfull_bar(acc), 3);        // accumulator complete in both CTAs
          if (++acc == 2) acc = 0, acc_phase ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    // Two warps per TMEM lane quarter (a warp can only read the quarter warp_id % 4): the first
    // four epilogue warps take columns 0-127 of the tile, the other four columns 128-255, so every
    // scheduler has two epilogue warps to hide each other's TMEM-load and MUFU latency.
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;
    const int c_begin = half * (BN / 64), c_end = c_begin + BN / 64;
    const int r_in_tile = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    const uint32_t tempty_leader0 = mapa_shared(tempty_bar(0), 0), tempty_leader1 = mapa_shared(tempty_bar(1), 0);
    for (int it = pair; ok && it < n_items; it += n_pairs) {
      const Tile t = decode_item<kMode>(g, sched, it, rank);
      uint32_t r[32];

      if (kMode == kFwd || kMode == kDz) {
        const int row = t.row0 + r_in_tile;
        const bool valid = r_in_tile < t.rows_valid;
        const int tok = valid ? g.tok_of_row[row] : -1;
        int y = -1;
        if (tok >= 0) {
          y = g.target[tok];
          if ((unsigned)y >= (unsigned)g.V) {
            raise_status(g.status, ATGRPO_ERR_BAD_INDEX);
            y = 0;
          }
        }
        float m2 = -INFINITY, ssum = 0.f, zt = 0.f;
        bool have_zt = false;
        float lse2 = 0.f, cf = 0.f;
        if (kMode == kDz && tok >= 0) lse2 = g.lse[tok] * kLog2e, cf = g.coef[tok];
        for (int nt = t.nt_begin; ok && nt < t.nt_end; ++nt) {
          const int n0 = t.n0 + (nt - t.nt_begin) * BN;
          if (!(ok = mbar_wait_backoff(tfull_bar(acc), acc_phase, s_abort, g.status))) break;
          tc_fence_after();
          for (int c = c_begin; c < c_end; ++c) {
            const int col0 = n0 + c * 32;
            if (kMode == kFwd && col0 >= g.V) break;
            __syncwarp();
            tmem_ld32(lane_addr + acc * BN + c * 32, r);
            tmem_ld_wait();
            if (kMode == kFwd) {
              if (y >= col0 && y < col0 + 32) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (col0 + i == y) zt = __uint_as_float(r[i]);
                have_zt = true;
              }
              // running (max, sum) in the log2 domain: max on the raw logits (log2 e > 0), then
              // one FFMA + ex2 + add per element
              const bool ragged = col0 + 32 > g.V;
              float cmax = -INFINITY;
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                if (ragged && col0 + i >= g.V) r[i] = 0xff800000u;     // -inf
                cmax = fmaxf(cmax, __uint_as_float(r[i]));
              }
              const float nm = fmaxf(m2, cmax * kLog2e);
              float add0 = 0.f, add1 = 0.f;
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                add0 += ex2(fmaf(__uint_as_float(r[i]), kLog2e, -nm));
                add1 += ex2(fmaf(__uint_as_float(r[i + 1]), kLog2e, -nm));
              }
              ssum = fmaf(ssum, ex2(m2 - nm), add0 + add1);
              m2 = nm;
            } else {
              // dZ = coef * softmax, minus coef at the target column; zero beyond the vocabulary
              float gz[32];
#pragma unroll
              for (int i = 0; i < 32; ++i)
                gz[i] = cf * ex2(fmaf(__uint_as_float(r[i]), kLog2e, -lse2));
              if (y >= col0 && y < col0 + 32) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (col0 + i == y) gz[i] -= cf;
              }
              if (col0 + 32 > g.V) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (col0 + i >= g.V) gz[i] = 0.f;
              }
              uint32_t packed[16];
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(gz[i], gz[i + 1]);
                packed[i >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
              }
              // 32-byte stores: one full sector per lane and half as many L1 wavefronts as 16-byte ones
              __nv_bfloat16* dst = g.dz + (size_t)row * g.vc + (col0 - g.v_begin);
              st_global_v8(dst, packed);
              st_global_v8(dst + 16, packed + 8);
            }
          }
          tc_fence_before();
          mbar_arrive_cluster(acc ? tempty_leader1 : tempty_leader0);
          if (++acc == 2) acc = 0, acc_phase ^= 1u;
        }
        if (kMode == kFwd && ok && tok >= 0) {
          g.part_m[(size_t)(2 * t.chunk + half) * g.T_pad + row] = m2;
          g.part_s[(size_t)(2 * t.chunk + half) * g.T_pad + row] = ssum;
          if (have_zt) g.zt[row] = zt;
        }
      } else {
        // kDh / kDw: plain accumulator write-out
        const bool has_acc = t.k_steps > 0;
        if (has_acc) {
          if (!(ok = mbar_wait_backoff(tfull_bar(acc), acc_phase, s_abort, g.status))) break;
          tc_fence_after();
        }
        bool valid;
        size_t out_row;
        if (kMode == kDh) {
          valid = r_in_tile < t.rows_valid;
          out_row = (size_t)(t.row0 + r_in_tile);
        } else {
          const int v = g.v_begin + t.v0 + r_in_tile;
          valid = (t.v0 + r_in_tile < g.vc_valid) && v < g.V;
          out_row = (size_t)v;
        }
        for (int c = c_begin; c < c_end; ++c) {
          const int col0 = t.n0 + c * 32;
          if (col0 >= g.d) break;
          if (has_acc) {
            __syncwarp();
            tmem_ld32(lane_addr + acc * BN + c * 32, r);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = 0u;
          }
          if (!valid) continue;
          if (kMode == kDh || !g.dw_bf16) {
            float* dst = (kMode == kDh ? g.dh_acc : static_cast<float*>(g.dW[t.head])) +
                         out_row * g.d + col0;
            const bool add = kMode == kDh ? !g.first_chunk : (g.dw_accumulate != 0);
            // 32 bytes per lane and instruction (d is a multiple of 8, rows are 32-byte aligned)
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              if (col0 + 8 * q8 < g.d) {
                uint32_t v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = r[8 * q8 + i];
                if (add) {
                  uint32_t o[8];
                  ld_global_v8(dst + 8 * q8, o);
#pragma unroll
                  for (int i = 0; i < 8; ++i)
                    v[i] = __float_as_uint(__uint_as_float(v[i]) + __uint_as_float(o[i]));
                }
                st_global_v8(dst + 8 * q8, v);
              }
            }
          } else {
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(g.dW[t.head]) + out_row * g.d + col0;
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              if (col0 + 8 * q8 < g.d) {
                uint4* p4 = reinterpret_cast<uint4*>(dst) + q8;
                float f[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(r[8 * q8 + i]);
                if (g.dw_accumulate) {
                  const uint4 o = *p4;
                  const __nv_bfloat162* oh = reinterpret_cast<const __nv_bfloat162*>(&o);
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const float2 of = __bfloat1622float2(oh[i]);
                    f[2 * i] += of.x, f[2 * i + 1] += of.y;
                  }
                }
                uint4 w;
                __nv_bfloat162* wh = reinterpret_cast<__nv_bfloat162*>(&w);
#pragma unroll
                for (int i = 0; i < 4; ++i) wh[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
                *p4 = w;
              }
            }
          }
        }
        if (has_acc) {
          tc_fence_before();
          mbar_arrive_cluster(acc ? tempty_leader1 : tempty_leader0);
          if (++acc == 2) acc = 0, acc_phase ^= 1u;
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  // Neither CTA may leave while its peer can still signal its barriers or read its shared memory.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    if (*s_abort) {
      // a wait gave up: let the loads this CTA may still have in flight land before its shared
      // memory is handed to the next CTA
      for (int i = 0; i < 64; ++i) __nanosleep(2000);
    }
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// Combines the per-item (max, sum) pairs into lse and logp, in token order.  Block = 32 rows x 8
// part groups: consecutive threads read consecutive rows of one part (coalesced), each thread
// merges every eighth part online, and thread group 0 merges the eight results in a fixed order.
__global__ void __launch_bounds__(256)
k_lse_combine(const Schedule* sched, int M, const int32_t* tok_of_row, int64_t T_pad, int n_parts,
              const float* __restrict__ part_m, const float* __restrict__ part_s,
              const float* __restrict__ zt, float* lse, float* logp) {
  __shared__ float s_m[8][32], s_s[8][32];
  const int64_t rows = (int64_t)sched->tile_begin[M] * BM;
  const int64_t p = (int64_t)blockIdx.x * 32 + threadIdx.x;
  const int grp = threadIdx.y;
  float mx = -INFINITY, s = 0.f;
  if (p < rows) {
    for (int c = grp; c < n_parts; c += 8) {
      const float ps = part_s[(size_t)c * T_pad + p];
      if (ps > 0.f) {                                   // a part without valid columns holds (-inf, 0)
        const float pm = part_m[(size_t)c * T_pad + p];
        const float nm = fmaxf(mx, pm);
        s = s * exp2f(mx - nm) + ps * exp2f(pm - nm);
        mx = nm;
      }
    }
  }
  s_m[grp][threadIdx.x] = mx, s_s[grp][threadIdx.x] = s;
  __syncthreads();
  if (grp != 0 || p >= rows) return;
  const int tok = tok_of_row[p];
  if (tok < 0) return;
  for (int g2 = 1; g2 < 8; ++g2) {
    const float ps = s_s[g2][threadIdx.x];
    if (ps > 0.f) {
      const float pm = s_m[g2][threadIdx.x];
      const float nm = fmaxf(mx, pm);
      s = s * exp2f(mx - nm) + ps * exp2f(pm - nm);
      mx = nm;
    }
  }
  const float l = (mx + log2f(s)) * kLn2;
  lse[tok] = l;
  logp[tok] = zt[p] - l;
}

template <bool kBf16>
__global__ void __launch_bounds__(256)
k_dh_finalize(const float* __restrict__ acc, const int32_t* __restrict__ row_of_token, int64_t T,
              int d, void* __restrict__ out) {
  const int d4 = d / 4;
  const int64_t total = T * d4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t tok = i / d4;
    const int c = (int)(i - tok * d4);
    const int row = row_of_token[tok];
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row >= 0) v = reinterpret_cast<const float4*>(acc + (size_t)row * d)[c];
    if (kBf16) {
      uint2 w;
      __nv_bfloat162* wh = reinterpret_cast<__nv_bfloat162*>(&w);
      wh[0] = __floats2bfloat162_rn(v.x, v.y);
      wh[1] = __floats2bfloat162_rn(v.z, v.w);
      reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + (size_t)tok * d)[c] = w;
    } else {
      reinterpret_cast<float4*>(static_cast<float*>(out) + (size_t)tok * d)[c] = v;
    }
  }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 matrix [outer, inner] with row stride ld elements; 128-byte swizzled boxes.
bool make_map(CUtensorMap* m, const void* base, int64_t inner, int64_t outer, int64_t ld,
              int box_inner, int box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)(outer > 0 ? outer : 1)};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Number of vocabulary chunks of the forward sweep.  Items are kept short (at most kMaxSweep
// tiles): the pairs that share a W tile then stay within a tile or two of each other, so the tile
// is still in L2 when the last of them reads it (with long items they drift apart and every pair
// ends up fetching W from HBM on its own).  Among the short sweeps, the one that fills the pairs
// most evenly wins.
constexpr int kMaxSweep = 4;
int fwd_chunks(int64_t n_pt, int n_vt, int n_pairs) {
  int best = n_vt;
  double best_eff = -1.0;
  for (int per = 1; per <= kMaxSweep && per <= n_vt; ++per) {
    const int c = (n_vt + per - 1) / per;
    const int64_t waves = (n_pt * c + n_pairs - 1) / n_pairs;
    const double eff = (double)(n_pt * (int64_t)n_vt) / ((double)waves * n_pairs * per);
    if (eff >= best_eff - 1e-9) best_eff = eff, best = c;       // ties: the longer sweep
  }
  return best;
}

// Pair tiles (256 rows) per block of the logits sweeps: as many as keep the block's rows of H
// within a quarter of the 126 MB L2 (the L2 is split over two dies, and rows read from both
// sides occupy space in each half).
int row_block_tiles(int64_t n_pt, int d) {
  int64_t gm = (32ll << 20) / ((int64_t)kPairRows * d * 2);
  if (gm < 1) gm = 1;
  if (gm > n_pt) gm = n_pt > 0 ? n_pt : 1;
  return (int)gm;
}

// Width of the dZ chunk buffer (a multiple of 256 columns, buffer <= 512 MiB): the width that
// minimises the modelled time of the three GEMM launches per chunk, counted in k-steps of one
// 256x256x64 pair tile per wave of CTA pairs plus a fixed cost per launch.  Wave quantisation of the dW GEMM
// (few, long tiles) is what this mostly avoids.
int bwd_chunk_width(int64_t T_pad, int d, int V, int M, int n_sm) {
  const int64_t budget = 512ll << 20;
  if (T_pad < kPairRows) T_pad = kPairRows;            // T = 0: keep the arithmetic below defined
  const int64_t vmax = (int64_t)(V + BN - 1) / BN * BN;
  int64_t cap = budget / (T_pad * 2) / BN * BN;
  if (cap < BN) cap = BN;
  if (cap > vmax) cap = vmax;
  const int64_t n_pt = T_pad / kPairRows, n_dt = (d + BN - 1) / BN, ksd = (d + BK - 1) / BK;
  const int64_t n_pairs = n_sm / 2 > 0 ? n_sm / 2 : 1;
  auto waves = [&](int64_t tiles) { return (tiles + n_pairs - 1) / n_pairs; };
  auto chunk_cost = [&](int64_t w) {
    const int64_t z = waves(n_pt * ((w + BN - 1) / BN)) * ksd;
    const int64_t h = waves(n_pt * n_dt) * ((w + BK - 1) / BK);
    const int64_t dw = waves((int64_t)M * ((w + kPairRows - 1) / kPairRows) * n_dt) * ((4 * n_pt + M - 1) / M);
    return z + h + dw + 3 * 24;
  };
  int64_t best = cap, best_cost = -1;
  for (int64_t vc = BN; vc <= cap; vc += BN) {
    const int64_t full = V / vc, tail = V - full * vc;
    const int64_t cost = full * chunk_cost(vc) + (tail > 0 ? chunk_cost(tail) : 0);
    if (best_cost < 0 || cost <= best_cost) best_cost = cost, best = vc;
  }
  return (int)best;
}

struct FwdPlan { size_t part_m, part_s, zt, total; int n_chunks, tiles_per_chunk, n_vt; };
FwdPlan fwd_plan(int64_t T_pad, int V, int n_sm) {
  FwdPlan p;
  p.n_vt = (V + BN - 1) / BN;
  const int64_t n_pt = T_pad / kPairRows;
  p.n_chunks = fwd_chunks(n_pt > 0 ? n_pt : 1, p.n_vt, n_sm / 2 > 0 ? n_sm / 2 : 1);
  p.tiles_per_chunk = (p.n_vt + p.n_chunks - 1) / p.n_chunks;
  Carver c(nullptr);
  p.part_m = c.off; c.take<float>((size_t)2 * p.n_chunks * T_pad);
  p.part_s = c.off; c.take<float>((size_t)2 * p.n_chunks * T_pad);
  p.zt = c.off; c.take<float>((size_t)T_pad);
  p.total = c.off;
  return p;
}

struct BwdPlan { size_t dz, dh_acc, total; int vc; };
BwdPlan bwd_plan(int64_t T_pad, int d, int V, int M, int n_sm, bool dH_direct) {
  BwdPlan p;
  p.vc = bwd_chunk_width(T_pad, d, V, M, n_sm);
  Carver c(nullptr);
  p.dz = c.off; c.take<__nv_bfloat16>((size_t)T_pad * p.vc);
  p.dh_acc = c.off;
  if (!dH_direct) c.take<float>((size_t)T_pad * d);
  p.total = c.off;
  return p;
}

// Launches `pairs` clusters of two CTAs (never more than can be resident at once).
template <int kMode>
int launch_gemm(const Maps& maps, const GemmArgs& g, int64_t items, int n_sm, cudaStream_t st) {
  if (cudaFuncSetAttribute(k_lm_head<kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSmemBytes) != cudaSuccess)
    return ATGRPO_ERR_CUDA;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2, attr[0].val.clusterDim.y = 1, attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int pairs = n_sm / 2;
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  int resident = 0;
  if (cudaOccupancyMaxActiveClusters(&resident, k_lm_head<kMode>, &cfg) == cudaSuccess && resident > 0 &&
      resident < pairs)
    pairs = resident;
  if (items < pairs) pairs = (int)(items > 0 ? items : 1);
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  if (cudaLaunchKernelEx(&cfg, k_lm_head<kMode>, maps, g) != cudaSuccess) return ATGRPO_ERR_CUDA;
  return launch_ok();
}

GemmArgs base_args(const LmHeadProblem& p) {
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.sched = p.sched, g.tok_of_row = p.tok_of_row, g.target = p.target, g.status = p.device_status;
  g.V = p.V, g.d = p.d, g.M = p.M, g.T_pad = p.T_pad;
  return g;
}

}  // namespace

int device_sm_count(int* n_sm, int* cc_major) {
  int dev = 0;
  ATGRPO_CUDA_OK(cudaGetDevice(&dev));
  ATGRPO_CUDA_OK(cudaDeviceGetAttribute(n_sm, cudaDevAttrMultiProcessorCount, dev));
  ATGRPO_CUDA_OK(cudaDeviceGetAttribute(cc_major, cudaDevAttrComputeCapabilityMajor, dev));
  return ATGRPO_OK;
}

int lm_head_bwd_chunks(int64_t T_pad, int32_t d, int32_t V, int32_t M, int32_t n_sm) {
  const int vc = bwd_chunk_width(T_pad, d, V, M, n_sm);
  return (V + vc - 1) / vc;
}

size_t lm_head_fwd_workspace_bytes(int64_t T_pad, int32_t d, int32_t V, int32_t n_sm) {
  (void)d;
  return fwd_plan(T_pad, V, n_sm).total;
}

int lm_head_fwd_launch(const LmHeadProblem& p, float* lse, float* logp, void* workspace,
                       cudaStream_t st) {
  const FwdPlan pl = fwd_plan(p.T_pad, p.V, p.n_sm);
  char* ws = static_cast<char*>(workspace);
  Maps maps;
  if (!make_map(&maps.a, p.A_rows, p.d, p.rows_bound, p.ldA, BK, BM)) return ATGRPO_ERR_CUDA;
  for (int m = 0; m < p.M; ++m)
    if (!make_map(&maps.b[m], p.W[m], p.d, p.V, p.d, BK, BN / 2)) return ATGRPO_ERR_CUDA;
  GemmArgs g = base_args(p);
  g.v_begin = 0, g.n_vtiles = pl.n_vt, g.tiles_per_chunk = pl.tiles_per_chunk, g.n_chunks = pl.n_chunks;
  g.m_block = row_block_tiles(p.T_pad / kPairRows, p.d);
  g.part_m = reinterpret_cast<float*>(ws + pl.part_m);
  g.part_s = reinterpret_cast<float*>(ws + pl.part_s);
  g.zt = reinterpret_cast<float*>(ws + pl.zt);
  int rc = launch_gemm<kFwd>(maps, g, (p.T_pad / kPairRows) * pl.n_chunks, p.n_sm, st);
  if (rc != ATGRPO_OK) return rc;
  const int cgrid = (int)((p.T_pad + 31) / 32 > 0 ? (p.T_pad + 31) / 32 : 1);
  k_lse_combine<<<cgrid, dim3(32, 8), 0, st>>>(p.sched, p.M, p.tok_of_row, p.T_pad, 2 * pl.n_chunks, g.part_m,
                                               g.part_s, g.zt, lse, logp);
  return launch_ok();
}

size_t lm_head_bwd_workspace_bytes(int64_t T_pad, int32_t d, int32_t V, int32_t M, int32_t n_sm,
                                   bool dH_direct) {
  return bwd_plan(T_pad, d, V, M, n_sm, dH_direct).total;
}

int lm_head_bwd_launch(const LmHeadProblem& p, const float* lse, const float* coef,
                       const int32_t* row_of_token, const atgrpo_params& prm, void* dH,
                       void* const* dW, void* workspace, cudaStream_t st) {
  const bool dH_direct = false;   // rows are compacted: dH always goes through the accumulator
  const BwdPlan pl = bwd_plan(p.T_pad, p.d, p.V, p.M, p.n_sm, dH_direct);
  char* ws = static_cast<char*>(workspace);
  __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(ws + pl.dz);
  float* dh_acc = dH_direct ? static_cast<float*>(dH) : reinterpret_cast<float*>(ws + pl.dh_acc);

  Maps m_dz, m_dh, m_dw;
  if (!make_map(&m_dz.a, p.A_rows, p.d, p.rows_bound, p.ldA, BK, BM)) return ATGRPO_ERR_CUDA;
  if (!make_map(&m_dh.a, dz, pl.vc, p.T_pad, pl.vc, BK, BM)) return ATGRPO_ERR_CUDA;
  if (!make_map(&m_dw.a, dz, pl.vc, p.T_pad, pl.vc, 64, 64)) return ATGRPO_ERR_CUDA;
  if (!make_map(&m_dw.b[0], p.A_rows, p.d, p.rows_bound, p.ldA, 64, 64)) return ATGRPO_ERR_CUDA;
  for (int m = 0; m < p.M; ++m) {
    if (!make_map(&m_dz.b[m], p.W[m], p.d, p.V, p.d, BK, BN / 2)) return ATGRPO_ERR_CUDA;
    if (!make_map(&m_dh.b[m], p.W[m], p.d, p.V, p.d, 64, 64)) return ATGRPO_ERR_CUDA;
  }
  const int64_t n_pt = p.T_pad / kPairRows;
  const int n_dt = (p.d + BN - 1) / BN;
  int chunk = 0;
  for (int v_begin = 0; v_begin < p.V; v_begin += pl.vc, ++chunk) {
    GemmArgs g = base_args(p);
    g.v_begin = v_begin;
    g.vc = pl.vc;
    g.vc_valid = p.V - v_begin < pl.vc ? p.V - v_begin : pl.vc;
    g.n_vtiles = (g.vc_valid + BN - 1) / BN;
    g.tiles_per_chunk = 1;
    g.m_block = row_block_tiles(n_pt, p.d);
    g.n_chunks = g.n_vtiles;
    g.lse = lse, g.coef = coef, g.dz = dz;
    g.dh_acc = dh_acc, g.first_chunk = chunk == 0;
    for (int m = 0; m < p.M; ++m) g.dW[m] = dW[m];
    g.dw_bf16 = prm.dW_dtype == ATGRPO_BF16, g.dw_accumulate = prm.accumulate_dW;
    int rc = launch_gemm<kDz>(m_dz, g, n_pt * g.n_vtiles, p.n_sm, st);
    if (rc != ATGRPO_OK) return rc;
    rc = launch_gemm<kDh>(m_dh, g, n_pt * n_dt, p.n_sm, st);
    if (rc != ATGRPO_OK) return rc;
    rc = launch_gemm<kDw>(m_dw, g, (int64_t)p.M * ((g.vc_valid + kPairRows - 1) / kPairRows) * n_dt, p.n_sm, st);
    if (rc != ATGRPO_OK) return rc;
  }
  if (!dH_direct) {
    const int64_t total = p.T * (p.d / 4);
    int64_t grid = (total + 255) / 256;
    if (grid > 148 * 16) grid = 148 * 16;
    if (grid < 1) grid = 1;
    if (prm.dH_dtype == ATGRPO_BF16)
      k_dh_finalize<true><<<(int)grid, 256, 0, st>>>(dh_acc, row_of_token, p.T, p.d, dH);
    else
      k_dh_finalize<false><<<(int)grid, 256, 0, st>>>(dh_acc, row_of_token, p.T, p.d, dH);
  }
  return launch_ok();
}

}  // namespace atgrpo
