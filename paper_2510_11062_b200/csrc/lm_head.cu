// LM-head contractions of the policy loss (pi_theta of Eq. 2 and the gradient of Eq. 2) on the
// sm_100a tensor cores.  One warp-specialised persistent kernel serves four kinds of work item:
//
//   kFwd : z = H W_m^T tile by tile, streaming logsumexp and target-logit gather in the epilogue;
//          the logits only ever exist in tensor memory.
//   kDz  : the same contraction for one vocabulary chunk; the epilogue turns the logits into
//          dZ = coef*(softmax - onehot) and writes them as bf16 into the chunk buffer.
//   kDh  : dH_rows += dZ_chunk * W_m[chunk, :]          (A K-major, B MN-major)
//   kDw  : dW_m[chunk, :] = dZ_chunk^T * H_rows          (A and B MN-major)
//
// The forward call is one kFwd launch.  The backward call is one kBwd launch per vocabulary chunk
// plus one: launch c holds the long dH and dW tiles of chunk c-1 and the short dZ tiles of chunk c
// (two chunk buffers, used alternately), ordered long-first with the short tiles topping up the
// pairs that got one long tile fewer, so a launch ends within about one short tile on every pair.
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
//
// Kept logits (optional): when the caller lends a [T, ldz] fp32 buffer, the kFwd epilogue also
// stores every logit it reads from tensor memory (rows of tokens whose response has advantage 0 are
// skipped: they pass no gradient whatever their ratio), and the backward call forms dZ from those
// instead of repeating the contraction: no kDz items, a quarter of the backward's tensor work
// gone for 4 bytes per logit written once and read once.  The conversion of chunk c is done by
// kConvWarps extra warps of the launch that holds the dH and dW tiles of chunk c-1 (plain loads
// and stores, no barriers), so it runs under the tensor work; chunk 0 has a small launch of its
// own.  Both ways give the same bits: the stored value is the accumulator the recomputation would
// produce again.  A compact format halves the traffic of the kept logits: per token and 32-column
// block the block's maximum in fp32 and, per logit, a 16-bit code q = round((max - z) * 1024) (clamped at
// 65535, i.e. 64 below the block's maximum, where exp(z - lse) no longer matters): |z - z~| <= 2^-11, a
// relative error of at most 4.9e-4 on every softmax value, a quarter of what rounding dZ to bf16 adds
// anyway; no longer bit-identical to the recomputing backward.
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
constexpr int kConvWarps = 8;                   // kBwd with kept logits: warps that turn logits into dZ
constexpr int kConvCols = 2048;                 // columns one conversion step covers (eight 32-byte loads per lane in flight)
constexpr int kCodeCols = 2048;                 // the same for 16-bit codes (16 columns per 32-byte load, four loads in flight)
constexpr float kCodeScale = 1024.f;            // 16-bit codes: steps per logit unit (2^-10 apart, 64 units of range)
constexpr int kTmemCols = 512;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

enum Mode { kFwd = 0, kDz = 1, kDh = 2, kDw = 3, kBwd = 4 /* a launch mixing kDz, kDh and kDw items */ };

struct Maps {
  CUtensorMap a_z;                       // rows of H (or their gathered copy): K-major boxes of BK x BM
  CUtensorMap a_h;                       // dZ chunk read by kDh: K-major boxes of BK x BM
  CUtensorMap a_w;                       // dZ chunk read by kDw as dZ^T: 64 x 64 boxes
  CUtensorMap b_w;                       // rows of H read by kDw: 64 x 64 boxes
  CUtensorMap b_z[ATGRPO_MAX_HEADS];     // W_m for the logits: K-major boxes of BK x BN/2
  CUtensorMap b_h[ATGRPO_MAX_HEADS];     // W_m read by kDh: 64 x 64 boxes
};

struct GemmArgs {
  const Schedule* sched;
  const int32_t* tok_of_row;
  const int32_t* target;
  int32_t* status;
  int V, d, M;
  int64_t T_pad;
  // kFwd / kDz: vocabulary tiling
  int has_z;              // kBwd: the launch holds kDz items
  int v_begin;            // first vocabulary row of the logits items (0 for kFwd)
  int n_vtiles;           // 256-wide vocabulary tiles of the logits items
  int tiles_per_chunk;    // kFwd: tiles one work item sweeps (1 for kDz)
  int n_chunks;
  int m_block;            // kFwd / kDz: row tiles swept together so their rows of H stay in L2
  float* part_m;          // kFwd out: running max (log2 domain) [2*n_chunks, T_pad]
  float* part_s;          // kFwd out: sum of 2^(t - max)        [2*n_chunks, T_pad]
  float* zt;              // kFwd out: target logit              [T_pad]
  const float* lse;       // kDz in, token order
  const float* coef;      // kDz in, token order
  __nv_bfloat16* dz;      // kDz out: [T_pad, vc]
  int vc;                 // chunk buffer width (multiple of 256)
  float* logits;          // kept logits [T, ldz] in token order (NULL: none): written by kFwd, read instead of kDz items
  int64_t ldz;            // row stride of `logits` in elements (V rounded up to a multiple of 256)
  int q16;                // kept logits are 16-bit codes: `logits` holds uint16 [T, ldz], `refs` fp32 [T, ldz/32]
  float* refs;            // q16: the maximum of every 32-column block; logit = ref - code / kCodeScale
  const int32_t* resp_of_token;   // kFwd with kept logits: a token whose response has advantage 0 passes no
  const float* adv;               // gradient whatever its ratio, so its logits are not stored
  int64_t n_resp;
  // kDh / kDw: the chunk whose dZ an earlier launch wrote (the maps a_h / a_w point at its buffer)
  int has_g;              // kBwd: the launch holds kDh and kDw items
  int g_begin;            // first vocabulary row of that chunk
  int vc_valid;           // vocabulary rows of that chunk that exist (<= vc)
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

// Streaming variants for the kept logits: every byte is written once and read once, far apart, so
// both directions ask L2 to drop the line first and leave the operands of the contractions alone.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}

__device__ __forceinline__ void st_stream_v8(void* p, const uint32_t* v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8}, %9;" ::"l"(p), "r"(v[0]),
               "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "l"(policy)
               : "memory");
}

__device__ __forceinline__ void ld_stream_v8(const void* p, uint32_t* v, uint64_t policy) {
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8], %9;"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "l"(p), "l"(policy)
               : "memory");
}

// 16-bit codes.  A float-to-integer cvt clamps to the range of its destination type (+inf, the code of a
// column beyond the vocabulary, becomes 65535).
__device__ __forceinline__ uint32_t pack_codes(float lo, float hi) {
  uint32_t r;
  asm("{\n\t.reg .b16 l, h;\n\tcvt.rni.u16.f32 l, %1;\n\tcvt.rni.u16.f32 h, %2;\n\tmov.b32 %0, {l, h};\n\t}"
      : "=r"(r) : "f"(lo), "f"(hi));
  return r;
}

__device__ __forceinline__ void unpack_codes(uint32_t v, float& lo, float& hi) {
  asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.rn.f32.u16 %0, l;\n\tcvt.rn.f32.u16 %1, h;\n\t}"
      : "=f"(lo), "=f"(hi) : "r"(v));
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
__device__ __forceinline__ Tile decode_item(int mode, const GemmArgs& g, const Schedule* s, int it, int rank) {
  Tile t;
  const int n_dt = (g.d + BN - 1) / BN;
  t.v0 = 0, t.chunk = 0, t.nt_begin = 0, t.nt_end = 1;
  if (mode == kFwd || mode == kDz) {
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
  } else if (mode == kDh) {
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

// The work items of one CTA pair, in the order the pair runs them.  A forward launch deals its
// items round-robin.  A backward launch holds long items (dH and dW tiles of one chunk: hundreds
// of k-steps) and short ones (dZ tiles of the next chunk: d/64 k-steps): the long items are dealt
// round-robin first, then the pairs that got one long item fewer receive `ratio` short items each
// (ratio = long/short k-steps), and what is left is dealt round-robin again.  Every role of both
// CTAs of a pair walks the same sequence.
struct ItemSeq {
  int pair, n_pairs;
  int n_h, n_big, n_small, small_mode;
  int lead, n_short, pre;
  int phase, k;

  __device__ __forceinline__ void init(int kMode, const GemmArgs& g, const Schedule* s, int pair_, int n_pairs_) {
    pair = pair_, n_pairs = n_pairs_;
    phase = 0, k = 0;
    const int n_pt = s->tile_begin[g.M] / 2;            // heads start on even 128-row tiles
    const int n_dt = (g.d + BN - 1) / BN;
    n_h = 0, n_big = 0, lead = 0, n_short = 0, pre = 0;
    if (kMode == kFwd) {
      small_mode = kFwd;
      n_small = n_pt * g.n_chunks;
      return;
    }
    small_mode = kDz;
    n_small = g.has_z && g.logits == nullptr ? n_pt * g.n_chunks : 0;   // kept logits: dZ comes from the conversion warps
    if (g.has_g) {
      const int n_vt = (g.vc_valid + kPairRows - 1) / kPairRows;
      n_h = n_pt * n_dt;
      n_big = n_h + g.M * n_vt * n_dt;
      lead = n_big % n_pairs;
      if (lead > 0 && n_small > 0) {
        const int k_long = ((g.vc_valid + BK - 1) / BK + (2 * n_pt * (BM / BK) + g.M - 1) / g.M) / 2;
        const int k_short = (g.d + BK - 1) / BK;
        const int ratio = max(1, (k_long + k_short / 2) / k_short);
        n_short = n_pairs - lead;
        pre = min(n_small, n_short * ratio);
      }
    }
  }

  __device__ __forceinline__ bool next(int& mode, int& it) {
    if (phase == 0) {
      const int b = pair + k * n_pairs;
      if (b < n_big) {
        ++k;
        mode = b < n_h ? kDh : kDw;
        it = b < n_h ? b : b - n_h;
        return true;
      }
      phase = 1, k = 0;
    }
    if (phase == 1) {
      if (pre > 0 && pair >= lead) {
        const int j = (pair - lead) + k * n_short;
        if (j < pre) {
          ++k;
          mode = small_mode, it = j;
          return true;
        }
      }
      phase = 2, k = 0;
    }
    const int j = pre + pair + k * n_pairs;
    if (j < n_small) {
      ++k;
      mode = small_mode, it = j;
      return true;
    }
    return false;
  }
};

// dZ of one vocabulary chunk from kept logits: the element-wise half of the kDz epilogue, for warps
// that hold no accumulator.  A step is one row of the chunk buffer x kConvCols columns (8 KiB of
// logits, lanes on consecutive 32-byte pieces); steps are dealt round-robin to `n_workers` warps.
// Same expression, same operand values, hence the same bits as the kDz epilogue.
__device__ __forceinline__ void dz_from_logits(const GemmArgs& g, int64_t rows, int worker, int n_workers,
                                               int lane) {
  const int n_cols = g.n_vtiles * BN;                       // columns of the chunk buffer this chunk fills
  const int n_seg = (n_cols + kConvCols - 1) / kConvCols;
  const uint64_t drop = l2_policy_evict_first();
  // step u = row * n_seg + seg for u = worker, worker + n_workers, ...: (row, seg) advanced without dividing
  const int d_row = n_workers / n_seg, d_seg = n_workers % n_seg;
  int64_t row = worker / n_seg;
  for (int seg = worker % n_seg; row < rows; row += d_row, seg += d_seg) {
    if (seg >= n_seg) seg -= n_seg, ++row;
    if (row >= rows) break;
    const int c0 = seg * kConvCols + lane * 8;              // this lane's first column in the buffer
    const int tok = g.tok_of_row[row];
    int y = -1;
    float lse2 = 0.f, cf = 0.f;
    const float* src = g.logits;
    if (tok >= 0) {
      y = g.target[tok];
      if ((unsigned)y >= (unsigned)g.V) {
        raise_status(g.status, ATGRPO_ERR_BAD_INDEX);
        y = 0;
      }
      lse2 = g.lse[tok] * kLog2e, cf = g.coef[tok];
      src = g.logits + (size_t)tok * g.ldz + g.v_begin + c0;
    }
    uint32_t z[kConvCols / BN][8];
#pragma unroll
    for (int j = 0; j < kConvCols / BN; ++j) {
      const int col = c0 + j * BN;
      // a padding row, or a piece that lies wholly beyond the vocabulary, is not read at all
      if (tok >= 0 && col < n_cols && g.v_begin + col < g.V) {
        ld_stream_v8(src + j * BN, z[j], drop);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) z[j][i] = 0u;
      }
    }
#pragma unroll
    for (int j = 0; j < kConvCols / BN; ++j) {
      const int col = c0 + j * BN;
      if (col >= n_cols) continue;
      const int v0 = g.v_begin + col;                        // vocabulary row of z[j][0]
      float gz[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) gz[i] = cf * ex2(fmaf(__uint_as_float(z[j][i]), kLog2e, -lse2));
      // (a padding row has z = 0, lse = 0 and cf = 0: exact zeros.)  Only the piece that holds the target
      // column or reaches beyond the vocabulary needs more
      if ((unsigned)(y - v0) < 8u || v0 + 8 > g.V) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (v0 + i == y) gz[i] -= cf;
          if (v0 + i >= g.V) gz[i] = 0.f;
        }
      }
      uint4 w;
      __nv_bfloat162* wh = reinterpret_cast<__nv_bfloat162*>(&w);
#pragma unroll
      for (int i = 0; i < 4; ++i) wh[i] = __floats2bfloat162_rn(gz[2 * i], gz[2 * i + 1]);
      *reinterpret_cast<uint4*>(g.dz + (size_t)row * g.vc + col) = w;
    }
  }
}

// The same from 16-bit codes.  A step is one row x kCodeCols columns (4 KiB of codes, lanes on consecutive
// 32-byte pieces of 16 codes, which lie inside one 32-column block and share its reference value).
__device__ __forceinline__ void dz_from_codes(const GemmArgs& g, int64_t rows, int worker, int n_workers,
                                              int lane) {
  constexpr int kLoads = 4, kStride = 32 * 16;               // 32-byte loads per lane and step; columns a warp covers per load
  static_assert(kLoads * kStride == kCodeCols, "a step is kLoads warp-wide loads");
  const int n_cols = g.n_vtiles * BN;
  const int n_seg = (n_cols + kCodeCols - 1) / kCodeCols;
  const int64_t n_blk = g.ldz / 32;
  const uint64_t drop = l2_policy_evict_first();
  const uint16_t* codes = reinterpret_cast<const uint16_t*>(g.logits);
  const float step2 = -kLog2e / kCodeScale;                  // log2-domain size of one code step, negated
  const int d_row = n_workers / n_seg, d_seg = n_workers % n_seg;
  int64_t row = worker / n_seg;
  for (int seg = worker % n_seg; row < rows; row += d_row, seg += d_seg) {
    if (seg >= n_seg) seg -= n_seg, ++row;
    if (row >= rows) break;
    const int c0 = seg * kCodeCols + lane * 16;
    const int tok = g.tok_of_row[row];
    int y = -1;
    float lse2 = 0.f, cf = 0.f;
    const uint16_t* src = codes;
    const float* ref = g.refs;
    if (tok >= 0) {
      y = g.target[tok];
      if ((unsigned)y >= (unsigned)g.V) {
        raise_status(g.status, ATGRPO_ERR_BAD_INDEX);
        y = 0;
      }
      lse2 = g.lse[tok] * kLog2e, cf = g.coef[tok];
      src = codes + (size_t)tok * g.ldz + g.v_begin + c0;
      ref = g.refs + (size_t)tok * n_blk + (g.v_begin + c0) / 32;
    }
    uint32_t z[kLoads][8];
    float base2[kLoads];                                     // (block maximum - lse) in the log2 domain
#pragma unroll
    for (int j = 0; j < kLoads; ++j) {
      const int col = c0 + j * kStride;
      base2[j] = 0.f;
      if (tok >= 0 && col < n_cols && g.v_begin + col < g.V) {
        ld_stream_v8(src + j * kStride, z[j], drop);
        base2[j] = fmaf(ref[j * (kStride / 32)], kLog2e, -lse2);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) z[j][i] = 0u;
      }
    }
#pragma unroll
    for (int j = 0; j < kLoads; ++j) {
      const int col = c0 + j * kStride;
      if (col >= n_cols) continue;
      const int v0 = g.v_begin + col;
      const bool edge = (unsigned)(y - v0) < 16u || v0 + 16 > g.V;   // this piece holds the target column or leaves the vocabulary
      uint32_t packed[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float qlo, qhi;
        unpack_codes(z[j][i], qlo, qhi);
        float lo = cf * ex2(fmaf(qlo, step2, base2[j]));
        float hi = cf * ex2(fmaf(qhi, step2, base2[j]));
        if (edge) {
          if (v0 + 2 * i == y) lo -= cf;
          if (v0 + 2 * i + 1 == y) hi -= cf;
          if (v0 + 2 * i >= g.V) lo = 0.f;
          if (v0 + 2 * i + 1 >= g.V) hi = 0.f;
        }
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
        packed[i] = *reinterpret_cast<const uint32_t*>(&h2);
      }
      st_global_v8(g.dz + (size_t)row * g.vc + col, packed);
    }
  }
}

// The conversion on its own, for the first chunk of a backward call (no tensor work to hide under yet).
__global__ void __launch_bounds__(256)
k_dz_from_logits(const GemmArgs g) {
  const int64_t rows = (int64_t)g.sched->tile_begin[g.M] * BM;
  if (g.q16)
    dz_from_codes(g, rows, blockIdx.x * 8 + (threadIdx.x >> 5), gridDim.x * 8, threadIdx.x & 31);
  else
    dz_from_logits(g, rows, blockIdx.x * 8 + (threadIdx.x >> 5), gridDim.x * 8, threadIdx.x & 31);
}

template <int kMode>    // kFwd or kBwd
__global__ void __launch_bounds__(kMode == kBwd ? kGemmThreads + 32 * kConvWarps : kGemmThreads, 1)
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
    prefetch_tmap(&maps.a_z);
    if (kMode == kBwd && g.has_g) prefetch_tmap(&maps.a_h), prefetch_tmap(&maps.a_w), prefetch_tmap(&maps.b_w);
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
  ItemSeq seq;
  seq.init(kMode, g, sched, pair, n_pairs);
  int item_mode = kFwd, it = 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t keep = l2_policy_evict_last();
      while (ok && seq.next(item_mode, it)) {
        const int mode = kMode == kFwd ? (int)kFwd : item_mode;
        const Tile t = decode_item(mode, g, sched, it, rank);
        for (int nt = t.nt_begin; ok && nt < t.nt_end; ++nt) {
          const int n0 = t.n0 + (nt - t.nt_begin) * BN + rank * (BN / 2);   // this CTA's half of B
          for (int ks = 0; ks < t.k_steps; ++ks) {
            if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, s_abort, g.status))) break;
            const uint32_t sa = smem_base + stage * kStageBytes, sb = sa + kABytes;
            const uint32_t fb = mapa_shared(full_bar(stage), 0);             // the leader's barrier
            if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * kStageBytes);
            if (mode == kFwd || mode == kDz) {
              tma_load_2d_pair_hint(sa, &maps.a_z, ks * BK, t.row0, fb, keep);        // rows of H: re-read per W tile
              tma_load_2d_pair(sb, &maps.b_z[t.head], ks * BK, n0, fb);
            } else if (mode == kDh) {
              tma_load_2d_pair(sa, &maps.a_h, ks * BK, t.row0, fb);                    // dZ: shared by the d tiles
#pragma unroll
              for (int b = 0; b < 2; ++b)                                             // W chunk: re-read per wave
                tma_load_2d_pair_hint(sb + b * kBoxBytes, &maps.b_h[t.head], n0 + 64 * b, g.g_begin + ks * BK, fb, keep);
            } else {
#pragma unroll
              for (int b = 0; b < 2; ++b)
                tma_load_2d_pair(sa + b * kBoxBytes, &maps.a_w, t.v0 + 64 * b, t.row0 + ks * BK, fb);
#pragma unroll
              for (int b = 0; b < 2; ++b)                                             // H: re-read per wave
                tma_load_2d_pair_hint(sb + b * kBoxBytes, &maps.b_w, n0 + 64 * b, t.row0 + ks * BK, fb, keep);
            }
            if (++stage == kStages) stage = 0, phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      while (ok && seq.next(item_mode, it)) {
        const int mode = kMode == kFwd ? (int)kFwd : item_mode;
        // Everything that depends on the item's kind is settled here, once per item: the single
        // issuing thread has about 128 cycles per MMA, so the inner loop only adds offsets.
        const bool a_mn = (mode == kDw), b_mn = (mode == kDh || mode == kDw);
        const uint32_t idesc = mode == kDw   ? idesc_bf16(kPairRows, BN, true, true)
                               : mode == kDh ? idesc_bf16(kPairRows, BN, false, true)
                                             : idesc_bf16(kPairRows, BN, false, false);
        const uint64_t a_desc0 = a_mn ? smem_desc(0, kBoxBytes, 1024) : smem_desc(0, 16, 1024);
        const uint64_t b_desc0 = b_mn ? smem_desc(0, kBoxBytes, 1024) : smem_desc(0, 16, 1024);
        const uint64_t a_kk = (a_mn ? 2048u : 32u) >> 4, b_kk = (b_mn ? 2048u : 32u) >> 4;   // K step of 16 elements
        const Tile t = decode_item(mode, g, sched, it, rank);
        if (t.k_steps == 0) continue;
        for (int nt = t.nt_begin; ok && nt < t.nt_end; ++nt) {
          if (!(ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, s_abort, g.status))) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * BN;
          for (int ks = 0; ks < t.k_steps; ++ks) {
            if (!(ok = mbar_wait(full_bar(stage), phase, s_abort, g.status))) break;
            tc_fence_after();
            // the start-address field holds (address >> 4) in 14 bits: shared memory stays below
            // 2^18 bytes, so adding the offsets never carries into the next field
            const uint32_t sa = smem_base + stage * kStageBytes, sb = sa + kABytes;
            const uint64_t ad = a_desc0 + (sa >> 4), bd = b_desc0 + (sb >> 4);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              umma_bf16_pair(d_tmem, ad + kk * a_kk, bd + kk * b_kk, idesc, (ks | kk) != 0 ? 1u : 0u);
            umma_commit_pair(empty_bar(stage), 3);   // frees the stage in both CTAs
            if (++stage == kStages) stage = 0, phase ^= 1u;
          }
          if (!ok) break;
          umma_commit_pair(tfull_bar(acc), 3);        // accumulator complete in both CTAs
          if (++acc == 2) acc = 0, acc_phase ^= 1u;
        }
      }
    }
  } else if (warp >= kGemmThreads / 32) {
    // ------------------------------------------------------------------ conversion warps (kBwd, kept logits)
    if (kMode == kBwd && g.has_z && g.logits != nullptr) {
      const int64_t rows = (int64_t)sched->tile_begin[g.M] * BM;
      const int worker = blockIdx.x * kConvWarps + (warp - kGemmThreads / 32);
      if (g.q16)
        dz_from_codes(g, rows, worker, gridDim.x * kConvWarps, lane);
      else
        dz_from_logits(g, rows, worker, gridDim.x * kConvWarps, lane);
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
    const uint64_t drop = l2_policy_evict_first();
    const uint32_t tempty_leader0 = mapa_shared(tempty_bar(0), 0), tempty_leader1 = mapa_shared(tempty_bar(1), 0);
    while (ok && seq.next(item_mode, it)) {
      const int mode = kMode == kFwd ? (int)kFwd : item_mode;
      const Tile t = decode_item(mode, g, sched, it, rank);
      uint32_t r[32];

      if (mode == kFwd || mode == kDz) {
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
        if (mode == kDz && tok >= 0) lse2 = g.lse[tok] * kLog2e, cf = g.coef[tok];
        float* keep_row = nullptr;            // fp32 logits of this token, or
        uint16_t* keep_codes = nullptr;       // its 16-bit codes and
        float* keep_refs = nullptr;           // the block maxima they refer to
        if (mode == kFwd && g.logits != nullptr && tok >= 0) {
          const int rsp = g.resp_of_token[tok];
          if ((unsigned)rsp < (unsigned)g.n_resp && g.adv[rsp] != 0.f) {
            if (g.q16) {
              keep_codes = reinterpret_cast<uint16_t*>(g.logits) + (size_t)tok * g.ldz;
              keep_refs = g.refs + (size_t)tok * (g.ldz / 32);
            } else {
              keep_row = g.logits + (size_t)tok * g.ldz;
            }
          }
        }
        for (int nt = t.nt_begin; ok && nt < t.nt_end; ++nt) {
          const int n0 = t.n0 + (nt - t.nt_begin) * BN;
          if (!(ok = mbar_wait_backoff(tfull_bar(acc), acc_phase, s_abort, g.status))) break;
          tc_fence_after();
          float ref0 = 0.f, ref1 = 0.f, ref2 = 0.f, ref3 = 0.f;   // q16: maxima of this warp's four column blocks
          for (int c = c_begin; c < c_end; ++c) {
            const int col0 = n0 + c * 32;
            if (mode == kFwd && col0 >= g.V) break;
            __syncwarp();
            tmem_ld32(lane_addr + acc * BN + c * 32, r);
            tmem_ld_wait();
            if (mode == kFwd) {
              if (keep_row != nullptr) {
                // the logits as the tensor cores delivered them, 128 bytes of this token's row
#pragma unroll
                for (int q8 = 0; q8 < 4; ++q8) st_stream_v8(keep_row + col0 + 8 * q8, r + 8 * q8, drop);
              }
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
              if (keep_codes != nullptr) {
                // code = (block maximum - logit) in steps of 1/kCodeScale, saturating (columns beyond V are -inf)
                const float top = cmax * kCodeScale;
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                  pk[i] = pack_codes(fmaf(__uint_as_float(r[2 * i]), -kCodeScale, top),
                                     fmaf(__uint_as_float(r[2 * i + 1]), -kCodeScale, top));
                st_stream_v8(keep_codes + col0, pk, drop);
                st_stream_v8(keep_codes + col0 + 16, pk + 8, drop);
                const int k = c - c_begin;
                if (k == 0) ref0 = cmax;
                else if (k == 1) ref1 = cmax;
                else if (k == 2) ref2 = cmax;
                else ref3 = cmax;
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
          if (keep_refs != nullptr)          // 16 bytes: the four blocks this warp covers of the tile at n0
            *reinterpret_cast<float4*>(keep_refs + n0 / 32 + c_begin) = make_float4(ref0, ref1, ref2, ref3);
        }
        if (mode == kFwd && ok && tok >= 0) {
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
        if (mode == kDh) {
          valid = r_in_tile < t.rows_valid;
          out_row = (size_t)(t.row0 + r_in_tile);
        } else {
          const int v = g.g_begin + t.v0 + r_in_tile;
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
          if (mode == kDh || !g.dw_bf16) {
            float* dst = (mode == kDh ? g.dh_acc : static_cast<float*>(g.dW[t.head])) +
                         out_row * g.d + col0;
            const bool add = mode == kDh ? !g.first_chunk : (g.dw_accumulate != 0);
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
    // four parts per round: their eight loads are issued together, then merged in ascending part order
    for (int c0 = grp; c0 < n_parts; c0 += 32) {
      float ps[4], pm[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = c0 + 8 * k;
        ps[k] = c < n_parts ? part_s[(size_t)c * T_pad + p] : 0.f;
        pm[k] = c < n_parts ? part_m[(size_t)c * T_pad + p] : 0.f;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (ps[k] > 0.f) {                              // a part without valid columns holds (-inf, 0)
          const float nm = fmaxf(mx, pm[k]);
          s = s * exp2f(mx - nm) + ps[k] * exp2f(pm[k] - nm);
          mx = nm;
        }
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

// Width of one dZ chunk buffer (a multiple of 256 columns).  A backward launch mixes the long
// tiles of one chunk with the short ones of the next, so wave quantisation does not depend on the
// width; wide chunks mean fewer launches and fewer read-modify-write passes over the dH
// accumulator, as long as the chunk's rows of W (vc * d * 2 bytes, re-read by every wave of dH
// tiles) still fit in L2: at the Qwen3-1.7B shape 256 MiB and 1 GiB buffers both measured 4-5 %
// slower than 512 MiB (vc = 16384 there, 64 MiB of W).  So: each buffer gets 512 MiB, or for
// batches whose 512 MiB would be narrower than that, as many columns as keep the chunk's rows of
// W within 64 MiB (at most 16384), up to 3 GiB per buffer (a long-response micro-batch of 78 K
// tokens then walks the vocabulary in 10 chunks instead of 46).  The vocabulary is cut into
// equal chunks.
int bwd_chunk_width(int64_t T_pad, int d, int V) {
  const int64_t budget = 512ll << 20, budget_max = 3072ll << 20, w_bytes = 64ll << 20;
  if (T_pad < kPairRows) T_pad = kPairRows;            // T = 0: keep the arithmetic below defined
  const int64_t vmax = (int64_t)(V + BN - 1) / BN * BN;
  int64_t cap = budget / (T_pad * 2) / BN * BN;
  int64_t wide = w_bytes / ((int64_t)(d > 0 ? d : 1) * 2) / BN * BN;
  const int64_t wide_fit = budget_max / (T_pad * 2) / BN * BN;
  if (wide > 16384) wide = 16384;
  if (wide > wide_fit) wide = wide_fit;
  if (cap < wide) cap = wide;
  if (cap < BN) cap = BN;
  if (cap > vmax) cap = vmax;
  const int64_t n_chunks = (V + cap - 1) / cap;
  const int64_t vc = ((V + n_chunks - 1) / n_chunks + BN - 1) / BN * BN;
  return (int)vc;
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

struct BwdPlan { size_t dz[2], dh_acc, total; int vc; };
BwdPlan bwd_plan(int64_t T_pad, int d, int V, bool dH_direct) {
  BwdPlan p;
  p.vc = bwd_chunk_width(T_pad, d, V);
  Carver c(nullptr);
  for (int i = 0; i < 2; ++i) {
    p.dz[i] = c.off;
    if (i == 0 || V > p.vc) c.take<__nv_bfloat16>((size_t)T_pad * p.vc);   // one chunk: one buffer
  }
  p.dh_acc = c.off;
  if (!dH_direct) c.take<float>((size_t)T_pad * d);
  p.total = c.off;
  return p;
}

// Launches `pairs` clusters of two CTAs (never more than can be resident at once); `items` is an
// upper bound of the launch's work items.
template <int kMode>
int launch_gemm(const Maps& maps, const GemmArgs& g, int64_t items, int n_sm, cudaStream_t st,
                int threads = kGemmThreads) {
  if (cudaFuncSetAttribute(k_lm_head<kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSmemBytes) != cudaSuccess)
    return ATGRPO_ERR_CUDA;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2, attr[0].val.clusterDim.y = 1, attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(threads, 1, 1);
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

int lm_head_bwd_chunks(int64_t T_pad, int32_t d, int32_t V) {
  const int vc = bwd_chunk_width(T_pad, d, V);
  return (V + vc - 1) / vc;
}

int lm_head_bwd_chunk_rows(int64_t T_pad, int32_t d, int32_t V) { return bwd_chunk_width(T_pad, d, V); }

size_t lm_head_fwd_workspace_bytes(int64_t T_pad, int32_t d, int32_t V, int32_t n_sm) {
  (void)d;
  return fwd_plan(T_pad, V, n_sm).total;
}

int64_t lm_head_logits_ld(int32_t V) { return ((int64_t)V + BN - 1) / BN * BN; }

size_t lm_head_logits_bytes(int64_t T, int32_t V, int32_t format) {
  const size_t n = (size_t)T * lm_head_logits_ld(V);
  return format == ATGRPO_LOGITS_Q16 ? n * 2 + n / 32 * 4 : n * 4;     // codes + one fp32 per 32-column block
}

namespace {
// Where the block maxima of the 16-bit format start inside the lent buffer: after the codes.
float* logits_refs(const void* buf, int64_t T, int32_t V) {
  return reinterpret_cast<float*>(static_cast<char*>(const_cast<void*>(buf)) + (size_t)T * lm_head_logits_ld(V) * 2);
}
}  // namespace

int lm_head_fwd_launch(const LmHeadProblem& p, float* lse, float* logp, void* workspace,
                       cudaStream_t st, float* keep_logits, int32_t logits_format) {
  const FwdPlan pl = fwd_plan(p.T_pad, p.V, p.n_sm);
  char* ws = static_cast<char*>(workspace);
  Maps maps;
  memset(&maps, 0, sizeof(maps));
  if (!make_map(&maps.a_z, p.A_rows, p.d, p.rows_bound, p.ldA, BK, BM)) return ATGRPO_ERR_CUDA;
  for (int m = 0; m < p.M; ++m)
    if (!make_map(&maps.b_z[m], p.W[m], p.d, p.V, p.d, BK, BN / 2)) return ATGRPO_ERR_CUDA;
  GemmArgs g = base_args(p);
  g.v_begin = 0, g.n_vtiles = pl.n_vt, g.tiles_per_chunk = pl.tiles_per_chunk, g.n_chunks = pl.n_chunks;
  g.m_block = row_block_tiles(p.T_pad / kPairRows, p.d);
  g.part_m = reinterpret_cast<float*>(ws + pl.part_m);
  g.part_s = reinterpret_cast<float*>(ws + pl.part_s);
  g.zt = reinterpret_cast<float*>(ws + pl.zt);
  g.logits = keep_logits, g.ldz = lm_head_logits_ld(p.V);
  g.q16 = logits_format == ATGRPO_LOGITS_Q16, g.refs = logits_refs(keep_logits, p.T, p.V);
  g.resp_of_token = p.resp_of_token, g.adv = p.adv, g.n_resp = p.n_resp;
  int rc = launch_gemm<kFwd>(maps, g, (p.T_pad / kPairRows) * pl.n_chunks, p.n_sm, st);
  if (rc != ATGRPO_OK) return rc;
  const int cgrid = (int)((p.T_pad + 31) / 32 > 0 ? (p.T_pad + 31) / 32 : 1);
  k_lse_combine<<<cgrid, dim3(32, 8), 0, st>>>(p.sched, p.M, p.tok_of_row, p.T_pad, 2 * pl.n_chunks, g.part_m,
                                               g.part_s, g.zt, lse, logp);
  return launch_ok();
}

size_t lm_head_bwd_workspace_bytes(int64_t T_pad, int32_t d, int32_t V, bool dH_direct) {
  return bwd_plan(T_pad, d, V, dH_direct).total;
}

int lm_head_bwd_launch(const LmHeadProblem& p, const float* lse, const float* coef,
                       const int32_t* row_of_token, const atgrpo_params& prm, void* dH,
                       void* const* dW, void* workspace, cudaStream_t st, void* const* chunk_events,
                       const float* kept_logits, int32_t logits_format) {
  const bool dH_direct = false;   // rows are compacted: dH always goes through the accumulator
  const BwdPlan pl = bwd_plan(p.T_pad, p.d, p.V, dH_direct);
  char* ws = static_cast<char*>(workspace);
  __nv_bfloat16* dz[2] = {reinterpret_cast<__nv_bfloat16*>(ws + pl.dz[0]),
                          reinterpret_cast<__nv_bfloat16*>(ws + pl.dz[1])};
  float* dh_acc = dH_direct ? static_cast<float*>(dH) : reinterpret_cast<float*>(ws + pl.dh_acc);

  // Maps that do not depend on the chunk buffer, then one pair (K-major / transposed view) per buffer.
  Maps base;
  memset(&base, 0, sizeof(base));
  if (!make_map(&base.a_z, p.A_rows, p.d, p.rows_bound, p.ldA, BK, BM)) return ATGRPO_ERR_CUDA;
  if (!make_map(&base.b_w, p.A_rows, p.d, p.rows_bound, p.ldA, 64, 64)) return ATGRPO_ERR_CUDA;
  for (int m = 0; m < p.M; ++m) {
    if (!make_map(&base.b_z[m], p.W[m], p.d, p.V, p.d, BK, BN / 2)) return ATGRPO_ERR_CUDA;
    if (!make_map(&base.b_h[m], p.W[m], p.d, p.V, p.d, 64, 64)) return ATGRPO_ERR_CUDA;
  }
  const int n_chunks = (p.V + pl.vc - 1) / pl.vc;
  const int n_buf = n_chunks > 1 ? 2 : 1;
  CUtensorMap a_h[2], a_w[2];
  for (int i = 0; i < n_buf; ++i) {
    if (!make_map(&a_h[i], dz[i], pl.vc, p.T_pad, pl.vc, BK, BM)) return ATGRPO_ERR_CUDA;
    if (!make_map(&a_w[i], dz[i], pl.vc, p.T_pad, pl.vc, 64, 64)) return ATGRPO_ERR_CUDA;
  }
  const int64_t n_pt = p.T_pad / kPairRows;
  const int n_dt = (p.d + BN - 1) / BN;
  // Launch c: dZ of chunk c (if there is one) into buffer c % 2, dH and dW of chunk c - 1.
  for (int c = 0; c <= n_chunks; ++c) {
    GemmArgs g = base_args(p);
    Maps maps = base;
    int64_t items = 0;
    g.vc = pl.vc;
    g.lse = lse, g.coef = coef;
    g.logits = const_cast<float*>(kept_logits), g.ldz = lm_head_logits_ld(p.V);
    g.q16 = logits_format == ATGRPO_LOGITS_Q16, g.refs = logits_refs(kept_logits, p.T, p.V);
    g.dh_acc = dh_acc;
    for (int m = 0; m < p.M; ++m) g.dW[m] = dW[m];
    g.dw_bf16 = prm.dW_dtype == ATGRPO_BF16, g.dw_accumulate = prm.accumulate_dW;
    if (c < n_chunks) {
      g.has_z = 1;
      g.v_begin = c * pl.vc;
      const int valid = p.V - g.v_begin < pl.vc ? p.V - g.v_begin : pl.vc;
      g.n_vtiles = (valid + BN - 1) / BN;
      g.tiles_per_chunk = 1;
      g.n_chunks = g.n_vtiles;
      g.m_block = row_block_tiles(n_pt, p.d);
      g.dz = dz[c % n_buf];
      items += n_pt * g.n_vtiles;
    }
    if (c > 0) {
      g.has_g = 1;
      g.g_begin = (c - 1) * pl.vc;
      g.vc_valid = p.V - g.g_begin < pl.vc ? p.V - g.g_begin : pl.vc;
      g.first_chunk = c == 1;
      maps.a_h = a_h[(c - 1) % n_buf];
      maps.a_w = a_w[(c - 1) % n_buf];
      items += n_pt * n_dt + (int64_t)p.M * ((g.vc_valid + kPairRows - 1) / kPairRows) * n_dt;
    }
    if (kept_logits != nullptr && c == 0) {
      // nothing to hide the first chunk's conversion under: a launch of its own, every SM full of warps
      k_dz_from_logits<<<4 * p.n_sm, 256, 0, st>>>(g);
      const int rc0 = launch_ok();
      if (rc0 != ATGRPO_OK) return rc0;
      continue;
    }
    const int rc = launch_gemm<kBwd>(maps, g, items, p.n_sm, st,
                                     kept_logits != nullptr && c < n_chunks ? kGemmThreads + 32 * kConvWarps
                                                                            : kGemmThreads);
    if (rc != ATGRPO_OK) return rc;
    if (chunk_events != nullptr && c > 0)             // the dW rows of chunk c - 1 are final
      ATGRPO_CUDA_OK(cudaEventRecord(static_cast<cudaEvent_t>(chunk_events[c - 1]), st));
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
