// K3 / K4: the two grouped GEMMs of the layer on the 5th-generation tensor cores.
//
//   K3 (stage 1, expansion side U_e of Sec. 4.1): for every source group, the rows of h of its
//       (token, source) slots, [rows,H] x [W_gate | W_up]^T with SiLU(gate)*up fused in the epilogue.
//       The epilogue writes each bf16 row of U straight to the stage-2 position of every path that
//       reuses it (Sec. 4.3: one U_i(h) per unique source, read by all of its targets), so stage 2
//       needs no gather.  While the first tile's MMAs run, the epilogue warps also clear y.
//   K4 (stage 2, projection side D_e and the weighted path sum of Sec. 4.3): for every target
//       group, [rows,F] x W_down^T, scaled by the path weight and added into y[token] with vector
//       reductions (the scatter-combine back to token order).
//   The shared expert rides in the same two launches as a second run of tiles (one identity group).
//
// One persistent CTA per SM walks a tile list derived on the device by the grouping step
// (groups padded to 128-row tiles).  Warp roles: warp 0 feeds a 4-stage shared-memory ring with
// TMA tile loads (128-byte swizzle), warp 1 issues tcgen05.mma (128 x 256 x 16, bf16 in, fp32
// accumulate in TMEM, two accumulator stages), warps 2-5 drain TMEM with tcgen05.ld and run the
// epilogue while the next tile's MMAs proceed.
// Every wait on an mbarrier is bounded: on expiry the CTA records PCOMOE_ERR_TIMEOUT, lets its
// copies land, frees TMEM and returns.
#include "tc_ptx.cuh"

namespace pcomoe {
namespace {

constexpr int STAGES = 4;
constexpr uint32_t A_BYTES = kTileM * BK * 2;       // 16 KB
constexpr uint32_t B_BYTES = 256 * BK * 2;          // 32 KB
constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
constexpr uint32_t ACC_COLS = 256;                  // fp32 accumulator columns per stage
constexpr uint32_t TMEM_COLS = 512;
constexpr int kThreads = 192;
constexpr int kEpiStride = 36;               // words per row staged by the epilogue: 16-byte aligned, conflict-free

// One run of tiles that share tensor maps, k-loop length and epilogue parameters: the routed groups, or
// the shared expert (a single group whose rows are the tokens themselves).
struct Seg {
  const int32_t *tile_base;    // [G+1] prefix of m-tiles per group (device); NULL: one group
  const int32_t *row_offsets;  // [G+1] unpadded row offsets per group (device); NULL: one group
  int32_t G;
  int32_t single_rows;         // rows of the single group when tile_base is NULL
  int32_t nt;                  // tiles along N
  int32_t kb;                  // k-blocks
  int32_t b_group_rows;        // rows of the weight tensor per group (0 for a single group)
  int32_t m_outer;             // tile order inside a group: 0 = the m-tiles of one n-tile run fastest (the group's rows
                               // stay in L2 and its weights stream), 1 = the n-tiles of one m-tile run fastest (for a
                               // group whose rows outweigh its weights: the shared expert on a large batch)
  // stage 1: where a row's SwiGLU output goes
  const int32_t *row_token;    // token of a padded row (routed), NULL: the row is its own destination
  const int32_t *path_prow1;   // [T,K] padded stage-1 row of every path
  const int32_t *path_pos2;    // [T,K] padded stage-2 row of every path (= row of u_out to write); a row that
                               //       several paths of the token feed is stored as -(row + 2)
  const float *path_w;         // [T,K] path weights: scale of a contribution to such a shared row
  __nv_bfloat16 *u_out;
  int32_t ldu;
  // stage 2: where a row's projection goes
  const int32_t *s2_token;     // token of an unpadded row; NULL: identity
  const float *s2_w;           // weight of an unpadded row; NULL: 1
};

struct TcParams {
  Seg seg[2];
  int32_t nseg;
  int32_t K;
  float *y;
  int32_t ldy;
  int32_t T;
  float4 *zero_ptr;            // stage 1 only: buffer the epilogue warps clear before their first tile
  int64_t zero_vec4;           //               (y, so that stage 2 can accumulate into it); 0: nothing
  DevPlan *plan;
  uint64_t wait_ns;            // limit of every mbarrier wait
};

// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 256
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
struct TileInfo {
  int seg, g, m_idx, n_idx;
  int prow0;    // first padded row of the tile
  int urow0;    // first unpadded row of the tile
  int valid;    // rows of the tile that exist
};

// Tiles are numbered segment by segment and group by group; inside a group the m-tiles run fastest so
// that CTAs working at the same time share one slice of the group's weights.
struct TileWalker {
  const int32_t *tb, *ro;      // [2][kMaxExperts + 2] each
  int nt0, nt1, G0, G1, mo0, mo1, nseg;   // per segment (scalars: indexed arrays would live in local memory)
  int seg, g;                  // current segment and group
  int tiles0;                  // tiles of segment 0
  __device__ void init() {
    seg = 0; g = 0;
    tiles0 = tb[G0] * nt0;
  }
  __device__ int total() const { return tiles0 + (nseg > 1 ? tb[(kMaxExperts + 2) + G1] * nt1 : 0); }
  __device__ int seg_of(int tile) const { return (nseg > 1 && tile >= tiles0) ? 1 : 0; }
  __device__ TileInfo at(int tile) {
    if (seg == 0 && nseg > 1 && tile >= tiles0) {
      seg = 1;
      g = 0;
    }
    const int32_t *b = tb + seg * (kMaxExperts + 2), *r = ro + seg * (kMaxExperts + 2);
    const int n_t = seg ? nt1 : nt0, Gs = seg ? G1 : G0, m_out = seg ? mo1 : mo0;
    const int local_seg = tile - (seg ? tiles0 : 0);
    while (g + 1 < Gs && local_seg >= b[g + 1] * n_t) ++g;
    TileInfo t;
    const int mt = b[g + 1] - b[g];
    const int local = local_seg - b[g] * n_t;
    t.seg = seg;
    t.g = g;
    if (m_out) {
      t.m_idx = local / n_t;
      t.n_idx = local - t.m_idx * n_t;
    } else {
      t.n_idx = local / mt;
      t.m_idx = local - t.n_idx * mt;
    }
    t.prow0 = (b[g] + t.m_idx) * kTileM;
    t.urow0 = r[g] + t.m_idx * kTileM;
    t.valid = min(kTileM, r[g + 1] - t.urow0);
    return t;
  }
};

// The stage-1 epilogue first lists the warp's (row, destination) pairs compactly in shared memory, so that the
// write-out below runs over the destinations that exist (about 1.1-1.3 per row) instead of over the warp's maximum.
constexpr int kDstList = 256;                // entries per epilogue warp (32 rows x up to 8 destinations)
struct DstList {
  int32_t *dst;      // [kDstList]
  uint8_t *row;      // [kDstList]
  float *w;          // [kDstList] (projection-side reuse only)
};

// What an epilogue thread needs to know about its row, looked up before the accumulator is ready so that
// the loads overlap the MMAs.
struct RowCtx {
  bool ok;            // the row exists and its token is in range
  int token;
  float wgt;          // stage 2: path weight
  int my_prow;        // padded row of this thread
  int n_dst;          // stage 1: entries of the warp's destination list; -1: too many for the list, look up on the spot
};

template <int STAGE, bool MERGE>
__device__ __forceinline__ RowCtx prepare_row(const TcParams &p, const Seg &S, const TileInfo &t, int r, const DstList dl) {
  RowCtx c;
  const int lane = threadIdx.x & 31;
  const bool valid = r < t.valid;
  c.token = 0;
  c.wgt = 0.0f;
  c.my_prow = t.prow0 + r;
  c.n_dst = 0;
  if (STAGE == 1) {
    if (valid && S.row_token) c.token = S.row_token[c.my_prow];
  } else if (valid) {
    const int urow = t.urow0 + r;
    c.token = S.s2_token ? S.s2_token[urow] : urow;
    c.wgt = S.s2_w ? S.s2_w[urow] : 1.0f;
  }
  c.ok = valid && (unsigned)c.token < (unsigned)p.T;
  if (valid && !c.ok) atomicCAS(&p.plan->status, 0, PCOMOE_ERR_INDEX);
  if (STAGE == 1) {
    // the warp's (row, destination) pairs, compacted with ballots: a (token, source) slot feeds every path of the
    // token that has this source (Sec. 4.3 reuse); a row of the shared expert feeds itself
    const unsigned below = (1u << lane) - 1u;
    if (!S.row_token) {
      const unsigned m = __ballot_sync(0xffffffffu, c.ok);
      if (c.ok) {
        const int pos = __popc(m & below);
        dl.dst[pos] = c.my_prow;
        dl.row[pos] = (uint8_t)lane;
      }
      c.n_dst = __popc(m);
    } else {
      int base = 0;
      const size_t q0 = (size_t)c.token * p.K;
      for (int k = 0; k < p.K; ++k) {
        const bool hit = c.ok && S.path_prow1[q0 + k] == c.my_prow;
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        const int n_hit = __popc(m);
        if (base + n_hit > kDstList) {   // the same decision in every lane
          base = -1;
          break;
        }
        if (hit) {
          const int pos = base + __popc(m & below);
          dl.dst[pos] = S.path_pos2[q0 + k];
          dl.row[pos] = (uint8_t)lane;
          if (MERGE) dl.w[pos] = S.path_w[q0 + k];
        }
        base += n_hit;
      }
      c.n_dst = base;
    }
    __syncwarp();
  }
  return c;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

// Stage 1: SiLU(gate) * up for 32 columns held in registers, packed to bf16 (16 words).
__device__ __forceinline__ void swiglu_pack32(const uint32_t (&g)[32], const uint32_t (&u)[32], uint4 (&out)[4]) {
  uint32_t *o = reinterpret_cast<uint32_t *>(out);
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    __nv_bfloat162 h2 = __floats2bfloat162_rn(silu_mul(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i])),
                                              silu_mul(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1])));
    o[i] = *reinterpret_cast<uint32_t *>(&h2);
  }
}

// Eight bf16 values scaled by `sc` and added to eight bf16 values in global memory (a stage-2 row that several
// paths of a token feed: the row starts from zero and collects beta * U of each of them).
__device__ __forceinline__ void red_add_scaled_bf16x8(__nv_bfloat16 *addr, uint4 x, float sc) {
  uint32_t *w = reinterpret_cast<uint32_t *>(&x);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h2 = *reinterpret_cast<__nv_bfloat162 *>(&w[i]);
    const float2 f = __bfloat1622float2(h2);
    h2 = __floats2bfloat162_rn(f.x * sc, f.y * sc);
    w[i] = *reinterpret_cast<uint32_t *>(&h2);
  }
  asm volatile("red.global.add.noftz.v4.bf16x2 [%0], {%1, %2, %3, %4};" ::"l"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3])
               : "memory");
}

// Direct store of 32 bf16 of this thread's row to every path that reuses it, looked up on the spot
// (only when a token has more paths than the destination registers hold).
template <bool MERGE>
__device__ __forceinline__ void store_row_lookup(const TcParams &p, const Seg &S, const RowCtx &c, size_t col,
                                                 const uint4 (&out)[4]) {
  for (int k = 0; k < p.K; ++k) {
    if (S.path_prow1[(size_t)c.token * p.K + k] != c.my_prow) continue;
    const int d = S.path_pos2[(size_t)c.token * p.K + k];
    if (d >= 0) {
      uint4 *d4 = reinterpret_cast<uint4 *>(S.u_out + (size_t)d * S.ldu + col);
#pragma unroll
      for (int q = 0; q < 4; ++q) d4[q] = out[q];
    } else if (MERGE && d <= -2) {
      const float sc = S.path_w[(size_t)c.token * p.K + k];
      __nv_bfloat16 *dr = S.u_out + (size_t)(-d - 2) * S.ldu + col;
#pragma unroll
      for (int q = 0; q < 4; ++q) red_add_scaled_bf16x8(dr + 8 * q, out[q], sc);
    }
  }
}


// Stage 2: this lane's 32 values (one row) are scaled by the path weight, staged, and added to y row by row.
__device__ __forceinline__ void scatter_add_32x32(const TcParams &p, float *stage, const uint32_t (&v)[32], float wgt,
                                                  int tok_or_neg, float *ycol, int lane) {
#pragma unroll
  for (int q = 0; q < 8; ++q)
    *reinterpret_cast<float4 *>(stage + lane * kEpiStride + 4 * q) =
        make_float4(wgt * __uint_as_float(v[4 * q]), wgt * __uint_as_float(v[4 * q + 1]),
                    wgt * __uint_as_float(v[4 * q + 2]), wgt * __uint_as_float(v[4 * q + 3]));
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = i * 4 + (lane >> 3);
    const int tok = __shfl_sync(0xffffffffu, tok_or_neg, row);
    const float4 x = *reinterpret_cast<const float4 *>(stage + row * kEpiStride + 4 * (lane & 7));
    if (tok >= 0) red_add_v4(ycol + (size_t)tok * p.ldy, x.x, x.y, x.z, x.w);
  }
  __syncwarp();
}

// Drains one accumulator (this thread's TMEM lane) and applies the stage's epilogue.  TMEM loads are issued
// one step ahead of the arithmetic: a tcgen05.ld queues behind the MMAs already issued, so its latency is
// long while the next tile is being computed, and must overlap the math and the stores of the previous step.
template <int STAGE, bool MERGE>
__device__ __forceinline__ void epilogue_tile(const TcParams &p, const Seg &S, const TileInfo &t, const RowCtx &c,
                                              uint32_t taddr, float *stage, const DstList dl) {
  if (STAGE == 1) {
    // 32 rows x 64 bf16 columns are collected in shared memory, then every destination row receives its
    // 128 contiguous bytes from eight lanes (whole lines), four rows per instruction.
    const int lane = threadIdx.x & 31;
    const size_t col0 = (size_t)t.n_idx * 128;
    const int n_dst = c.n_dst;
    unsigned char *srow = reinterpret_cast<unsigned char *>(stage) + lane * (kEpiStride * 4);
    uint32_t g0[32], u0[32], g1[32], u1[32];
    tmem_ld32_issue(taddr, g0);
    tmem_ld32_issue(taddr + 128, u0);
#pragma unroll
    for (int c0 = 0; c0 < 128; c0 += 64) {
      uint4 out[4];
      tmem_wait_ld();
      reg_fence32(g0); reg_fence32(u0);
      tmem_ld32_issue(taddr + c0 + 32, g1);
      tmem_ld32_issue(taddr + 128 + c0 + 32, u1);
      swiglu_pack32(g0, u0, out);
      if (c.ok && n_dst < 0) store_row_lookup<MERGE>(p, S, c, col0 + c0, out);
#pragma unroll
      for (int q = 0; q < 4; ++q) reinterpret_cast<uint4 *>(srow)[q] = out[q];
      tmem_wait_ld();
      reg_fence32(g1); reg_fence32(u1);
      if (c0 + 64 < 128) {
        tmem_ld32_issue(taddr + c0 + 64, g0);
        tmem_ld32_issue(taddr + 128 + c0 + 64, u0);
      }
      swiglu_pack32(g1, u1, out);
      if (c.ok && n_dst < 0) store_row_lookup<MERGE>(p, S, c, col0 + c0 + 32, out);
#pragma unroll
      for (int q = 0; q < 4; ++q) reinterpret_cast<uint4 *>(srow + 64)[q] = out[q];
      __syncwarp();
      for (int e0 = 0; e0 < n_dst; e0 += 4) {
        const int e = e0 + (lane >> 3);
        if (e < n_dst) {
          const int row = dl.row[e], d = dl.dst[e];
          const uint4 x = *reinterpret_cast<const uint4 *>(reinterpret_cast<unsigned char *>(stage) +
                                                           row * (kEpiStride * 4) + (lane & 7) * 16);
          if (d >= 0) *reinterpret_cast<uint4 *>(S.u_out + (size_t)d * S.ldu + col0 + c0 + (lane & 7) * 8) = x;
          else if (MERGE && d <= -2)
            red_add_scaled_bf16x8(S.u_out + (size_t)(-d - 2) * S.ldu + col0 + c0 + (lane & 7) * 8, x, dl.w[e]);
        }
      }
      __syncwarp();
    }
  } else {
    // The warp's 32 rows x 32 columns are turned around in shared memory so that one instruction adds
    // 128 contiguous bytes to each of four token rows (whole lines) instead of 16 bytes to 32 rows.
    const int lane = threadIdx.x & 31;
    const int tok_or_neg = c.ok ? c.token : -1;
    float *ybase = p.y + (size_t)t.n_idx * 256 + 4 * (lane & 7);
    uint32_t v0[32], v1[32];
    tmem_ld32_issue(taddr, v0);
#pragma unroll 1
    for (int c0 = 0; c0 < 256; c0 += 64) {
      tmem_wait_ld();
      reg_fence32(v0);
      tmem_ld32_issue(taddr + c0 + 32, v1);
      scatter_add_32x32(p, stage, v0, c.wgt, tok_or_neg, ybase + c0, lane);
      tmem_wait_ld();
      reg_fence32(v1);
      if (c0 + 64 < 256) tmem_ld32_issue(taddr + c0 + 64, v0);
      scatter_add_32x32(p, stage, v1, c.wgt, tok_or_neg, ybase + c0 + 32, lane);
    }
  }
}

// STAGE = 1: SwiGLU epilogue (B = 128 gate rows | 128 up rows);  STAGE = 2: weighted scatter-add epilogue.
// Tensor maps: A, B (gate or down), B2 (up; unused in stage 2) for segment 0 and for segment 1.
template <int STAGE, bool MERGE = false>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                    const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmA1,
                    const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmC1,
                    const TcParams p) {
  extern __shared__ unsigned char smem_dyn[];
  pdl_grid_wait();
  __shared__ int32_t s_tb[2 * (kMaxExperts + 2)], s_ro[2 * (kMaxExperts + 2)];
  __shared__ __align__(8) uint64_t s_bar[2 * STAGES + 4];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ __align__(16) float s_epi[4 * 32 * kEpiStride];   // per epilogue warp: 32 rows being turned around
  __shared__ int32_t s_dl_dst[STAGE == 1 ? 4 * kDstList : 1];
  __shared__ uint8_t s_dl_row[STAGE == 1 ? 4 * kDstList : 1];
  __shared__ float s_dl_w[(STAGE == 1 && MERGE) ? 4 * kDstList : 1];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = (smem_u32(smem_dyn) + 1023u) & ~1023u;   // 1024-byte aligned for the swizzle
  const uint32_t bar0 = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };

  for (int sg = 0; sg < p.nseg; ++sg) {
    const Seg &S = p.seg[sg];
    int32_t *tb = s_tb + sg * (kMaxExperts + 2), *ro = s_ro + sg * (kMaxExperts + 2);
    if (S.tile_base) {
      for (int i = threadIdx.x; i <= S.G; i += blockDim.x) {
        tb[i] = S.tile_base[i];
        ro[i] = S.row_offsets[i];
      }
    } else if (threadIdx.x == 0) {
      tb[0] = 0; tb[1] = (S.single_rows + kTileM - 1) / kTileM;
      ro[0] = 0; ro[1] = S.single_rows;
    }
  }
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar(a), 1);
      mbar_init(acce_bar(a), 128);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem;
  volatile int *abort_flag = &s_abort;

  TileWalker walk;
  walk.tb = s_tb; walk.ro = s_ro; walk.nseg = p.nseg;
  walk.nt0 = p.seg[0].nt; walk.nt1 = p.seg[1].nt;
  walk.mo0 = p.seg[0].m_outer; walk.mo1 = p.seg[1].m_outer;
  walk.G0 = p.seg[0].tile_base ? p.seg[0].G : 1; walk.G1 = p.seg[1].tile_base ? p.seg[1].G : 1;
  walk.init();
  const int total = walk.total();
  const int kb0 = p.seg[0].kb, kb1 = p.seg[1].kb;

  if (warp == 0) {
    // ---------------- producer: TMA into the ring ----------------
    if (lane == 0) {
      const uint64_t w_policy = l2_policy_evict_first();
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      for (int tile = blockIdx.x; tile < total && alive; tile += gridDim.x) {
        const TileInfo t = walk.at(tile);
        const Seg &S = p.seg[t.seg];
        const CUtensorMap *mA = t.seg ? &tmA1 : &tmA0, *mB = t.seg ? &tmB1 : &tmB0, *mC = t.seg ? &tmC1 : &tmC0;
        const int a_row0 = t.prow0;
        const int b_row = t.g * S.b_group_rows + t.n_idx * (STAGE == 1 ? 128 : 256);
        for (int kb = 0; kb < S.kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.wait_ns)) { alive = false; break; }
          const uint32_t sa = ring + stage * STAGE_BYTES, sb = sa + A_BYTES;
          mbar_arrive_expect_tx(full_bar(stage), STAGE_BYTES);
          tma_load_2d(sa, mA, kb * BK, a_row0, full_bar(stage));
          if (STAGE == 1) {
            tma_load_2d_hint(sb, mB, kb * BK, b_row, full_bar(stage), w_policy);
            tma_load_2d_hint(sb + B_BYTES / 2, mC, kb * BK, b_row, full_bar(stage), w_policy);
          } else {
            tma_load_2d_hint(sb, mB, kb * BK, b_row, full_bar(stage), w_policy);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool alive = true;
      for (int tile = blockIdx.x; tile < total && alive; tile += gridDim.x) {
        const int nkb = walk.seg_of(tile) ? kb1 : kb0;   // all the issuer needs to know about the tile
        if (!mbar_wait(acce_bar(acc), acc_phase ^ 1u, abort_flag, p.wait_ns)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * ACC_COLS;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.wait_ns)) { alive = false; break; }
          tc_fence_after();
          const uint32_t sa = ring + stage * STAGE_BYTES, sb = sa + A_BYTES;
          const uint64_t da = umma_desc(sa), db = umma_desc(sb);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16(d_tmem, da + 2u * k, db + 2u * k, (kb | k) != 0 ? 1u : 0u);
          umma_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        umma_commit(accf_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue: TMEM -> registers -> global ----------------
    const int quarter = warp & 3;               // the TMEM lanes this warp may read
    const int r = quarter * 32 + lane;          // row of the tile
    if (STAGE == 1 && p.zero_vec4 > 0) {
      // clear this CTA's slice of y while the first tile's MMAs are in flight
      const int et = (warp - 2) * 32 + lane;    // 0..127
      const int64_t per = (p.zero_vec4 + gridDim.x - 1) / gridDim.x;
      const int64_t lo = per * blockIdx.x, hi = min(p.zero_vec4, lo + per);
      const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int64_t i = lo + et; i < hi; i += 128) p.zero_ptr[i] = z;
    }
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x) {
      const TileInfo t = walk.at(tile);
      const Seg &S = p.seg[t.seg];
      const DstList dl{s_dl_dst + (STAGE == 1 ? (warp - 2) * kDstList : 0), s_dl_row + (STAGE == 1 ? (warp - 2) * kDstList : 0),
                       s_dl_w + ((STAGE == 1 && MERGE) ? (warp - 2) * kDstList : 0)};
      const RowCtx c = prepare_row<STAGE, MERGE>(p, S, t, r, dl);
      if (!mbar_wait(accf_bar(acc), acc_phase, abort_flag, p.wait_ns)) break;
      tc_fence_after();
      epilogue_tile<STAGE, MERGE>(p, S, t, c, tmem_base + acc * ACC_COLS + ((uint32_t)(quarter * 32) << 16),
                           s_epi + (warp - 2) * 32 * kEpiStride, dl);
      tc_fence_before();
      mbar_arrive(acce_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (s_abort) {
    timeout_record_and_drain(&p.plan->status);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// =====================================================================================================
// CTA-pair variant: two CTAs of a cluster (two SMs) share one 256 x 256 tile.  Each CTA stages its own 128
// rows of A and its own 128-row half of B (the leader: gate rows / first half of W_down; the peer: up rows /
// second half), so a pair moves 64 KB per k-block where two independent CTAs would move 96 KB, and each
// SM's shared memory serves half the operand reads.  One thread of the leader issues
// tcgen05.mma.cta_group::2 (M = 256: rows 0-127 accumulate in the leader's TMEM, rows 128-255 in the
// peer's); completion is broadcast to both CTAs' barriers with tcgen05.commit ... multicast::cluster.
// Both CTAs' TMA loads report their bytes to the leader's "full" barrier; both CTAs' epilogues release
// the leader's "accumulator empty" barrier.  A group with an odd number of 128-row tiles ends with a pair
// whose peer half has no rows: it is computed and dropped.
// =====================================================================================================
constexpr int STAGES2 = 6;
constexpr uint32_t HALF_BYTES = kTileM * BK * 2;            // 16 KB: A tile, and one CTA's half of B
constexpr uint32_t STAGE2_BYTES = 2 * HALF_BYTES;           // per CTA
constexpr uint32_t kIdescPair = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of `local_addr` in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// tile load whose completion bytes are reported to a barrier that may live in the peer CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y,
                                                 uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(cluster_bar)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdescPair), "r"(accumulate)
      : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}

// Pair tiles are numbered segment by segment, group by group; inside a group the pairs of one n-tile
// run fastest.  CTA `rank` of the pair owns m-tile 2*pair + rank of the group.
struct PairWalker {
  const int32_t *tb, *ro, *pb;   // [2][kMaxExperts + 2] each: m-tile prefix, row offsets, pair prefix
  int nt0, nt1, G0, G1, mo0, mo1, nseg;   // per segment (scalars: indexed arrays would live in local memory)
  int seg, g;
  int tiles0;                    // pair tiles of segment 0
  __device__ void init() {
    seg = 0; g = 0;
    tiles0 = pb[G0] * nt0;
  }
  __device__ int total() const { return tiles0 + (nseg > 1 ? pb[(kMaxExperts + 2) + G1] * nt1 : 0); }
  __device__ int seg_of(int tile) const { return (nseg > 1 && tile >= tiles0) ? 1 : 0; }
  __device__ TileInfo at(int tile, int rank) {
    if (seg == 0 && nseg > 1 && tile >= tiles0) {
      seg = 1;
      g = 0;
    }
    const int o = seg * (kMaxExperts + 2);
    const int32_t *b = tb + o, *r = ro + o, *q = pb + o;
    const int n_t = seg ? nt1 : nt0, Gs = seg ? G1 : G0, m_out = seg ? mo1 : mo0;
    const int local_seg = tile - (seg ? tiles0 : 0);
    while (g + 1 < Gs && local_seg >= q[g + 1] * n_t) ++g;
    TileInfo t;
    const int np = q[g + 1] - q[g];
    const int local = local_seg - q[g] * n_t;
    t.seg = seg;
    t.g = g;
    if (m_out) {
      const int pr = local / n_t;
      t.n_idx = local - pr * n_t;
      t.m_idx = 2 * pr + rank;
    } else {
      t.n_idx = local / np;
      t.m_idx = 2 * (local - t.n_idx * np) + rank;
    }
    t.prow0 = (b[g] + t.m_idx) * kTileM;
    t.urow0 = r[g] + t.m_idx * kTileM;
    t.valid = t.m_idx < b[g + 1] - b[g] ? min(kTileM, r[g + 1] - t.urow0) : 0;
    return t;
  }
};

// A ring stage holds KSUB k-blocks (KSUB x 32 KB per CTA): with KSUB = 2 the barrier round trips, the producer's
// wake-ups and the issuer's waits happen once per 128 columns of K instead of once per 64.
template <int STAGE, bool MERGE = false, int NST = STAGES2, int KSUB = 1>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
grouped_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                         const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmA1,
                         const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmC1,
                         const TcParams p) {
  extern __shared__ unsigned char smem_dyn[];
  pdl_grid_wait();
  __shared__ int32_t s_tb[2 * (kMaxExperts + 2)], s_ro[2 * (kMaxExperts + 2)], s_pb[2 * (kMaxExperts + 2)];
  __shared__ __align__(8) uint64_t s_bar[2 * NST + 4];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ __align__(16) float s_epi[4 * 32 * kEpiStride];   // per epilogue warp: 32 rows being turned around
  __shared__ int32_t s_dl_dst[STAGE == 1 ? 4 * kDstList : 1];
  __shared__ uint8_t s_dl_row[STAGE == 1 ? 4 * kDstList : 1];
  __shared__ float s_dl_w[(STAGE == 1 && MERGE) ? 4 * kDstList : 1];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader (issues the MMAs), 1 = peer
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const uint32_t ring = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const uint32_t bar0 = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (NST + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * NST + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * NST + 2 + a); };

  for (int sg = 0; sg < p.nseg; ++sg) {
    const Seg &S = p.seg[sg];
    int32_t *tb = s_tb + sg * (kMaxExperts + 2), *ro = s_ro + sg * (kMaxExperts + 2);
    if (S.tile_base) {
      for (int i = threadIdx.x; i <= S.G; i += blockDim.x) {
        tb[i] = S.tile_base[i];
        ro[i] = S.row_offsets[i];
      }
    } else if (threadIdx.x == 0) {
      tb[0] = 0; tb[1] = (S.single_rows + kTileM - 1) / kTileM;
      ro[0] = 0; ro[1] = S.single_rows;
    }
  }
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < NST; ++s) {
      mbar_init(full_bar(s), 1);      // the leader's expect_tx arrival; bytes come from both CTAs
      mbar_init(empty_bar(s), 1);     // one commit (broadcast to both CTAs)
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar(a), 1);      // one commit (broadcast)
      mbar_init(acce_bar(a), 256);    // the epilogue threads of both CTAs
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (warp == 0 && lane < p.nseg) {   // pair prefix per group: ceil(m-tiles / 2)
    const int sg = lane, o = sg * (kMaxExperts + 2);
    const int G = p.seg[sg].tile_base ? p.seg[sg].G : 1;
    int acc = 0;
    for (int g = 0; g < G; ++g) {
      s_pb[o + g] = acc;
      acc += (s_tb[o + g + 1] - s_tb[o + g] + 1) >> 1;
    }
    s_pb[o + G] = acc;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                 // both CTAs' barriers exist before anything is signalled across
  tc_fence_after();
  const uint32_t tmem_base = s_tmem;
  volatile int *abort_flag = &s_abort;

  PairWalker walk;
  walk.tb = s_tb; walk.ro = s_ro; walk.pb = s_pb; walk.nseg = p.nseg;
  walk.nt0 = p.seg[0].nt; walk.nt1 = p.seg[1].nt;
  walk.mo0 = p.seg[0].m_outer; walk.mo1 = p.seg[1].m_outer;
  walk.G0 = p.seg[0].tile_base ? p.seg[0].G : 1; walk.G1 = p.seg[1].tile_base ? p.seg[1].G : 1;
  walk.init();
  const int total = walk.total();
  const int kb0 = p.seg[0].kb, kb1 = p.seg[1].kb;

  if (warp == 0) {
    // ---------------- producer (both CTAs): own A rows and own half of B ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      for (int tile = pair_id; tile < total && alive; tile += n_pairs) {
        const TileInfo t = walk.at(tile, rank);
        const Seg &S = p.seg[t.seg];
        const CUtensorMap *mA = t.seg ? &tmA1 : &tmA0;
        const CUtensorMap *mB;
        int b_row;
        // a pair half without a tile reads rows far outside the tensor: TMA fills them with zeros
        const int a_row = t.valid > 0 ? t.prow0 : 0x3fffff80;
        if (STAGE == 1) {            // leader: 128 gate rows; peer: the matching 128 up rows
          mB = rank == 0 ? (t.seg ? &tmB1 : &tmB0) : (t.seg ? &tmC1 : &tmC0);
          b_row = t.g * S.b_group_rows + t.n_idx * 128;
        } else {                     // halves of a 256-row slice of W_down
          mB = t.seg ? &tmB1 : &tmB0;
          b_row = t.g * S.b_group_rows + t.n_idx * 256 + (int)rank * 128;
        }
        for (int kb = 0; kb < S.kb; kb += KSUB) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.wait_ns)) { alive = false; break; }
          const uint32_t s0 = ring + stage * (KSUB * STAGE2_BYTES);
          const uint32_t lead_full = map_to_cta(full_bar(stage), 0);
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * KSUB * STAGE2_BYTES);
#pragma unroll
          for (int j = 0; j < KSUB; ++j) {
            tma_load_2d_pair(s0 + j * STAGE2_BYTES, mA, (kb + j) * BK, a_row, lead_full);
            tma_load_2d_pair(s0 + j * STAGE2_BYTES + HALF_BYTES, mB, (kb + j) * BK, b_row, lead_full);
          }
          if (++stage == NST) { stage = 0; phase ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader only) ----------------
    if (lane == 0 && rank == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool alive = true;
      for (int tile = pair_id; tile < total && alive; tile += n_pairs) {
        const int nkb = walk.seg_of(tile) ? kb1 : kb0;   // all the issuer needs to know about the tile
        if (!mbar_wait(acce_bar(acc), acc_phase ^ 1u, abort_flag, p.wait_ns)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * ACC_COLS;
        for (int kb = 0; kb < nkb; kb += KSUB) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.wait_ns)) { alive = false; break; }
          tc_fence_after();
          const uint32_t s0 = ring + stage * (KSUB * STAGE2_BYTES);
#pragma unroll
          for (int j = 0; j < KSUB; ++j) {
            const uint64_t da = umma_desc(s0 + j * STAGE2_BYTES), db = umma_desc(s0 + j * STAGE2_BYTES + HALF_BYTES);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
              umma_bf16_pair(d_tmem, da + 2u * k, db + 2u * k, (kb | j | k) != 0 ? 1u : 0u);
          }
          umma_commit_pair(empty_bar(stage));
          if (++stage == NST) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        umma_commit_pair(accf_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue (both CTAs, own 128 rows) ----------------
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    if (STAGE == 1 && p.zero_vec4 > 0) {
      const int et = (warp - 2) * 32 + lane;
      const int64_t per = (p.zero_vec4 + gridDim.x - 1) / gridDim.x;
      const int64_t lo = per * blockIdx.x, hi = min(p.zero_vec4, lo + per);
      const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int64_t i = lo + et; i < hi; i += 128) p.zero_ptr[i] = z;
    }
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = pair_id; tile < total; tile += n_pairs) {
      const TileInfo t = walk.at(tile, rank);
      const Seg &S = p.seg[t.seg];
      const DstList dl{s_dl_dst + (STAGE == 1 ? (warp - 2) * kDstList : 0), s_dl_row + (STAGE == 1 ? (warp - 2) * kDstList : 0),
                       s_dl_w + ((STAGE == 1 && MERGE) ? (warp - 2) * kDstList : 0)};
      const RowCtx c = prepare_row<STAGE, MERGE>(p, S, t, r, dl);
      if (!mbar_wait(accf_bar(acc), acc_phase, abort_flag, p.wait_ns)) break;
      tc_fence_after();
      epilogue_tile<STAGE, MERGE>(p, S, t, c, tmem_base + acc * ACC_COLS + ((uint32_t)(quarter * 32) << 16),
                           s_epi + (warp - 2) * 32 * kEpiStride, dl);
      tc_fence_before();
      mbar_arrive_cluster(map_to_cta(acce_bar(acc), 0));   // the leader's MMA waits for both halves
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (s_abort) timeout_record_and_drain(&p.plan->status);
  cluster_sync_all();                 // no signal may reach a CTA that has already exited
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// Copies rows idx[r] of src into consecutive rows of dst (the A operand of stage 1 in group order); a negative
// index marks a padding row, which is written as zeros (zero operands keep the tensor cores' switching power
// down for rows whose results are dropped).  One warp per row; up to eight 16-byte loads in flight per lane.
// With projection-side reuse it also clears the stage-2 rows that several paths of a token feed (stored in the
// path map as -(row + 2)), which stage 1 then fills by adding.
__global__ void __launch_bounds__(256) gather_rows_kernel(uint4 *dst, const uint4 *src, const int32_t *idx,
                                                          const int32_t *tile_base, int G, int vec_per_row,
                                                          const int32_t *pos2, int n_paths, uint4 *u, int u_vec_per_row) {
  pdl_grid_wait();
  const int rows = tile_base[G] * kTileM;
  const int warps_per_block = blockDim.x >> 5, lane = threadIdx.x & 31;
  for (int r = blockIdx.x * warps_per_block + (threadIdx.x >> 5); r < rows; r += gridDim.x * warps_per_block) {
    const int tok = idx[r];
    const uint4 *s = src + (size_t)(tok < 0 ? 0 : tok) * vec_per_row;
    uint4 *d = dst + (size_t)r * vec_per_row;
    for (int v0 = 0; v0 < vec_per_row; v0 += 256) {
      uint4 x[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int v = v0 + i * 32 + lane;
        x[i] = make_uint4(0u, 0u, 0u, 0u);
        if (v < vec_per_row && tok >= 0) x[i] = __ldg(s + v);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int v = v0 + i * 32 + lane;
        if (v < vec_per_row) d[v] = x[i];
      }
    }
  }
  if (pos2) {
    for (int q = blockIdx.x * warps_per_block + (threadIdx.x >> 5); q < n_paths; q += gridDim.x * warps_per_block) {
      const int d = pos2[q];
      if (d > -2) continue;
      uint4 *row = u + (size_t)(-d - 2) * u_vec_per_row;
      for (int v = lane; v < u_vec_per_row; v += 32) row[v] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

// Tile order of a single large group (the shared expert): when its rows [rows, k] are more than its weights
// [w_rows, k] and too many to stay in L2 across a sweep over them, the n-tiles of one m-tile run fastest, so the
// rows are read from DRAM once and the weights stay cached; otherwise the usual order.
inline int rows_outweigh(int64_t rows, int64_t w_rows, int64_t k) {
  return rows > w_rows && rows * k * 2 > ((int64_t)48 << 20);
}

constexpr size_t kSmemDyn = (size_t)STAGES * STAGE_BYTES + 1024;
static_assert((size_t)STAGES2 * STAGE2_BYTES + 1024 == kSmemDyn, "both kernels use the same ring size");

}  // namespace

// Stage 1 of the shared expert alone, with a 4-stage ring and the largest shared-memory carve-out, so that the
// routing, grouping and gather kernels running on another stream at the same time fit on the same SMs (the
// shared expert needs nothing from them).  Device-side problems go to the router's status word: the grouping
// step running beside this launch clears the layer's own word.
constexpr int kPairSub = 2;                        // k-blocks per ring stage of the stage-1 pair kernel (measured: stage 1
constexpr int kPairStages = STAGES2 / kPairSub;    // 0.5-2 % faster with three stages of 64 KB, stage 2 no faster)
constexpr int kSideStages = 4;
constexpr size_t kSmemSide = (size_t)kSideStages * STAGE2_BYTES + 1024;

pcomoe_status launch_shared_stage1_side(const pcomoe_layer *L, int32_t T, const void *h, const void *sg,
                                        const void *su, char *ws, const WsLayout &lay, cudaStream_t st, int32_t rows) {
  const pcomoe_config &c = L->cfg;
  const int H = c.hidden, Fsh = c.shared_ffn;
  if (!L->tc_ok || Fsh <= 0) return PCOMOE_ERR_UNSUPPORTED;
  DevPlan *plan = reinterpret_cast<DevPlan *>(ws + lay.plan);
  __nv_bfloat16 *Ush = reinterpret_cast<__nv_bfloat16 *>(ws + lay.u_sh);
  static PerDeviceOnce attr_once;
  auto kern = grouped_gemm_pair_kernel<1, false, kSideStages>;
  if (attr_once.first_use(L->device)) {
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemSide));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
    attr_once.done(L->device);
  }
  CUtensorMap mA, mB, mC;
  // tokens [0, rows) only: the rest of the shared expert's stage 1 rides in the main stage-1 launch
  if (!(make_map(&mA, h, (uint64_t)rows, H, kTileM) && make_map(&mB, sg, Fsh, H, 128) && make_map(&mC, su, Fsh, H, 128)))
    return PCOMOE_ERR_CUDA;
  TcParams p{};
  p.wait_ns = wait_limit_ns();
  p.K = c.top_k; p.T = T; p.y = nullptr; p.ldy = H;
  // only the status word of the plan is touched by the kernel: point it at the router's word
  p.plan = reinterpret_cast<DevPlan *>(reinterpret_cast<char *>(plan) + offsetof(DevPlan, status_router));
  Seg &S = p.seg[0];
  S.G = 1; S.single_rows = rows; S.nt = Fsh / 128; S.kb = H / BK; S.b_group_rows = 0; S.u_out = Ush; S.ldu = Fsh;
  S.m_outer = rows_outweigh(rows, 2 * Fsh, H);
  p.nseg = 1;
  PCOMOE_CUDA_TRY(launch_pdl(kern, dim3(L->sm_count & ~1), dim3(kThreads), kSmemSide, st, mA, mB, mC, mA, mB, mC, p));
  count_launch();
  return PCOMOE_OK;
}

pcomoe_status launch_ffn_tc(const pcomoe_layer *L, int32_t T, const void *h, const void *wg,
                            const void *wu, const void *wd, const void *sg, const void *su,
                            const void *sd, const pcomoe_groups *g, float *y, char *ws,
                            const WsLayout &lay, cudaStream_t st, int stages, cudaEvent_t wait_before_stage2,
                            int32_t shared_row0) {
  const pcomoe_config &c = L->cfg;
  if (!L->tc_ok) return PCOMOE_ERR_UNSUPPORTED;
  const int n = c.n_experts, H = c.hidden, F = c.ffn, Fsh = c.shared_ffn;
  DevPlan *plan = reinterpret_cast<DevPlan *>(ws + lay.plan);
  const int32_t *tb1 = reinterpret_cast<const int32_t *>(ws + lay.tile_base1);
  const int32_t *tb2 = reinterpret_cast<const int32_t *>(ws + lay.tile_base2);
  const int32_t *a1 = reinterpret_cast<const int32_t *>(ws + lay.a1_idx);
  const int32_t *prow1 = reinterpret_cast<const int32_t *>(ws + lay.path_prow1);
  const int32_t *pos2 = reinterpret_cast<const int32_t *>(ws + lay.path_pos2);
  __nv_bfloat16 *U = reinterpret_cast<__nv_bfloat16 *>(ws + lay.u);        // padded stage-2 order
  __nv_bfloat16 *Ush = reinterpret_cast<__nv_bfloat16 *>(ws + lay.u_sh);
  uint4 *Hg = reinterpret_cast<uint4 *>(ws + lay.h_gath);                   // padded stage-1 order
  const size_t pad_rows = (size_t)lay.mt_max * kTileM;
  if (Fsh == 0) stages &= ~(kStage1Shared | kStage2Shared);

  static PerDeviceOnce attr_once;
  if (attr_once.first_use(L->device)) {
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_pair_kernel<1, false, kPairStages, kPairSub>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_pair_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_pair_kernel<1, true, kPairStages, kPairSub>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    attr_once.done(L->device);
  }
  const bool pair = use_cta_pairs(L, T);
  const int grid = pair ? (L->sm_count & ~1) : L->sm_count;
  // Decode-sized batches (every group at most one 128-row tile): the tile count is known up front, and a grid that
  // divides it evenly avoids a last wave in which a handful of CTAs stream their weights alone at a fraction of the
  // HBM rate (Mixtral shape: 896 stage-1 tiles run as 7 waves of 128 CTAs instead of 6 waves of 148 plus 8 tiles).
  auto even_grid = [&](int64_t tiles) {
    if (pair || (int64_t)T * c.top_k > kTileM || tiles <= 0) return grid;
    const int64_t waves = (tiles + grid - 1) / grid;
    return (int)((tiles + waves - 1) / waves);
  };
  const int mt_sh = (T + kTileM - 1) / kTileM;
  const int grid1 = even_grid(((stages & kStage1Routed) ? (int64_t)n * (F / 128) : 0) +
                              ((stages & kStage1Shared) ? (int64_t)mt_sh * (Fsh / 128) : 0));
  const int grid2 = even_grid(((stages & kStage2Routed) ? (int64_t)n * (H / 256) : 0) +
                              ((stages & kStage2Shared) ? (int64_t)mt_sh * (H / 256) : 0));
  const bool merge = c.target_reuse != 0;
  const uint32_t down_box = pair ? 128 : 256;   // a CTA of a pair loads half of the 256-row slice of W_down

  // ---- stage 1: rows of h gathered into group order, then one launch over routed + shared tiles ----
  if (stages & (kStage1Routed | kStage1Shared)) {
    CUtensorMap mA[2], mB[2], mC[2];
    TcParams p{};
    p.wait_ns = wait_limit_ns();
    p.K = c.top_k; p.T = T; p.plan = plan; p.y = y; p.ldy = H;
    int ns = 0;
    bool ok = true;
    if (stages & kStage1Routed) {
      PCOMOE_CUDA_TRY(launch_pdl(gather_rows_kernel, dim3(L->sm_count * 8), dim3(256), 0, st, Hg,
                                 reinterpret_cast<const uint4 *>(h), a1, tb1, n, H / 8,
                                 merge ? pos2 : (const int32_t *)nullptr, (int)(T * c.top_k),
                                 reinterpret_cast<uint4 *>(U), F / 8));
      count_launch();
      ok = ok && make_map(&mA[ns], Hg, pad_rows, H, kTileM) && make_map(&mB[ns], wg, (uint64_t)n * F, H, 128) &&
           make_map(&mC[ns], wu, (uint64_t)n * F, H, 128);
      Seg &S = p.seg[ns++];
      S.tile_base = tb1; S.row_offsets = g->s1_offsets; S.G = n; S.nt = F / 128; S.kb = H / BK; S.b_group_rows = F;
      S.row_token = a1; S.path_prow1 = prow1; S.path_pos2 = pos2; S.u_out = U; S.ldu = F;
      S.path_w = merge ? reinterpret_cast<const float *>(ws + lay.path_wgt) : nullptr;
    }
    if (stages & kStage1Shared) {
      // tokens [shared_row0, T): the single-call forward runs the first tokens on its second stream
      const int32_t rows = T - shared_row0;
      ok = ok && make_map(&mA[ns], reinterpret_cast<const __nv_bfloat16 *>(h) + (size_t)shared_row0 * H, (uint64_t)rows, H, kTileM) &&
           make_map(&mB[ns], sg, Fsh, H, 128) && make_map(&mC[ns], su, Fsh, H, 128);
      Seg &S = p.seg[ns++];
      S.G = 1; S.single_rows = rows; S.nt = Fsh / 128; S.kb = H / BK; S.b_group_rows = 0;
      S.u_out = Ush + (size_t)shared_row0 * Fsh; S.ldu = Fsh;
      S.m_outer = rows_outweigh(rows, 2 * Fsh, H);
    }
    if (!ok) return PCOMOE_ERR_CUDA;
    if (ns == 1) { mA[1] = mA[0]; mB[1] = mB[0]; mC[1] = mC[0]; }
    p.nseg = ns;
    if (stages & kStage2Routed) {   // a full forward: y is cleared here, under the first tile's MMAs
      p.zero_ptr = reinterpret_cast<float4 *>(y);
      p.zero_vec4 = (int64_t)T * H / 4;
    }
    auto k3 = merge ? (pair ? grouped_gemm_pair_kernel<1, true, kPairStages, kPairSub> : grouped_gemm_kernel<1, true>)
                    : (pair ? grouped_gemm_pair_kernel<1, false, kPairStages, kPairSub> : grouped_gemm_kernel<1, false>);
    PCOMOE_CUDA_TRY(launch_pdl(k3, dim3(grid1), dim3(kThreads), kSmemDyn, st, mA[0], mB[0], mC[0], mA[1], mB[1], mC[1], p));
    count_launch();
  }

  // ---- stage 2: one launch over routed + shared tiles, accumulating into y ----
  if (wait_before_stage2) PCOMOE_CUDA_TRY(cudaStreamWaitEvent(st, wait_before_stage2, 0));
  if (stages & (kStage2Routed | kStage2Shared)) {
    CUtensorMap mA[2], mB[2];
    TcParams p{};
    p.wait_ns = wait_limit_ns();
    p.K = c.top_k; p.T = T; p.plan = plan; p.y = y; p.ldy = H;
    int ns = 0;
    bool ok = true;
    if (stages & kStage2Routed) {
      if (!(stages & (kStage1Routed | kStage1Shared))) {   // stage 2 on its own: clear y first
        PCOMOE_CUDA_TRY(cudaMemsetAsync(y, 0, sizeof(float) * (size_t)T * H, st));
        count_launch();
      }
      ok = ok && make_map(&mA[ns], U, pad_rows, F, kTileM) && make_map(&mB[ns], wd, (uint64_t)n * H, F, down_box);
      Seg &S = p.seg[ns++];
      S.tile_base = tb2; S.row_offsets = g->s2_offsets; S.G = n; S.nt = H / 256; S.kb = F / BK; S.b_group_rows = H;
      S.s2_token = g->s2_token; S.s2_w = g->s2_w;
    }
    if (stages & kStage2Shared) {
      ok = ok && make_map(&mA[ns], Ush, (uint64_t)lay.t_pad, Fsh, kTileM) && make_map(&mB[ns], sd, H, Fsh, down_box);
      Seg &S = p.seg[ns++];
      S.G = 1; S.single_rows = T; S.nt = H / 256; S.kb = Fsh / BK; S.b_group_rows = 0;
      S.m_outer = rows_outweigh(T, H, Fsh);
    }
    if (!ok) return PCOMOE_ERR_CUDA;
    if (ns == 1) { mA[1] = mA[0]; mB[1] = mB[0]; }
    p.nseg = ns;
    PCOMOE_CUDA_TRY(launch_pdl(pair ? grouped_gemm_pair_kernel<2> : grouped_gemm_kernel<2>, dim3(grid2), dim3(kThreads),
                               kSmemDyn, st, mA[0], mB[0], mB[0], mA[1], mB[1], mB[1], p));
    count_launch();
  }
  PCOMOE_CUDA_TRY(cudaGetLastError());
  return PCOMOE_OK;
}

}  // namespace pcomoe
