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
#include <cuda.h>

#include "common.cuh"

namespace pcomoe {
namespace {

constexpr int BK = 64;                      // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int STAGES = 4;
constexpr uint32_t A_BYTES = kTileM * BK * 2;       // 16 KB
constexpr uint32_t B_BYTES = 256 * BK * 2;          // 32 KB
constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
constexpr uint32_t ACC_COLS = 256;                  // fp32 accumulator columns per stage
constexpr uint32_t TMEM_COLS = 512;
constexpr int kThreads = 192;
constexpr int kDstRegs = 8;                 // stage-1 epilogue keeps up to this many destinations in registers
constexpr uint64_t kWaitLimitNs = 2000000000ull;    // 2 s

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
  // stage 1: where a row's SwiGLU output goes
  const int32_t *row_token;    // token of a padded row (routed), NULL: the row is its own destination
  const int32_t *path_prow1;   // [T,K] padded stage-1 row of every path
  const int32_t *path_pos2;    // [T,K] padded stage-2 row of every path (= row of u_out to write)
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
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the CTA is giving up (this or another role timed out).
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (uint32_t it = 1; it < (1u << 30); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) break;
    }
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// K-major operand tile in shared memory, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
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
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 16 accumulator columns of this thread's TMEM lane, and the wait for them, in one statement
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// the same for two column ranges at once (gate and up halves of a stage-1 accumulator)
__device__ __forceinline__ void tmem_ld16x2(uint32_t ta, uint32_t tb, float *a, float *b) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%32];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%33];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(ta), "r"(tb)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    a[i] = __uint_as_float(r[i]);
    b[i] = __uint_as_float(r[16 + i]);
  }
}

__device__ __forceinline__ void red_add_v4(float *addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
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
  int nt[2], G[2], nseg;
  int seg, g, seg_first;       // current segment, group, and the first tile id of the segment
  __device__ int seg_tiles(int s) const { return tb[s * (kMaxExperts + 2) + G[s]] * nt[s]; }
  __device__ int total() const {
    int t = 0;
    for (int s = 0; s < nseg; ++s) t += seg_tiles(s);
    return t;
  }
  __device__ TileInfo at(int tile) {
    while (seg + 1 < nseg && tile >= seg_first + seg_tiles(seg)) {
      seg_first += seg_tiles(seg);
      ++seg;
      g = 0;
    }
    const int32_t *b = tb + seg * (kMaxExperts + 2), *r = ro + seg * (kMaxExperts + 2);
    const int n_t = nt[seg], local_seg = tile - seg_first;
    while (g + 1 < G[seg] && local_seg >= b[g + 1] * n_t) ++g;
    TileInfo t;
    const int mt = b[g + 1] - b[g];
    const int local = local_seg - b[g] * n_t;
    t.seg = seg;
    t.g = g;
    t.n_idx = local / mt;
    t.m_idx = local - t.n_idx * mt;
    t.prow0 = (b[g] + t.m_idx) * kTileM;
    t.urow0 = r[g] + t.m_idx * kTileM;
    t.valid = min(kTileM, r[g + 1] - t.urow0);
    return t;
  }
};

__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.0f + __expf(-g)) * u; }

// STAGE = 1: SwiGLU epilogue (B = 128 gate rows | 128 up rows);  STAGE = 2: weighted scatter-add epilogue.
// Tensor maps: A, B (gate or down), B2 (up; unused in stage 2) for segment 0 and for segment 1.
template <int STAGE>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                    const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmA1,
                    const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmC1,
                    const TcParams p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ int32_t s_tb[2 * (kMaxExperts + 2)], s_ro[2 * (kMaxExperts + 2)];
  __shared__ __align__(8) uint64_t s_bar[2 * STAGES + 4];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

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
  for (int sg = 0; sg < 2; ++sg) {
    walk.nt[sg] = p.seg[sg].nt;
    walk.G[sg] = p.seg[sg].tile_base ? p.seg[sg].G : 1;
  }
  walk.seg = 0; walk.g = 0; walk.seg_first = 0;
  const int total = walk.total();

  if (warp == 0) {
    // ---------------- producer: TMA into the ring ----------------
    if (lane == 0) {
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
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { alive = false; break; }
          const uint32_t sa = ring + stage * STAGE_BYTES, sb = sa + A_BYTES;
          mbar_arrive_expect_tx(full_bar(stage), STAGE_BYTES);
          tma_load_2d(sa, mA, kb * BK, a_row0, full_bar(stage));
          if (STAGE == 1) {
            tma_load_2d(sb, mB, kb * BK, b_row, full_bar(stage));
            tma_load_2d(sb + B_BYTES / 2, mC, kb * BK, b_row, full_bar(stage));
          } else {
            tma_load_2d(sb, mB, kb * BK, b_row, full_bar(stage));
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
        const TileInfo t = walk.at(tile);
        const int nkb = p.seg[t.seg].kb;
        if (!mbar_wait(acce_bar(acc), acc_phase ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * ACC_COLS;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { alive = false; break; }
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
      const bool valid = r < t.valid;
      // destinations are looked up before the wait so the loads overlap the MMAs
      int token = 0;
      float wgt = 0.0f;
      int my_prow = t.prow0 + r;
      if (STAGE == 1) {
        if (valid && S.row_token) token = S.row_token[my_prow];
      } else if (valid) {
        const int urow = t.urow0 + r;
        token = S.s2_token ? S.s2_token[urow] : urow;
        wgt = S.s2_w ? S.s2_w[urow] : 1.0f;
      }
      bool ok = valid && (unsigned)token < (unsigned)p.T;
      if (valid && !ok) atomicCAS(&p.plan->status, 0, PCOMOE_ERR_INDEX);
      // stage 1, routed rows: the stage-2 rows this (token, source) slot feeds, one per path that reuses it
      int dst[kDstRegs];
      int nd = 0;
      const bool dst_in_regs = p.K <= kDstRegs;
      if (STAGE == 1 && ok && S.row_token && dst_in_regs) {
#pragma unroll
        for (int k = 0; k < kDstRegs; ++k) {
          if (k < p.K && S.path_prow1[(size_t)token * p.K + k] == my_prow) {
            const int d = S.path_pos2[(size_t)token * p.K + k];
#pragma unroll
            for (int j = 0; j < kDstRegs; ++j)
              if (j == nd) dst[j] = d;
            ++nd;
          }
        }
      }
      if (!mbar_wait(accf_bar(acc), acc_phase, abort_flag)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + acc * ACC_COLS + ((uint32_t)(quarter * 32) << 16);
      if (STAGE == 1) {
        const size_t col0 = (size_t)t.n_idx * 128;
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 16) {
          float gv[16], uv[16];
          tmem_ld16x2(taddr + c0, taddr + 128 + c0, gv, uv);
          if (!ok) continue;
          uint32_t packed[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            __nv_bfloat162 h2 = __floats2bfloat162_rn(silu_mul(gv[2 * i], uv[2 * i]), silu_mul(gv[2 * i + 1], uv[2 * i + 1]));
            packed[i] = *reinterpret_cast<uint32_t *>(&h2);
          }
          const uint4 lo = make_uint4(packed[0], packed[1], packed[2], packed[3]);
          const uint4 hi = make_uint4(packed[4], packed[5], packed[6], packed[7]);
          if (S.row_token && dst_in_regs) {
#pragma unroll
            for (int j = 0; j < kDstRegs; ++j) {
              if (j < nd) {
                uint4 *d4 = reinterpret_cast<uint4 *>(S.u_out + (size_t)dst[j] * S.ldu + col0 + c0);
                d4[0] = lo;
                d4[1] = hi;
              }
            }
          } else if (S.row_token) {
            // more paths per token than destination registers: look the copies up again per chunk
            for (int k = 0; k < p.K; ++k) {
              if (S.path_prow1[(size_t)token * p.K + k] != my_prow) continue;
              const int dst_row = S.path_pos2[(size_t)token * p.K + k];
              uint4 *d4 = reinterpret_cast<uint4 *>(S.u_out + (size_t)dst_row * S.ldu + col0 + c0);
              d4[0] = lo;
              d4[1] = hi;
            }
          } else {
            uint4 *d4 = reinterpret_cast<uint4 *>(S.u_out + (size_t)my_prow * S.ldu + col0 + c0);
            d4[0] = lo;
            d4[1] = hi;
          }
        }
      } else {
        float *dst = p.y + (size_t)token * p.ldy + (size_t)t.n_idx * 256;
#pragma unroll 1
        for (int c0 = 0; c0 < 256; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + c0, v);
          if (ok) {
#pragma unroll
            for (int i = 0; i < 16; i += 4)
              red_add_v4(dst + c0 + i, wgt * v[i], wgt * v[i + 1], wgt * v[i + 2], wgt * v[i + 3]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(acce_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (s_abort) {
    if (threadIdx.x == 0) atomicCAS(&p.plan->status, 0, PCOMOE_ERR_TIMEOUT);
    // let copies and MMAs already issued finish before shared memory and TMEM are given back
    const uint64_t t0 = global_ns();
    for (int it = 0; it < (1 << 22) && global_ns() - t0 < 200000ull; ++it) __nanosleep(256);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// Copies rows idx[r] of src into consecutive rows of dst (the gather-free fallback of the A operand).
__global__ void gather_rows_kernel(uint4 *dst, const uint4 *src, const int32_t *idx, const int32_t *tile_base,
                                   int G, int vec_per_row) {
  const int rows = tile_base[G] * kTileM;
  const int warps_per_block = blockDim.x >> 5;
  for (int r = blockIdx.x * warps_per_block + (threadIdx.x >> 5); r < rows; r += gridDim.x * warps_per_block) {
    const uint4 *s = src + (size_t)idx[r] * vec_per_row;
    uint4 *d = dst + (size_t)r * vec_per_row;
    for (int v = threadIdx.x & 31; v < vec_per_row; v += 32) d[v] = s[v];
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// bf16 row-major [rows, cols] tensor, boxes of box_rows x 64 columns, 128-byte swizzle
bool make_map(CUtensorMap *m, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t kSmemDyn = (size_t)STAGES * STAGE_BYTES + 1024;

}  // namespace

pcomoe_status launch_ffn_tc(const pcomoe_layer *L, int32_t T, const void *h, const void *wg,
                            const void *wu, const void *wd, const void *sg, const void *su,
                            const void *sd, const pcomoe_groups *g, float *y, char *ws,
                            const WsLayout &lay, cudaStream_t st, int stages) {
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

  static bool attr_done = false;
  if (!attr_done) {
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemDyn));
    attr_done = true;
  }
  const int grid = L->sm_count;

  // ---- stage 1: rows of h gathered into group order, then one launch over routed + shared tiles ----
  if (stages & (kStage1Routed | kStage1Shared)) {
    CUtensorMap mA[2], mB[2], mC[2];
    TcParams p{};
    p.K = c.top_k; p.T = T; p.plan = plan; p.y = y; p.ldy = H;
    int ns = 0;
    bool ok = true;
    if (stages & kStage1Routed) {
      gather_rows_kernel<<<L->sm_count * 4, 256, 0, st>>>(Hg, reinterpret_cast<const uint4 *>(h), a1, tb1, n, H / 8);
      count_launch();
      ok = ok && make_map(&mA[ns], Hg, pad_rows, H, kTileM) && make_map(&mB[ns], wg, (uint64_t)n * F, H, 128) &&
           make_map(&mC[ns], wu, (uint64_t)n * F, H, 128);
      Seg &S = p.seg[ns++];
      S.tile_base = tb1; S.row_offsets = g->s1_offsets; S.G = n; S.nt = F / 128; S.kb = H / BK; S.b_group_rows = F;
      S.row_token = a1; S.path_prow1 = prow1; S.path_pos2 = pos2; S.u_out = U; S.ldu = F;
    }
    if (stages & kStage1Shared) {
      ok = ok && make_map(&mA[ns], h, (uint64_t)T, H, kTileM) && make_map(&mB[ns], sg, Fsh, H, 128) &&
           make_map(&mC[ns], su, Fsh, H, 128);
      Seg &S = p.seg[ns++];
      S.G = 1; S.single_rows = T; S.nt = Fsh / 128; S.kb = H / BK; S.b_group_rows = 0; S.u_out = Ush; S.ldu = Fsh;
    }
    if (!ok) return PCOMOE_ERR_CUDA;
    if (ns == 1) { mA[1] = mA[0]; mB[1] = mB[0]; mC[1] = mC[0]; }
    p.nseg = ns;
    if (stages & kStage2Routed) {   // a full forward: y is cleared here, under the first tile's MMAs
      p.zero_ptr = reinterpret_cast<float4 *>(y);
      p.zero_vec4 = (int64_t)T * H / 4;
    }
    grouped_gemm_kernel<1><<<grid, kThreads, kSmemDyn, st>>>(mA[0], mB[0], mC[0], mA[1], mB[1], mC[1], p);
    count_launch();
  }

  // ---- stage 2: one launch over routed + shared tiles, accumulating into y ----
  if (stages & (kStage2Routed | kStage2Shared)) {
    CUtensorMap mA[2], mB[2];
    TcParams p{};
    p.K = c.top_k; p.T = T; p.plan = plan; p.y = y; p.ldy = H;
    int ns = 0;
    bool ok = true;
    if (stages & kStage2Routed) {
      if (!(stages & (kStage1Routed | kStage1Shared))) {   // stage 2 on its own: clear y first
        PCOMOE_CUDA_TRY(cudaMemsetAsync(y, 0, sizeof(float) * (size_t)T * H, st));
        count_launch();
      }
      ok = ok && make_map(&mA[ns], U, pad_rows, F, kTileM) && make_map(&mB[ns], wd, (uint64_t)n * H, F, 256);
      Seg &S = p.seg[ns++];
      S.tile_base = tb2; S.row_offsets = g->s2_offsets; S.G = n; S.nt = H / 256; S.kb = F / BK; S.b_group_rows = H;
      S.s2_token = g->s2_token; S.s2_w = g->s2_w;
    }
    if (stages & kStage2Shared) {
      ok = ok && make_map(&mA[ns], Ush, (uint64_t)lay.t_pad, Fsh, kTileM) && make_map(&mB[ns], sd, H, Fsh, 256);
      Seg &S = p.seg[ns++];
      S.G = 1; S.single_rows = T; S.nt = H / 256; S.kb = Fsh / BK; S.b_group_rows = 0;
    }
    if (!ok) return PCOMOE_ERR_CUDA;
    if (ns == 1) { mA[1] = mA[0]; mB[1] = mB[0]; }
    p.nseg = ns;
    grouped_gemm_kernel<2><<<grid, kThreads, kSmemDyn, st>>>(mA[0], mB[0], mB[0], mA[1], mB[1], mB[1], p);
    count_launch();
  }
  PCOMOE_CUDA_TRY(cudaGetLastError());
  return PCOMOE_OK;
}

}  // namespace pcomoe
