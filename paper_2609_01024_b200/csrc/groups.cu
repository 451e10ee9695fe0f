// K2: source grouping with reuse and target grouping (Sec. 4.3, "Source-Grouped Compute Reuse").
//
// A stable counting sort in three launches, bit-exact and free of inter-block waiting:
//   count    each block histograms the sources (first occurrences only when reuse is on) and the
//            targets of its contiguous chunk of tokens;
//   colscan  one warp per (stage, expert) turns the per-block counts into per-block offsets and a total;
//   scatter  each block derives the per-expert offsets and the 128-row tile schedule of the two GEMM stages
//            from the totals (block 0 publishes them), ranks its own paths with a bit matrix [expert][flat id in chunk]
//            (rank = set bits below mine) and writes every output at its final position.
// Orders are canonical: stage-1 rows by (source, token) - or (source, flat path id) without
// reuse - and stage-2 rows by (target, flat path id).
#include "common.cuh"

namespace pcomoe {

struct GroupParams {
  const int32_t *src;   // [T,K]
  const int32_t *tgt;   // [T,K]
  const float *w;       // [T,K]
  pcomoe_groups g;
  DevPlan *plan;
  int32_t *tile_base1, *tile_base2;   // [n+1]
  int32_t *col_tot;                   // [2][n] rows per (stage, expert)
  int32_t *blk_cnt;                   // [2][n][NB]: per-block counts, turned into per-block offsets by the scan
  int32_t *a1_idx;                    // token of every padded stage-1 row
  int32_t *path_prow1, *path_pos2;    // [T,K] padded stage-1 / stage-2 row of every path
  float *path_wgt;                    // [T,K] copy of the path weights (projection-side reuse only)
  int32_t T, n, K, dedup, chunk, nb;
  int32_t tgt_reuse;                  // 1: stage-2 rows are unique (token, target) pairs
};

__device__ __forceinline__ void flag_error(DevPlan *plan, int code) { atomicCAS(&plan->status, 0, code); }

// Loads the block's chunk of path sources / targets into shared memory; returns tokens in chunk.
__device__ __forceinline__ int stage_chunk(const GroupParams &p, int32_t *ssrc, int32_t *stgt) {
  const int t0 = blockIdx.x * p.chunk;
  const int nt = min(p.chunk, p.T - t0);
  const size_t base = (size_t)t0 * p.K;
  for (int x = threadIdx.x; x < nt * p.K; x += blockDim.x) {
    int s = p.src[base + x], t = p.tgt[base + x];
    if ((unsigned)s >= (unsigned)p.n || (unsigned)t >= (unsigned)p.n) {
      flag_error(p.plan, PCOMOE_ERR_INDEX);
      s = -1;  // the path is skipped everywhere
      t = -1;
    }
    ssrc[x] = s;
    stgt[x] = t;
  }
  return nt;
}

__device__ __forceinline__ int first_occurrence(const int32_t *row, int k, int dedup) {
  if (!dedup) return k;
  for (int k2 = 0; k2 < k; ++k2)
    if (row[k2] == row[k]) return k2;
  return k;
}

__global__ void group_count_kernel(const GroupParams p) {
  extern __shared__ int32_t sm[];
  pdl_grid_wait();
  int32_t *ssrc = sm, *stgt = sm + p.chunk * p.K;
  int32_t *h1 = stgt + p.chunk * p.K, *h2 = h1 + p.n;
  for (int e = threadIdx.x; e < 2 * p.n; e += blockDim.x) h1[e] = 0;
  const int nt = stage_chunk(p, ssrc, stgt);
  __syncthreads();
  if ((int)threadIdx.x < nt) {
    const int32_t *rs = ssrc + threadIdx.x * p.K, *rt = stgt + threadIdx.x * p.K;
    for (int k = 0; k < p.K; ++k) {
      if (rs[k] < 0) continue;
      if (first_occurrence(rs, k, p.dedup) == k) atomicAdd(&h1[rs[k]], 1);
      if (first_occurrence(rt, k, p.tgt_reuse) == k) atomicAdd(&h2[rt[k]], 1);
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 2 * p.n; e += blockDim.x) p.blk_cnt[(size_t)e * p.nb + blockIdx.x] = h1[e];
}

__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, v, off);
    if (lane >= off) v += o;
  }
  return v;
}

// One warp per (stage, expert) column: exclusive prefix of the per-block counts over the blocks, in place,
// and the column total.  A lane owns a contiguous run of blocks, so all its loads are issued at once.
__global__ void __launch_bounds__(128) group_colscan_kernel(const GroupParams p) {
  pdl_grid_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int col = blockIdx.x * (blockDim.x >> 5) + warp;
  if (col >= 2 * p.n) return;
  constexpr int kRun = 8;
  int32_t *c = p.blk_cnt + (size_t)col * p.nb;
  int carry = 0;
  for (int b0 = 0; b0 < p.nb; b0 += 32 * kRun) {
    int v[kRun];
#pragma unroll
    for (int i = 0; i < kRun; ++i) {
      const int b = b0 + lane * kRun + i;
      v[i] = b < p.nb ? c[b] : 0;
    }
    int sum = 0;
#pragma unroll
    for (int i = 0; i < kRun; ++i) sum += v[i];
    const int incl = warp_incl_scan(sum, lane);
    int run = carry + incl - sum;
#pragma unroll
    for (int i = 0; i < kRun; ++i) {
      const int b = b0 + lane * kRun + i;
      if (b < p.nb) c[b] = run;
      run += v[i];
    }
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) p.col_tot[col] = carry;
}

// Offsets over the experts and the 128-row tile schedule of one stage, from the column totals (one warp).
// Every scatter block computes them for itself; block 0 also publishes them, the statistics, and the
// padding entries of the stage-1 gather map.
__device__ __forceinline__ void expert_prefix(const GroupParams &p, int stage, const int32_t *cnt, int32_t *offs_s,
                                              int32_t *tb_s, bool publish, int lane) {
  int32_t *offs = stage == 0 ? p.g.s1_offsets : p.g.s2_offsets;
  int32_t *tb = stage == 0 ? p.tile_base1 : p.tile_base2;
  int carry_rows = 0, carry_tiles = 0, empty = 0;
  for (int e0 = 0; e0 < p.n; e0 += 32) {
    const int e = e0 + lane;
    const int c = e < p.n ? cnt[e] : 0;
    const int tl = (c + kTileM - 1) / kTileM;
    const int ir = warp_incl_scan(c, lane), it = warp_incl_scan(tl, lane);
    if (e < p.n) {
      const int o = carry_rows + ir - c, t0 = carry_tiles + it - tl;
      offs_s[e] = o;
      tb_s[e] = t0;
      if (publish) {
        offs[e] = o;
        tb[e] = t0;
      }
    }
    empty += __popc(__ballot_sync(0xffffffffu, e < p.n && c == 0));
    carry_rows += __shfl_sync(0xffffffffu, ir, 31);
    carry_tiles += __shfl_sync(0xffffffffu, it, 31);
  }
  if (publish && lane == 0) {
    offs[p.n] = carry_rows;
    tb[p.n] = carry_tiles;
    if (stage == 0) {
      p.plan->R1 = carry_rows; p.plan->mt1 = carry_tiles; p.plan->empty1 = empty;
      p.plan->T = p.T;
      p.g.stats[0] = carry_rows; p.g.stats[2] = carry_tiles; p.g.stats[4] = empty;
      p.g.stats[6] = 0; p.g.stats[7] = 0;
    } else {
      p.plan->P = carry_rows; p.plan->mt2 = carry_tiles; p.plan->empty2 = empty;
      p.g.stats[1] = carry_rows; p.g.stats[3] = carry_tiles; p.g.stats[5] = empty;
    }
  }
}

__device__ __forceinline__ int bits_below(const uint32_t *row, int idx) {
  int r = 0;
  const int word = idx >> 5;
  for (int w = 0; w < word; ++w) r += __popc(row[w]);
  return r + __popc(row[word] & ((1u << (idx & 31)) - 1u));
}

// Body of the scatter step for one block.  `cnt` = rows per (stage, expert) over the whole batch; `single` = the
// batch is this one block (its per-block offsets are zero).
__device__ __forceinline__ void scatter_block(const GroupParams &p, int32_t *sm, const int32_t *cnt, bool single) {
  const int CK = p.chunk * p.K;
  const int W = (CK + 31) >> 5;
  int32_t *ssrc = sm, *stgt = ssrc + CK, *srow = stgt + CK, *spos = srow + CK;
  int32_t *off1 = spos + CK, *off2 = off1 + p.n, *tb1 = off2 + p.n, *tb2 = tb1 + p.n;
  int32_t *bo1 = tb2 + p.n, *bo2 = bo1 + p.n;
  uint32_t *bits1 = reinterpret_cast<uint32_t *>(bo2 + p.n), *bits2 = bits1 + (size_t)p.n * W;

  for (int x = threadIdx.x; x < 2 * p.n * W; x += blockDim.x) bits1[x] = 0u;
  if (threadIdx.x < 32) {
    expert_prefix(p, 0, cnt, off1, tb1, blockIdx.x == 0, threadIdx.x);
    expert_prefix(p, 1, cnt + p.n, off2, tb2, blockIdx.x == 0, threadIdx.x);
  }
  if (p.nb > 0) {
    for (int e = threadIdx.x; e < p.n; e += blockDim.x) {
      bo1[e] = single ? 0 : p.blk_cnt[(size_t)e * p.nb + blockIdx.x];
      bo2[e] = single ? 0 : p.blk_cnt[(size_t)(p.n + e) * p.nb + blockIdx.x];
    }
  }
  const int nt = p.nb > 0 ? stage_chunk(p, ssrc, stgt) : 0;
  __syncthreads();

  // the padding rows of the source groups have no token: they are gathered as zeros (marked -1).  The blocks
  // share the groups among themselves.
  for (int e = blockIdx.x; e < p.n; e += gridDim.x) {
    const int c = cnt[e];
    const int rows = (c + kTileM - 1) / kTileM * kTileM;
    for (int x = c + threadIdx.x; x < rows; x += blockDim.x) p.a1_idx[(size_t)tb1[e] * kTileM + x] = -1;
  }

  const int tl = threadIdx.x;
  const int32_t *rs = ssrc + tl * p.K, *rt = stgt + tl * p.K;
  if (tl < nt) {
    for (int k = 0; k < p.K; ++k) {
      if (rs[k] < 0) continue;
      const int idx = tl * p.K + k;
      if (first_occurrence(rs, k, p.dedup) == k) atomicOr(&bits1[(size_t)rs[k] * W + (idx >> 5)], 1u << (idx & 31));
      if (first_occurrence(rt, k, p.tgt_reuse) == k) atomicOr(&bits2[(size_t)rt[k] * W + (idx >> 5)], 1u << (idx & 31));
    }
  }
  __syncthreads();
  if (tl >= nt) return;

  const int t = blockIdx.x * p.chunk + tl;
  int32_t *myrow = srow + tl * p.K;
  for (int k = 0; k < p.K; ++k) {
    const int s = rs[k];
    if (s < 0) continue;
    const int fk = first_occurrence(rs, k, p.dedup);
    if (fk == k) {
      const int idx = tl * p.K + k;
      const int row = off1[s] + bo1[s] + bits_below(bits1 + (size_t)s * W, idx);
      myrow[k] = row;
      p.g.s1_token[row] = t;
      p.a1_idx[(size_t)tb1[s] * kTileM + (row - off1[s])] = t;
    } else {
      myrow[k] = myrow[fk];
    }
    p.g.path_s1row[(size_t)t * p.K + k] = myrow[k];
  }
  for (int k = 0; k < p.K; ++k) {
    const int j = rt[k];
    if (j < 0) {  // a path with an out-of-range expert id feeds no row
      p.path_prow1[(size_t)t * p.K + k] = -1;
      p.path_pos2[(size_t)t * p.K + k] = -1;
      continue;
    }
    const int q = t * p.K + k;
    const int s = rs[k];
    int32_t *mypos = spos + tl * p.K;
    const int fk = first_occurrence(rt, k, p.tgt_reuse);
    if (fk == k) {
      // with projection-side reuse a row fed by several of the token's paths is marked: its position is stored
      // as -(position + 2), its weight is 1, and stage 1 adds the weighted intermediates into it
      bool merged = false;
      if (p.tgt_reuse)
        for (int k2 = k + 1; k2 < p.K; ++k2) merged |= rt[k2] == j;
      const int idx = tl * p.K + k;
      const int r2 = off2[j] + bo2[j] + bits_below(bits2 + (size_t)j * W, idx);
      p.g.s2_path[r2] = q;
      p.g.s2_s1row[r2] = myrow[k];
      p.g.s2_token[r2] = t;
      p.g.s2_w[r2] = merged ? 1.0f : p.w[q];
      const int pos = tb2[j] * kTileM + (r2 - off2[j]);
      mypos[k] = merged ? -(pos + 2) : pos;
    } else {
      mypos[k] = mypos[fk];
    }
    p.path_prow1[q] = tb1[s] * kTileM + (myrow[k] - off1[s]);
    p.path_pos2[q] = mypos[k];
    if (p.tgt_reuse) p.path_wgt[q] = p.w[q];
  }
}

__global__ void group_scatter_kernel(const GroupParams p) {
  extern __shared__ int32_t sm[];
  pdl_grid_wait();
  scatter_block(p, sm, p.col_tot, false);
}

// A batch that fits one block (decode steps): histogram, offsets and scatter in a single launch.  The block
// also clears the plan header itself, so no memset precedes it.
__global__ void group_single_block_kernel(const GroupParams p) {
  extern __shared__ int32_t sm[];
  __shared__ int32_t cnt[2 * kMaxExperts];
  pdl_grid_wait();
  if (threadIdx.x == 0) p.plan->status = 0;
  for (int e = threadIdx.x; e < 2 * p.n; e += blockDim.x) cnt[e] = 0;
  __syncthreads();
  {
    int32_t *ssrc = sm, *stgt = sm + p.chunk * p.K;
    const int nt = stage_chunk(p, ssrc, stgt);
    __syncthreads();
    if ((int)threadIdx.x < nt) {
      const int32_t *rs = ssrc + threadIdx.x * p.K, *rt = stgt + threadIdx.x * p.K;
      for (int k = 0; k < p.K; ++k) {
        if (rs[k] < 0) continue;
        if (first_occurrence(rs, k, p.dedup) == k) atomicAdd(&cnt[rs[k]], 1);
        if (first_occurrence(rt, k, p.tgt_reuse) == k) atomicAdd(&cnt[p.n + rt[k]], 1);
      }
    }
    __syncthreads();
  }
  scatter_block(p, sm, cnt, true);
}

pcomoe_status launch_groups(const pcomoe_layer *L, int32_t T, const int32_t *src, const int32_t *tgt,
                            const float *w, const pcomoe_groups *g, char *ws, const WsLayout &lay,
                            cudaStream_t st) {
  const pcomoe_config &c = L->cfg;
  GroupParams p;
  p.src = src; p.tgt = tgt; p.w = w; p.g = *g;
  p.plan = reinterpret_cast<DevPlan *>(ws + lay.plan);
  p.tile_base1 = reinterpret_cast<int32_t *>(ws + lay.tile_base1);
  p.tile_base2 = reinterpret_cast<int32_t *>(ws + lay.tile_base2);
  p.blk_cnt = reinterpret_cast<int32_t *>(ws + lay.blk_cnt);
  p.col_tot = reinterpret_cast<int32_t *>(ws + lay.col_tot);
  p.a1_idx = reinterpret_cast<int32_t *>(ws + lay.a1_idx);
  p.path_prow1 = reinterpret_cast<int32_t *>(ws + lay.path_prow1);
  p.path_pos2 = reinterpret_cast<int32_t *>(ws + lay.path_pos2);
  p.T = T; p.n = c.n_experts; p.K = c.top_k; p.dedup = c.dedup; p.chunk = group_chunk_for(L, T);
  p.tgt_reuse = c.target_reuse;
  p.path_wgt = c.target_reuse ? reinterpret_cast<float *>(ws + lay.path_wgt) : nullptr;
  p.nb = (T + p.chunk - 1) / p.chunk;

  const int CK = p.chunk * p.K, W = (CK + 31) / 32;
  const size_t smem_count = sizeof(int32_t) * ((size_t)2 * CK + 2 * p.n);
  const size_t smem_scatter = sizeof(int32_t) * ((size_t)4 * CK + 6 * p.n + (size_t)2 * p.n * W);
  if (smem_scatter > 200 * 1024) return PCOMOE_ERR_UNSUPPORTED;
  if (smem_count > 48 * 1024)
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(group_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_count));
  if (smem_scatter > 48 * 1024)
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(group_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_scatter));
  if (p.nb <= 1) {   // the whole batch in one block: one launch does everything
    if (smem_scatter > 48 * 1024)
      PCOMOE_CUDA_TRY(cudaFuncSetAttribute(group_single_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_scatter));
    PCOMOE_CUDA_TRY(launch_pdl(group_single_block_kernel, dim3(1), dim3(p.chunk), smem_scatter, st, p));
    count_launch();
    return PCOMOE_OK;
  }
  // the status word and the plan start from zero
  PCOMOE_CUDA_TRY(cudaMemsetAsync(ws + lay.plan, 0, kPlanClearBytes, st));
  PCOMOE_CUDA_TRY(launch_pdl(group_count_kernel, dim3(p.nb), dim3(p.chunk), smem_count, st, p));
  count_launch(2);
  PCOMOE_CUDA_TRY(launch_pdl(group_colscan_kernel, dim3((2 * p.n + 3) / 4), dim3(128), 0, st, p));
  PCOMOE_CUDA_TRY(launch_pdl(group_scatter_kernel, dim3(p.nb), dim3(p.chunk), smem_scatter, st, p));
  count_launch(2);
  PCOMOE_CUDA_TRY(cudaGetLastError());
  return PCOMOE_OK;
}

}  // namespace pcomoe
