// K1: compatibility-aware path routing.  One warp per token.
//
// For every active path a = (i,j) the warp evaluates the score of Sec. 4.2,
//     s_a = (z[i] + b_ij) + lambda * u[j],
// with three separately rounded fp32 operations, keeps the K best under the total order
// (score descending, flat id ascending) - the TopK of Sec. 4.3 over the active set only -
// and turns the selected scores into path weights with a softmax.  The selection first filters the
// paths with a warp-wide threshold and ranks the few survivors; heavy ties use per-lane sorted lists.
#include <cfloat>

#include "common.cuh"

namespace pcomoe {

struct RouteParams {
  const ActiveEntry *table;  // [A], sorted by flat id, so table order == flat-id order
  const float *z;            // [T,n]
  const float *u;            // [T,n] (may alias z)
  int32_t *src;              // [T,K]
  int32_t *tgt;              // [T,K]
  float *w;                  // [T,K]
  int32_t T, n, K, A;
  float lambda, scale;
  int32_t norm_topk;
  int32_t table_in_smem;
  int32_t cache_scores;      // pass 1 keeps the scores in shared memory for pass 2
};

// A NaN or infinite score takes the path out of the token's active set: it becomes -inf, which ranks after every
// finite score and is never written out as a selection (a token with fewer than K finite scores gets -1 ids and
// weight 0 in the ranks it cannot fill; the grouping step skips such paths and reports PCOMOE_ERR_INDEX).
__device__ __forceinline__ float drop_non_finite(float s) { return fabsf(s) <= FLT_MAX ? s : -INFINITY; }

__device__ __forceinline__ float path_score(const ActiveEntry e, const float *zs, const float *us,
                                            float lambda) {
  float a = __fadd_rn(zs[e.src], e.bias);
  float b = __fmul_rn(lambda, us[e.tgt]);
  return drop_non_finite(__fadd_rn(__fadd_rn(a, b), 0.0f));  // the last add turns -0 into +0
}

// true when (s1,a1) ranks before (s2,a2)
__device__ __forceinline__ bool ranks_before(float s1, int a1, float s2, int a2) {
  return s1 > s2 || (s1 == s2 && a1 < a2);
}

// Exact TopK by per-lane sorted lists: every lane keeps the best KMAX of its own entries (ties keep the
// smaller table index first, because a lane visits its entries in ascending order and only a strictly
// larger score moves up), then K rounds of a warp arg-max over the list heads pop the winners.
// Lane k returns the k-th selection.  Used when the threshold filter below finds too many candidates.
template <int KMAX>
__device__ __noinline__ void topk_by_lists(const RouteParams &p, const ActiveEntry *tab, const float *zs,
                                           const float *us, int lane, float &my_s, int &my_a) {
  float ls[KMAX];
  int la[KMAX];
#pragma unroll
  for (int i = 0; i < KMAX; ++i) {
    ls[i] = -INFINITY;
    la[i] = 0x7fffffff;
  }
  for (int a = lane; a < p.A; a += 32) {
    const float s = path_score(tab[a], zs, us, p.lambda);
    if (s > ls[KMAX - 1] || la[KMAX - 1] == 0x7fffffff) {
      ls[KMAX - 1] = s;
      la[KMAX - 1] = a;
#pragma unroll
      for (int i = KMAX - 1; i > 0; --i) {
        if (ranks_before(ls[i], la[i], ls[i - 1], la[i - 1])) {
          float ts = ls[i]; ls[i] = ls[i - 1]; ls[i - 1] = ts;
          int ta = la[i]; la[i] = la[i - 1]; la[i - 1] = ta;
        }
      }
    }
  }
  for (int k = 0; k < p.K; ++k) {
    float bs = ls[0];
    int ba = la[0];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float os = __shfl_xor_sync(0xffffffffu, bs, off);
      const int oa = __shfl_xor_sync(0xffffffffu, ba, off);
      if (ranks_before(os, oa, bs, ba)) {
        bs = os;
        ba = oa;
      }
    }
    if (la[0] == ba) {  // this lane owns the winner: pop it
#pragma unroll
      for (int i = 0; i < KMAX - 1; ++i) {
        ls[i] = ls[i + 1];
        la[i] = la[i + 1];
      }
      ls[KMAX - 1] = -INFINITY;
      la[KMAX - 1] = 0x7fffffff;
    }
    if (lane == k) {
      my_s = bs;
      my_a = ba;
    }
  }
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
  return v;
}

template <int KMAX>
__global__ void __launch_bounds__(256) route_kernel(const RouteParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_grid_wait();
  const int warps = blockDim.x >> 5;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float *zrows = reinterpret_cast<float *>(smem_raw);                 // [warps][2][n]
  float *cand_all = zrows + (size_t)warps * 2 * p.n;                  // [warps][64]: 32 scores, 32 indices
  const ActiveEntry *tab = p.table;
  if (p.table_in_smem) {
    ActiveEntry *st = reinterpret_cast<ActiveEntry *>(smem_raw + (((size_t)warps * (2 * p.n + 64) * 4 + 15) & ~size_t(15)));
    for (int a = threadIdx.x; a < p.A; a += blockDim.x) st[a] = p.table[a];
    tab = st;
    __syncthreads();
  }
  float *zs = zrows + (size_t)warp * 2 * p.n;
  float *us = zs + p.n;
  float *cand_s = cand_all + warp * 64;
  int *cand_a = reinterpret_cast<int *>(cand_s + 32);
  const int rounds = (p.A + 31) >> 5;
  // optional per-warp score cache behind the table: [warps][rounds*32]
  float *cache = nullptr;
  if (p.cache_scores) {
    size_t off = ((size_t)warps * (2 * p.n + 64) * 4 + 15) & ~size_t(15);
    if (p.table_in_smem) off += (sizeof(ActiveEntry) * (size_t)p.A + 15) & ~size_t(15);
    cache = reinterpret_cast<float *>(smem_raw + off) + (size_t)warp * rounds * 32;
  }

  for (int t = blockIdx.x * warps + warp; t < p.T; t += gridDim.x * warps) {
    __syncwarp();
    for (int e = lane; e < p.n; e += 32) {
      zs[e] = p.z[(size_t)t * p.n + e];
      us[e] = p.u[(size_t)t * p.n + e];
    }
    __syncwarp();

    // Threshold filter.  tau = the K-th largest of the 32 per-lane maxima: at least K paths score >= tau,
    // so every path of the TopK scores >= tau, and usually only a handful of paths do.  Those candidates
    // (ties with tau included) are compacted one per lane and ranked exactly; when more than 32 qualify
    // (heavy ties) the token falls back to the per-lane lists, which give the same selection.
    float m = -INFINITY;
    for (int a = lane; a < p.A; a += 32) {
      const float s = path_score(tab[a], zs, us, p.lambda);
      if (cache) cache[a] = s;
      m = fmaxf(m, s);
    }
    float tau = 0.0f;
    for (int k = 0; k < p.K; ++k) {
      tau = warp_max(m);
      const unsigned hit = __ballot_sync(0xffffffffu, m == tau);
      if (lane == __ffs(hit) - 1) m = -INFINITY;
    }
    int cnt = 0;
    for (int i = 0; i < rounds; ++i) {
      const int a = (i << 5) + lane;
      float s = 0.0f;
      bool q = false;
      if (a < p.A) {
        s = cache ? cache[a] : path_score(tab[a], zs, us, p.lambda);
        q = s >= tau;
      }
      const unsigned b = __ballot_sync(0xffffffffu, q);
      if (q) {
        const int pos = cnt + __popc(b & ((1u << lane) - 1u));
        if (pos < 32) {
          cand_s[pos] = s;
          cand_a[pos] = a;
        }
      }
      cnt += __popc(b);
    }
    __syncwarp();

    float my_s = -INFINITY;
    int my_a = 0;
    if (cnt <= 32) {
      float cs = lane < cnt ? cand_s[lane] : -INFINITY;
      int ca = lane < cnt ? cand_a[lane] : 0x7fffffff;
      for (int k = 0; k < p.K; ++k) {
        float bs = cs;
        int ba = ca;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          const float os = __shfl_xor_sync(0xffffffffu, bs, off);
          const int oa = __shfl_xor_sync(0xffffffffu, ba, off);
          if (ranks_before(os, oa, bs, ba)) {
            bs = os;
            ba = oa;
          }
        }
        if (ca == ba) {
          cs = -INFINITY;
          ca = 0x7fffffff;
        }
        if (lane == k) {
          my_s = bs;
          my_a = ba;
        }
      }
    } else {
      topk_by_lists<KMAX>(p, tab, zs, us, lane, my_s, my_a);
    }

    const float s0 = __shfl_sync(0xffffffffu, my_s, 0);
    const bool live = lane < p.K && my_s > -INFINITY && (unsigned)my_a < (unsigned)p.A;
    float e = live ? expf(my_s - s0) : 0.0f;
    float den;
    if (p.norm_topk) {
      den = e;
    } else {
      den = 0.0f;
      for (int a = lane; a < p.A; a += 32) den += expf(path_score(tab[a], zs, us, p.lambda) - s0);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
    if (lane < p.K) {
      const size_t o = (size_t)t * p.K + lane;
      if (live) {
        const ActiveEntry en = tab[my_a];
        p.src[o] = en.src;
        p.tgt[o] = en.tgt;
        p.w[o] = e / den * p.scale;
      } else {   // no finite score left for this rank
        p.src[o] = -1;
        p.tgt[o] = -1;
        p.w[o] = 0.0f;
      }
    }
  }
}


// The same selection with fewer instructions per path, used when the expanded table and a per-warp score
// cache fit in shared memory.  Table entries are expanded to 16 bytes (byte offsets of z[src] and lambda*u[tgt]
// inside the warp's row buffer, and the bias), pass 1 keeps every score, pass 2 scans the cached scores four at
// a time and appends the few that reach the threshold to the candidate list, and the candidates are ranked by
// counting.  The result is the one the kernel above gives, bit for bit.
struct FastEntry {
  uint32_t z_off, u_off;   // byte offsets into the warp's [z | lambda*u] row buffer
  float bias;
  uint32_t pad;
};

template <int KMAX>
__global__ void __launch_bounds__(256) route_fast_kernel(const RouteParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_grid_wait();
  const int warps = blockDim.x >> 5;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int A = p.A, A128 = (A + 127) & ~127;
  float *cache = reinterpret_cast<float *>(smem_raw) + (size_t)warp * A128;          // [warps][A128]
  FastEntry *st = reinterpret_cast<FastEntry *>(smem_raw + (size_t)warps * A128 * 4);   // [A]
  float *rows = reinterpret_cast<float *>(st + A) + (size_t)warp * 2 * p.n;            // [warps][2][n]
  float *cand_s = reinterpret_cast<float *>(st + A) + (size_t)warps * 2 * p.n + warp * 68;   // [warps][68]
  int *cand_a = reinterpret_cast<int *>(cand_s + 32);
  int *cand_n = cand_a + 32;
  for (int a = threadIdx.x; a < A; a += blockDim.x) {
    const ActiveEntry e = p.table[a];
    FastEntry f;
    f.z_off = 4u * e.src;
    f.u_off = 4u * (p.n + e.tgt);
    f.bias = e.bias;
    f.pad = 0;
    st[a] = f;
  }
  for (int a = A + lane; a < A128; a += 32) cache[a] = -INFINITY;   // the tail of the last group of four
  __syncthreads();
  const unsigned char *rb = reinterpret_cast<const unsigned char *>(rows);
  const uint4 *st4 = reinterpret_cast<const uint4 *>(st);

  for (int t = blockIdx.x * warps + warp; t < p.T; t += gridDim.x * warps) {
    __syncwarp();
    for (int e = lane; e < p.n; e += 32) {
      rows[e] = p.z[(size_t)t * p.n + e];
      rows[p.n + e] = __fmul_rn(p.lambda, p.u[(size_t)t * p.n + e]);
    }
    if (lane == 0) *cand_n = 0;
    __syncwarp();

    // pass 1: every score once, kept in the cache; per-lane maxima
    float m = -INFINITY;
#pragma unroll 4
    for (int a = lane; a < A; a += 32) {
      const uint4 e = st4[a];
      const float zi = *reinterpret_cast<const float *>(rb + e.x);
      const float uj = *reinterpret_cast<const float *>(rb + e.y);
      const float s = drop_non_finite(__fadd_rn(__fadd_rn(zi, __uint_as_float(e.z)), uj));
      cache[a] = s;
      m = fmaxf(m, s);
    }
    // tau = the K-th largest lane maximum: at least K paths score >= tau, so the TopK all do
    float tau = 0.0f;
    for (int k = 0; k < p.K; ++k) {
      tau = warp_max(m);
      const unsigned hit = __ballot_sync(0xffffffffu, m == tau);
      if (lane == __ffs(hit) - 1) m = -INFINITY;
    }
    __syncwarp();
    // pass 2: four cached scores per load; the rare ones that reach tau join the candidate list
    const float4 *c4 = reinterpret_cast<const float4 *>(cache);
    for (int q = lane; q < (A128 >> 2); q += 32) {
      const float4 v = c4[q];
      if (fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)) >= tau) {
        const float vs[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (vs[c] >= tau && 4 * q + c < A) {
            const int pos = atomicAdd(cand_n, 1);
            if (pos < 32) {
              cand_s[pos] = vs[c];
              cand_a[pos] = 4 * q + c;
            }
          }
        }
      }
    }
    __syncwarp();
    const int cnt = *cand_n;

    float my_s = -INFINITY;
    int my_a = 0;
    if (cnt <= 32) {
      // rank by counting: the position of a candidate is the number of candidates that rank before it
      const float cs = lane < cnt ? cand_s[lane] : -INFINITY;
      const int ca = lane < cnt ? cand_a[lane] : 0x7fffffff;
      int rank = 0;
      for (int j = 0; j < cnt; ++j) {
        const float os = __shfl_sync(0xffffffffu, cs, j);
        const int oa = __shfl_sync(0xffffffffu, ca, j);
        rank += ranks_before(os, oa, cs, ca) ? 1 : 0;
      }
      __syncwarp();
      if (lane < cnt && rank < p.K) {   // rank order onto lanes 0..K-1, through the candidate buffer
        cand_s[rank] = cs;
        cand_a[rank] = ca;
      }
      __syncwarp();
      if (lane < p.K) {
        my_s = cand_s[lane];
        my_a = cand_a[lane];
      }
    } else {
      RouteParams q = p;      // the row buffer already holds lambda*u: the lists multiply by one
      q.lambda = 1.0f;
      topk_by_lists<KMAX>(q, p.table, rows, rows + p.n, lane, my_s, my_a);
    }

    const float s0 = __shfl_sync(0xffffffffu, my_s, 0);
    const bool live = lane < p.K && my_s > -INFINITY && (unsigned)my_a < (unsigned)A;
    float e = live ? expf(my_s - s0) : 0.0f;
    float den;
    if (p.norm_topk) {
      den = e;
    } else {
      den = 0.0f;
      for (int a = lane; a < A; a += 32) den += expf(cache[a] - s0);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
    if (lane < p.K) {
      const size_t o = (size_t)t * p.K + lane;
      if (live) {
        const ActiveEntry en = p.table[my_a];
        p.src[o] = en.src;
        p.tgt[o] = en.tgt;
        p.w[o] = e / den * p.scale;
      } else {   // no finite score left for this rank
        p.src[o] = -1;
        p.tgt[o] = -1;
        p.w[o] = 0.0f;
      }
    }
  }
}

pcomoe_status launch_route(const pcomoe_layer *L, int32_t T, const float *z, const float *u,
                           int32_t *src, int32_t *tgt, float *w, cudaStream_t st) {
  const pcomoe_config &c = L->cfg;
  RouteParams p;
  p.table = L->d_table;
  p.z = z; p.u = u; p.src = src; p.tgt = tgt; p.w = w;
  p.T = T; p.n = c.n_experts; p.K = c.top_k; p.A = L->n_active;
  p.lambda = c.lambda; p.scale = c.routed_scale; p.norm_topk = c.norm_topk;
  const int threads = 256, warps = threads / 32;
  const int cap_rows = (T + warps - 1) / warps;
  // fast kernel: expanded table + per-warp score cache + row and candidate buffers in shared memory
  const size_t a128 = ((size_t)p.A + 127) & ~size_t(127);
  const size_t smem_fast = (size_t)warps * a128 * 4 + (size_t)p.A * sizeof(FastEntry) +
                           (size_t)warps * (2 * p.n + 68) * 4;
  void (*kern)(const RouteParams) = nullptr;
  size_t smem;
  if (smem_fast <= 100 * 1024) {
    smem = smem_fast;
    p.table_in_smem = 1;
    p.cache_scores = 1;
    if (p.K <= 2) kern = route_fast_kernel<2>;
    else if (p.K <= 4) kern = route_fast_kernel<4>;
    else if (p.K <= 8) kern = route_fast_kernel<8>;
    else if (p.K <= 16) kern = route_fast_kernel<16>;
    else kern = route_fast_kernel<32>;
  } else {
    smem = ((size_t)warps * (2 * p.n + 64) * 4 + 15) & ~size_t(15);
    const size_t tab_bytes = sizeof(ActiveEntry) * (size_t)p.A;
    p.table_in_smem = smem + tab_bytes <= 160 * 1024;
    if (p.table_in_smem) smem += (tab_bytes + 15) & ~size_t(15);
    const size_t cache_bytes = (size_t)warps * ((p.A + 31) / 32 * 32) * 4;
    p.cache_scores = smem + cache_bytes <= 100 * 1024;
    if (p.cache_scores) smem += cache_bytes;
    if (p.K <= 2) kern = route_kernel<2>;
    else if (p.K <= 4) kern = route_kernel<4>;
    else if (p.K <= 8) kern = route_kernel<8>;
    else if (p.K <= 16) kern = route_kernel<16>;
    else kern = route_kernel<32>;
  }
  // as many blocks as stay resident together (the token loop strides over the grid)
  int per_sm = (int)((227 * 1024) / (smem + 1024));
  per_sm = per_sm < 1 ? 1 : (per_sm > 8 ? 8 : per_sm);
  int grid = cap_rows;
  if (grid > L->sm_count * per_sm) grid = L->sm_count * per_sm;
  if (smem > 48 * 1024)
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  PCOMOE_CUDA_TRY(launch_pdl(kern, dim3(grid), dim3(threads), smem, st, p));
  count_launch();
  return PCOMOE_OK;
}

}  // namespace pcomoe
