// Memory-bound kernels of the pQuant layer: weight scale reduction and
// binarize-and-pack (Eq. 3, 4, 6), router (Sec. 3.3), expert sort, activation
// quantisation (Eq. 7-9), and the small gather / scale / reduce helpers of the
// backward pass.
#include "pq_kernels.cuh"

namespace pq {

ProfileSlot g_profile[KID_COUNT] = {};
long long g_launches = 0;

// ---------------------------------------------------------------------------
// K2a: partial sums of W and |W| in fp64 (Eq. 6).  Fixed grid and a fixed
// reduction tree, so the result does not depend on scheduling.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_weight_partial_sums(const float4* __restrict__ W4, long long n4, double* __restrict__ partial) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  double s = 0.0, a = 0.0;
  const long long stride = gridDim.x * 256LL;
  long long i = blockIdx.x * 256LL + threadIdx.x;
  // One conversion to fp64 per element (the conversion is the slow instruction here); |x| is taken on the double,
  // which is the same number as the double of |x|.  The order of the additions is fixed by the launch shape alone.
  auto sums = [](const float4& v, double& ts, double& ta) {
    const double d0 = (double)v.x, d1 = (double)v.y, d2 = (double)v.z, d3 = (double)v.w;
    ts = d0 + d1 + d2 + d3;
    ta = fabs(d0) + fabs(d1) + fabs(d2) + fabs(d3);
  };
  // four loads in flight per thread
  for (; i + 3 * stride < n4; i += 4 * stride) {
    const float4 v0 = __ldg(W4 + i), v1 = __ldg(W4 + i + stride), v2 = __ldg(W4 + i + 2 * stride), v3 = __ldg(W4 + i + 3 * stride);
    double s0, a0, s1, a1, s2, a2, s3, a3;
    sums(v0, s0, a0); sums(v1, s1, a1); sums(v2, s2, a2); sums(v3, s3, a3);
    s += s0 + s1;
    s += s2 + s3;
    a += a0 + a1;
    a += a2 + a3;
  }
  for (; i < n4; i += stride) {
    double s0, a0;
    sums(__ldg(W4 + i), s0, a0);
    s += s0;
    a += a0;
  }
  for (int d = 16; d > 0; d >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, d);
    a += __shfl_xor_sync(0xffffffffu, a, d);
  }
  __shared__ double sh[2][8];
  if ((threadIdx.x & 31) == 0) { sh[0][threadIdx.x >> 5] = s; sh[1][threadIdx.x >> 5] = a; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double ts = 0.0, ta = 0.0;
    for (int w = 0; w < 8; ++w) { ts += sh[0][w]; ta += sh[1][w]; }
    partial[2 * blockIdx.x] = ts;
    partial[2 * blockIdx.x + 1] = ta;
  }
}

// Every block re-reduces the (few hundred) partials in the same order, so all blocks agree on mu without
// a grid-wide barrier: thread t sums partials t, t + 256, ... (ascending), then a fixed tree over the block.
// The partials were written by the kernel before this one and the buffer is reused from call to call, so they are
// read with L2 loads (ld.global.cg): a kernel launched with programmatic stream serialisation can be resident while
// an older kernel still reads the previous call's values on the same SM, and the read-only data path gives no
// guarantee against finding those in L1.
__device__ __forceinline__ void reduce_partials(const double* partial, int nparts, double inv_count, float* mu, float* lam) {
  __shared__ double sh[2][8];
  __shared__ double fin[2];
  double s = 0.0, a = 0.0;
  for (int i = threadIdx.x; i < nparts; i += 256) { s += __ldcg(partial + 2 * i); a += __ldcg(partial + 2 * i + 1); }
  for (int d = 16; d > 0; d >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, d);
    a += __shfl_xor_sync(0xffffffffu, a, d);
  }
  if ((threadIdx.x & 31) == 0) { sh[0][threadIdx.x >> 5] = s; sh[1][threadIdx.x >> 5] = a; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double ts = 0.0, ta = 0.0;
    for (int w = 0; w < 8; ++w) { ts += sh[0][w]; ta += sh[1][w]; }
    fin[0] = ts; fin[1] = ta;
  }
  __syncthreads();
  *mu = (float)(fin[0] * inv_count);
  *lam = (float)(fin[1] * inv_count);
}

// ---------------------------------------------------------------------------
// K2b: S = Sign(W - mu) as the comparison W >= mu (Eq. 3-4); emits the packed
// words (bit j of word i <-> k = 32 i + j, 1 <-> +1; App. A) and the +-1 int8
// tile the tensor cores read.  Each thread owns 4 consecutive k.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_binarize_pack(const float4* __restrict__ W4, long long n4, const double* partial,
                                                       int nparts, double inv_count, uint32_t* __restrict__ bits,
                                                       uint32_t* __restrict__ s8x4, float* __restrict__ scales) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  float mu, lam;
  reduce_partials(partial, nparts, inv_count, &mu, &lam);
  if (blockIdx.x == 0 && threadIdx.x == 0) { scales[0] = lam; scales[1] = mu; }
  // n4 is a multiple of 8 (K % 32 == 0), so whole groups of 8 lanes stay together
  const long long n4_pad = (n4 + 31) & ~31LL;
  const long long stride = gridDim.x * 256LL;
  for (long long i0 = blockIdx.x * 256LL + threadIdx.x; i0 < n4_pad; i0 += 2 * stride) {
    float4 v[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const long long i = i0 + u * stride;
      v[u] = i < n4 ? __ldg(W4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const long long i = i0 + u * stride;
      if (i >= n4_pad) break;          // uniform over the warp: stride and n4_pad are multiples of 32
      uint32_t nib = 0;
      if (i < n4) {
        const uint32_t b0 = v[u].x >= mu, b1 = v[u].y >= mu, b2 = v[u].z >= mu, b3 = v[u].w >= mu;
        nib = b0 | (b1 << 1) | (b2 << 2) | (b3 << 3);
        // +1 -> 0x01, -1 -> 0xFF, little endian: byte j <-> k + j
        const uint32_t bytes = (b0 ? 0x01u : 0xFFu) | (b1 ? 0x0100u : 0xFF00u) | (b2 ? 0x010000u : 0xFF0000u) | (b3 ? 0x01000000u : 0xFF000000u);
        if (s8x4) s8x4[i] = bytes;
      }
      uint32_t word = nib << (4 * (threadIdx.x & 7));
      word |= __shfl_xor_sync(0xffffffffu, word, 1);
      word |= __shfl_xor_sync(0xffffffffu, word, 2);
      word |= __shfl_xor_sync(0xffffffffu, word, 4);
      if ((threadIdx.x & 7) == 0 && i < n4) bits[i >> 3] = word;
    }
  }
}

// RMSNorm fused in front of the quantiser (App. A): what every consumer of a token sees is
//   bf16( fl32( fl32(x * s_t) * g_k ) ),   s_t = fl32( 1 / sqrt(mean_k x^2 + eps) )  (mean and root in fp64, k_row_rms),
// the values a separate bf16 norm layer would have handed over.  One 16-byte piece (8 values) at a time.
__device__ __forceinline__ uint4 rms_apply(const uint4& v, float s, const uint4& g) {
  uint4 o;
  o.x = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.x), s), bf16lo(g.x)), __fmul_rn(__fmul_rn(bf16hi(v.x), s), bf16hi(g.x)));
  o.y = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.y), s), bf16lo(g.y)), __fmul_rn(__fmul_rn(bf16hi(v.y), s), bf16hi(g.y)));
  o.z = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.z), s), bf16lo(g.z)), __fmul_rn(__fmul_rn(bf16hi(v.z), s), bf16hi(g.z)));
  o.w = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.w), s), bf16lo(g.w)), __fmul_rn(__fmul_rn(bf16hi(v.w), s), bf16hi(g.w)));
  return o;
}

// s_t for every token: one warp per row, squares summed in fp64 (lane-strided pieces ascending, then the butterfly).
__global__ void __launch_bounds__(256) k_row_rms(const uint4* __restrict__ X, int T, int K, float eps, float* __restrict__ rms) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= T) return;
  const int chunks = K >> 3;
  const uint4* row = X + (long long)t * chunks;
  double ss = 0.0;
  for (int c = lane; c < chunks; c += 32) {
    const uint4 v = __ldg(row + c);
    const double d0 = bf16lo(v.x), d1 = bf16hi(v.x), d2 = bf16lo(v.y), d3 = bf16hi(v.y);
    const double d4 = bf16lo(v.z), d5 = bf16hi(v.z), d6 = bf16lo(v.w), d7 = bf16hi(v.w);
    ss += ((d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3)) + ((d4 * d4 + d5 * d5) + (d6 * d6 + d7 * d7));
  }
  for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
  if (lane == 0) rms[t] = (float)(1.0 / sqrt(ss / (double)K + (double)eps));
}

// ---------------------------------------------------------------------------
// K4a: router (Sec. 3.3).  One warp per token (or per two).  Logits in fp32 with a fixed
// summation order -- lane j owns the 8-element chunks c with c mod 32 == j,
// ascending k, fused multiply-add; lanes combined by the xor butterfly
// 16, 8, 4, 2, 1 -- so that the top-1 index is reproducible bit for bit.
// Softmax in fp32; ties go to the lowest index.  Also counts tokens per
// expert for each block of kRouterTokensPerBlock consecutive tokens.
// ---------------------------------------------------------------------------
// EMAX: compile-time bound on E (the loops over experts are unrolled to it); TPW: tokens per warp -- the warp
// walks the chunks once and applies each unpacked piece of Wr to TPW tokens.  Neither changes any token's
// arithmetic: a lane's partial sum of (token, expert) is the same chain of fused multiply-adds.
template <int EMAX, int TPW>
__global__ void __launch_bounds__(32 * kRouterTokensPerBlock / TPW, TPW >= 4 ? 2 : 1) k_router(const uint4* __restrict__ X, const uint4* __restrict__ Wr, int T, int K,
                                                                             int E, int* __restrict__ expert, float* __restrict__ gate_tok,
                                                                             float* __restrict__ probs_tok, int* __restrict__ block_counts,
                                                                             const uint4* __restrict__ norm_w, const float* __restrict__ rms) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  __shared__ int cnt[kMaxExperts];
  if (threadIdx.x < kMaxExperts) cnt[threadIdx.x] = 0;
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = K >> 3;
  const int t0 = blockIdx.x * kRouterTokensPerBlock + warp * TPW;   // this warp's first token
  if (t0 < T) {
    float acc[TPW][EMAX];
#pragma unroll
    for (int u = 0; u < TPW; ++u)
#pragma unroll
      for (int e = 0; e < EMAX; ++e) acc[u][e] = 0.f;
    const uint4* xrow[TPW];
#pragma unroll
    for (int u = 0; u < TPW; ++u) xrow[u] = X + (long long)min(t0 + u, T - 1) * chunks;   // a token past the end repeats the last one, unused
    auto fold = [&](const uint4 (&xv)[TPW], const uint4 (&wr)[EMAX]) {
      float x[TPW][8];
#pragma unroll
      for (int u = 0; u < TPW; ++u) {
        x[u][0] = bf16lo(xv[u].x); x[u][1] = bf16hi(xv[u].x); x[u][2] = bf16lo(xv[u].y); x[u][3] = bf16hi(xv[u].y);
        x[u][4] = bf16lo(xv[u].z); x[u][5] = bf16hi(xv[u].z); x[u][6] = bf16lo(xv[u].w); x[u][7] = bf16hi(xv[u].w);
      }
#pragma unroll
      for (int e = 0; e < EMAX; ++e) {
        if (e < E) {
          const uint4 wv = wr[e];
          const float w[8] = {bf16lo(wv.x), bf16hi(wv.x), bf16lo(wv.y), bf16hi(wv.y), bf16lo(wv.z), bf16hi(wv.z), bf16lo(wv.w), bf16hi(wv.w)};
#pragma unroll
          for (int u = 0; u < TPW; ++u) {
            float a = acc[u][e];
#pragma unroll
            for (int i = 0; i < 8; ++i) a = fmaf(x[u][i], w[i], a);
            acc[u][e] = a;
          }
        }
      }
    };
    // the tokens' chunks in ascending order; the next chunk of every row and this chunk's pieces of Wr are
    // requested before the current chunk is folded in
    float srow[TPW];
#pragma unroll
    for (int u = 0; u < TPW; ++u) srow[u] = norm_w ? rms[min(t0 + u, T - 1)] : 1.0f;
    auto fetch_x = [&](int u, int cc) {
      if (cc >= chunks) return make_uint4(0u, 0u, 0u, 0u);
      const uint4 v = __ldg(xrow[u] + cc);
      return norm_w ? rms_apply(v, srow[u], __ldg(norm_w + cc)) : v;      // the router sees the normalised token
    };
    int c = lane;
    uint4 xc[TPW];
#pragma unroll
    for (int u = 0; u < TPW; ++u) xc[u] = fetch_x(u, c);
    while (c < chunks) {
      const int cn = c + 32;
      uint4 xn[TPW];
#pragma unroll
      for (int u = 0; u < TPW; ++u) xn[u] = fetch_x(u, cn);
      uint4 wr[EMAX];
#pragma unroll
      for (int e = 0; e < EMAX; ++e) wr[e] = e < E ? __ldg(Wr + (long long)e * chunks + c) : make_uint4(0u, 0u, 0u, 0u);
      fold(xc, wr);
#pragma unroll
      for (int u = 0; u < TPW; ++u) xc[u] = xn[u];
      c = cn;
    }
#pragma unroll
    for (int u = 0; u < TPW; ++u) {
      const int t = t0 + u;
      if (t >= T) break;
#pragma unroll
      for (int e = 0; e < EMAX; ++e) {
        if (e < E) {
          float a = acc[u][e];
          for (int d = 16; d > 0; d >>= 1) a = a + __shfl_xor_sync(0xffffffffu, a, d);
          acc[u][e] = a;
        }
      }
      // every lane now holds all logits; lane 0 finishes the token
      int best = 0;
      float lmax = acc[u][0];
#pragma unroll
      for (int e = 1; e < EMAX; ++e)
        if (e < E && acc[u][e] > lmax) { lmax = acc[u][e]; best = e; }
      float den = 0.f;
      float pe[EMAX];
#pragma unroll
      for (int e = 0; e < EMAX; ++e) {
        pe[e] = (e < E) ? expf(acc[u][e] - lmax) : 0.f;
        den += pe[e];
      }
      const float inv = 1.0f / den;
      if (lane == 0) {
        expert[t] = best;
        atomicAdd(&cnt[best], 1);
      }
#pragma unroll
      for (int e = 0; e < EMAX; ++e) {
        if (e < E) {
          const float pr = pe[e] * inv;
          if (lane == 0) probs_tok[(long long)t * E + e] = pr;
          if (e == best && lane == 0) gate_tok[t] = pr;
        }
      }
    }
  }
  __syncthreads();
  if (threadIdx.x < E) block_counts[blockIdx.x * E + threadIdx.x] = cnt[threadIdx.x];
}

// ---------------------------------------------------------------------------
// K4b: expert offsets, per-block bases for the stable scatter, and the item
// table.  An item is the intersection of a 128-row tile of the sorted token
// order with one expert's range: {tile, expert, first row, end row} (rows
// relative to the tile).  Items are sorted by tile and therefore by expert.
// One block; the work is a few hundred integers.
// ---------------------------------------------------------------------------
// Items of one 128-row tile [r0, r1) of the sorted order: experts e0 <= e < E whose non-empty range
// [off[e], off[e+1]) meets the tile.  Returns the number of items; calls f(k, e, lo, hi) for the k-th.
template <class F>
__device__ __forceinline__ int tile_items(const int* off, int Ee, int r0, int r1, F f) {
  int n = 0;
  for (int e = 0; e < Ee; ++e) {
    const int lo = max(off[e], r0), hi = min(off[e + 1], r1);
    if (hi > lo) { f(n, e, lo, hi); ++n; }
  }
  return n;
}

__global__ void __launch_bounds__(512) k_route_scan(int T, int E, int nblocks, const int* __restrict__ block_counts,
                                                    int* __restrict__ block_base, int* __restrict__ offsets, RoutingTables rt) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  __shared__ int off[kMaxExperts + 1];
  __shared__ int total[kMaxExperts];
  __shared__ int warp_sums[16];
  __shared__ int carry_sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int Ee = E < 1 ? 1 : E;
  if (E > 1 && warp < E) {
    // exclusive scan of this expert's per-block counts, 32 blocks at a time
    int carry = 0;
    for (int b0 = 0; b0 < nblocks; b0 += 32) {
      const int b = b0 + lane;
      const int v = b < nblocks ? block_counts[b * E + warp] : 0;
      int inc = v;
      for (int d = 1; d < 32; d <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += u;
      }
      if (b < nblocks) block_base[b * E + warp] = carry + inc - v;
      carry += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) total[warp] = carry;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (E <= 1) {
      off[0] = 0; off[1] = T;
    } else {
      int run = 0;
      for (int e = 0; e < E; ++e) { off[e] = run; run += total[e]; }
      off[E] = run;
    }
    carry_sh = 0;
  }
  __syncthreads();
  if (threadIdx.x <= Ee) offsets[threadIdx.x] = off[threadIdx.x];

  // items: one thread per tile counts its items, a block-wide scan places them
  const int mtiles = (T + kTileRows - 1) / kTileRows;
  for (int base = 0; base < mtiles; base += blockDim.x) {
    const int tile = base + threadIdx.x;
    const int r0 = tile * kTileRows, r1 = min(T, r0 + kTileRows);
    const int cnt = tile < mtiles ? tile_items(off, Ee, r0, r1, [](int, int, int, int) {}) : 0;
    int inc = cnt;
    for (int d = 1; d < 32; d <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += u;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    int before = carry_sh;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    const int first = before + inc - cnt;
    if (tile < mtiles) {
      rt.tile_item_begin[tile] = first;
      tile_items(off, Ee, r0, r1, [&](int k, int e, int lo, int hi) { rt.items[first + k] = make_int4(tile, e, lo - r0, hi - r0); });
    }
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_sh = first + cnt;
    __syncthreads();
  }
  const int n_items = carry_sh;
  if (threadIdx.x == 0) { rt.tile_item_begin[mtiles] = n_items; rt.n_items[0] = n_items; }
  // first item of each expert: the first item of the tile holding its first row, plus the items of the
  // non-empty experts below it in that tile; an empty expert points at its successor's first item
  if (threadIdx.x <= Ee) {
    int e = threadIdx.x;
    while (e < Ee && off[e + 1] == off[e]) ++e;
    int idx = n_items;
    if (e < Ee) {
      const int tile = off[e] / kTileRows, r0 = tile * kTileRows;
      idx = rt.tile_item_begin[tile];   // written above by this block, ordered by the barriers of the loop
      for (int f = 0; f < e; ++f)
        if (min(off[f + 1], r0 + kTileRows) > max(off[f], r0)) ++idx;
    }
    rt.expert_item_begin[threadIdx.x] = idx;
  }
}

// ---------------------------------------------------------------------------
// K1: activation quantisation (Eq. 7-9), one warp per token.  gamma_t = 128 /
// max(amax, 1e-5) (IEEE division), q = clamp(rint(x * gamma_t), -128, 127).
// Rows are written at their sorted position p (tokens ordered by expert,
// stable): q (int8), xt = q / gamma (bf16, the backward's operand) and, with
// routing, a bf16 copy of the row itself plus its gate and probabilities.
// ---------------------------------------------------------------------------
// WPR warps share one token row.  CH > 0: every lane keeps its CH 16-byte pieces of the row in registers
// between the absmax pass and the quantising pass (rows of up to 256 * CH * WPR elements), so X is read
// once; CH = 0 reads the row twice.
template <int CH, int WPR>
__global__ void __launch_bounds__(256) k_act_quant(const uint4* __restrict__ X, int T, int K, int E, const int* __restrict__ expert,
                                                   const int* __restrict__ block_base, const int* __restrict__ offsets,
                                                   const float* __restrict__ gate_tok, const float* __restrict__ probs_tok,
                                                   uint2* __restrict__ q, uint4* __restrict__ xt, uint4* __restrict__ xs,
                                                   float* __restrict__ gamma_s, float* __restrict__ gate_s, float* __restrict__ probs_s,
                                                   int* __restrict__ perm, int* __restrict__ pos, const uint4* __restrict__ norm_w,
                                                   const float* __restrict__ rms) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  __shared__ float amax_sh[8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = warp % WPR, slot = sub * 32 + lane;   // this lane's first 16-byte piece of the row
  const int t_raw = blockIdx.x * (8 / WPR) + warp / WPR;
  const bool valid = t_raw < T;
  if (WPR == 1 && !valid) return;
  const int t = valid ? t_raw : T - 1;                  // idle warps of a shared row keep the barrier company
  const int chunks = K >> 3;
  const uint4* xrow = X + (long long)t * chunks;
  const float srow = norm_w ? rms[t] : 1.0f;
  auto fetch_x = [&](int c) {                      // with a fused RMSNorm every later step sees the normalised token
    const uint4 v = __ldg(xrow + c);
    return norm_w ? rms_apply(v, srow, __ldg(norm_w + c)) : v;
  };
  uint4 held[CH > 0 ? CH : 1];
  float amax = 0.f;
  auto fold = [&](const uint4& v) {
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.x)), fabsf(bf16hi(v.x))), fmaxf(fabsf(bf16lo(v.y)), fabsf(bf16hi(v.y)))));
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.z)), fabsf(bf16hi(v.z))), fmaxf(fabsf(bf16lo(v.w)), fabsf(bf16hi(v.w)))));
  };
  if (CH > 0) {
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int c = slot + 32 * WPR * i;
      held[i] = c < chunks ? fetch_x(c) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int i = 0; i < CH; ++i) fold(held[i]);
  } else {
    for (int c = slot; c < chunks; c += 32 * WPR) fold(fetch_x(c));
  }
  int p = t;
  if (E > 1) {
    const int e = expert[t];
    const int blk = t / kRouterTokensPerBlock, first = blk * kRouterTokensPerBlock;
    const int other = (first + lane < T) ? expert[first + lane] : -1;
    const unsigned same = __ballot_sync(0xffffffffu, other == e);
    const int rank = __popc(same & ((1u << (t - first)) - 1u));
    p = offsets[e] + block_base[blk * E + e] + rank;
  }
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  if (WPR > 1) {
    if (lane == 0) amax_sh[warp] = amax;
    __syncthreads();
    const int w0 = warp - sub;
#pragma unroll
    for (int w = 0; w < WPR; ++w) amax = fmaxf(amax, amax_sh[w0 + w]);
    if (!valid) return;
  }
  const float gamma = __fdiv_rn(kActQmax, fmaxf(amax, kActAmaxFloor));
  const float inv_gamma = __fdiv_rn(1.0f, gamma);
  if (lane == 0 && sub == 0) {
    gamma_s[p] = gamma;
    perm[p] = t;
    pos[t] = p;
    gate_s[p] = (E > 1) ? gate_tok[t] : 1.0f;
  }
  if (E > 1 && sub == 0 && lane < E) probs_s[(long long)p * E + lane] = probs_tok[(long long)t * E + lane];
  uint2* qrow = q + (long long)p * chunks;
  uint4* xtrow = xt ? xt + (long long)p * chunks : nullptr;
  uint4* xsrow = xs ? xs + (long long)p * chunks : nullptr;
  auto emit = [&](int c, const uint4& v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int qi[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float lo = __fmul_rn(bf16lo(w[j]), gamma), hi = __fmul_rn(bf16hi(w[j]), gamma);
      qi[2 * j] = max(-128, min(127, __float2int_rn(lo)));
      qi[2 * j + 1] = max(-128, min(127, __float2int_rn(hi)));
    }
    uint2 qo;
    qo.x = (qi[0] & 0xFF) | ((qi[1] & 0xFF) << 8) | ((qi[2] & 0xFF) << 16) | ((qi[3] & 0xFF) << 24);
    qo.y = (qi[4] & 0xFF) | ((qi[5] & 0xFF) << 8) | ((qi[6] & 0xFF) << 16) | ((qi[7] & 0xFF) << 24);
    qrow[c] = qo;
    if (xtrow) {
      uint4 o;
      o.x = pack_bf16x2(qi[0] * inv_gamma, qi[1] * inv_gamma);
      o.y = pack_bf16x2(qi[2] * inv_gamma, qi[3] * inv_gamma);
      o.z = pack_bf16x2(qi[4] * inv_gamma, qi[5] * inv_gamma);
      o.w = pack_bf16x2(qi[6] * inv_gamma, qi[7] * inv_gamma);
      xtrow[c] = o;
    }
    if (xsrow) xsrow[c] = v;
  };
  if (CH > 0) {
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int c = slot + 32 * WPR * i;
      if (c < chunks) emit(c, held[i]);
    }
  } else {
    for (int c = slot; c < chunks; c += 32 * WPR) emit(c, fetch_x(c));
  }
}

// dst[pos[t], :] = src[t, :]  (rows of `chunks` 16-byte pieces), one warp per row
__global__ void __launch_bounds__(256) k_scatter_rows(const uint4* __restrict__ src, uint4* __restrict__ dst, const int* __restrict__ pos,
                                                      int T, int chunks) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= T) return;
  const uint4* s = src + (long long)t * chunks;
  uint4* d = dst + (long long)pos[t] * chunks;
  for (int c = lane; c < chunks; c += 32) d[c] = __ldg(s + c);
}

// Sb[n,k] = bf16(scale_n) * S[n,k]; scale_n = beta_n (vector form) or 1
__global__ void __launch_bounds__(256) k_scaled_sign(const uint4* __restrict__ s8, uint4* __restrict__ out, const float* __restrict__ beta,
                                                     int beta_stride, int N, int K, unsigned* __restrict__ arrivals) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  // first kernel of every backward call: it also clears the arrival counter of the call's last kernel (k_finalize_scales)
  if (arrivals && blockIdx.x == 0 && threadIdx.x == 0) *arrivals = 0u;
  const long long n16 = (long long)N * K / 16;
  const int per_row = K / 16;
  for (long long i = blockIdx.x * 256LL + threadIdx.x; i < n16; i += gridDim.x * 256LL) {
    const int n = (int)(i / per_row);
    const float sc = beta_stride ? beta[n] : 1.0f;
    const uint4 v = __ldg(s8 + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint4 o[2];
    uint32_t* ow = reinterpret_cast<uint32_t*>(o);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = (float)(int8_t)(w[j] & 0xFF) * sc, b = (float)(int8_t)((w[j] >> 8) & 0xFF) * sc;
      const float c = (float)(int8_t)((w[j] >> 16) & 0xFF) * sc, d = (float)(int8_t)(w[j] >> 24) * sc;
      ow[2 * j] = pack_bf16x2(a, b);
      ow[2 * j + 1] = pack_bf16x2(c, d);
    }
    out[2 * i] = o[0];
    out[2 * i + 1] = o[1];
  }
}

// Ba[e,n,j] = bf16(alpha_n * B[e,n,j])  (vector alpha only)
__global__ void __launch_bounds__(256) k_scaled_b(const uint32_t* __restrict__ B2, uint32_t* __restrict__ out, const float* __restrict__ alpha,
                                                  int E, int N, int r) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  const long long n2 = (long long)E * N * r / 2;
  const int per_row = r / 2;
  for (long long i = blockIdx.x * 256LL + threadIdx.x; i < n2; i += gridDim.x * 256LL) {
    const int n = (int)((i / per_row) % N);
    const uint32_t v = __ldg(B2 + i);
    out[i] = pack_bf16x2(bf16lo(v) * alpha[n], bf16hi(v) * alpha[n]);
  }
}

// Feature-scale gradients from their per-tile partials, one thread per output feature:
//   dbeta_n = lam * sum_s dbeta_partial[s, n]      dalpha_n = sum_e dalpha_partial[e, n]   (slots / experts ascending)
// Vector scales: written per feature.  Scalar scales (blk_sums != null): every block adds its features in fp64 (fixed
// tree) into blk_sums[2 * block], the block that arrives last adds the blocks' sums in index order -- the result does
// not depend on which block that is -- and writes the two scalars; `arrivals` was cleared by the call's first kernel.
__global__ void __launch_bounds__(128) k_finalize_scales(const float* __restrict__ dbeta_partial, int nslots,
                                                         const float* __restrict__ dalpha_partial, int E, int N,
                                                         const float* __restrict__ w_scales, float* __restrict__ dbeta,
                                                         float* __restrict__ dalpha, double* blk_sums, unsigned* arrivals) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  const int n = blockIdx.x * 128 + threadIdx.x;
  float b = 0.f, a = 0.f;
  if (n < N) {
#pragma unroll 8
    for (int s = 0; s < nslots; ++s) b += dbeta_partial[(long long)s * N + n];
    b *= w_scales[0];
    if (dalpha_partial) {
#pragma unroll 8
      for (int e = 0; e < E; ++e) a += dalpha_partial[(long long)e * N + n];
    }
  }
  if (!blk_sums) {
    if (n < N) {
      dbeta[n] = b;
      if (dalpha_partial) dalpha[n] = a;
    }
    return;
  }
  __shared__ double sh[2][4];
  __shared__ bool last;
  double sb = (double)b, sa = (double)a;
  for (int d = 16; d > 0; d >>= 1) {
    sb += __shfl_xor_sync(0xffffffffu, sb, d);
    sa += __shfl_xor_sync(0xffffffffu, sa, d);
  }
  if ((threadIdx.x & 31) == 0) { sh[0][threadIdx.x >> 5] = sb; sh[1][threadIdx.x >> 5] = sa; }
  __syncthreads();
  if (threadIdx.x == 0) {
    blk_sums[2 * blockIdx.x] = (sh[0][0] + sh[0][1]) + (sh[0][2] + sh[0][3]);
    blk_sums[2 * blockIdx.x + 1] = (sh[1][0] + sh[1][1]) + (sh[1][2] + sh[1][3]);
    __threadfence();
    last = atomicAdd(arrivals, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!last || threadIdx.x >= 32) return;
  __threadfence();
  double tb = 0.0, ta = 0.0;
  for (int i = threadIdx.x; i < (int)gridDim.x; i += 32) { tb += __ldcg(blk_sums + 2 * i); ta += __ldcg(blk_sums + 2 * i + 1); }
  for (int d = 16; d > 0; d >>= 1) {
    tb += __shfl_xor_sync(0xffffffffu, tb, d);
    ta += __shfl_xor_sync(0xffffffffu, ta, d);
  }
  if (threadIdx.x == 0) {
    dbeta[0] = (float)tb;
    if (dalpha_partial) dalpha[0] = (float)ta;
  }
}

// ---------------------------------------------------------------------------
// INT8 high-precision branch (Sec. 3.2): the expert matrices quantised the way the 8-bit activations are
// (Eq. 7-9 with one scale per matrix): gamma = 128 / max(amax, 1e-5), code = clamp(rint(w * gamma), -128, 127).
// Matrix id = 2 e + (0: A_e [r,K], 1: B_e [N,r]); grid (blocks, 2 E).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_expert_amax(const uint4* __restrict__ A, const uint4* __restrict__ B, long long nA, long long nB,
                                                     uint32_t* amax_bits) {
  pdl_launch_dependents();
  pdl_wait();
  const int mat = blockIdx.y, e = mat >> 1;
  const long long n = (mat & 1) ? nB : nA;                      // 16-byte pieces (8 values) of one matrix
  const uint4* src = ((mat & 1) ? B : A) + (long long)e * n;
  float amax = 0.f;
  for (long long i = blockIdx.x * 256LL + threadIdx.x; i < n; i += gridDim.x * 256LL) {
    const uint4 v = __ldg(src + i);
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.x)), fabsf(bf16hi(v.x))), fmaxf(fabsf(bf16lo(v.y)), fabsf(bf16hi(v.y)))));
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.z)), fabsf(bf16hi(v.z))), fmaxf(fabsf(bf16lo(v.w)), fabsf(bf16hi(v.w)))));
  }
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  // non-negative floats order like their bit patterns; the maximum does not depend on the order of the updates
  if ((threadIdx.x & 31) == 0) atomicMax(amax_bits + mat, __float_as_uint(amax));
}

__global__ void __launch_bounds__(256) k_expert_quant(const uint4* __restrict__ A, const uint4* __restrict__ B, long long nA, long long nB,
                                                      const uint32_t* amax_bits, uint2* __restrict__ A8, uint2* __restrict__ B8,
                                                      float* __restrict__ hp_scales) {
  pdl_launch_dependents();
  pdl_wait();
  const int mat = blockIdx.y, e = mat >> 1;
  const long long n = (mat & 1) ? nB : nA;
  const uint4* src = ((mat & 1) ? B : A) + (long long)e * n;
  uint2* dst = ((mat & 1) ? B8 : A8) + (long long)e * n;
  const float gamma = __fdiv_rn(kActQmax, fmaxf(__uint_as_float(__ldcg(amax_bits + mat)), kActAmaxFloor));
  if (blockIdx.x == 0 && threadIdx.x == 0) hp_scales[mat] = gamma;
  for (long long i = blockIdx.x * 256LL + threadIdx.x; i < n; i += gridDim.x * 256LL) {
    const uint4 v = __ldg(src + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int qi[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      qi[2 * j] = max(-128, min(127, __float2int_rn(__fmul_rn(bf16lo(w[j]), gamma))));
      qi[2 * j + 1] = max(-128, min(127, __float2int_rn(__fmul_rn(bf16hi(w[j]), gamma))));
    }
    uint2 o;
    o.x = (qi[0] & 0xFF) | ((qi[1] & 0xFF) << 8) | ((qi[2] & 0xFF) << 16) | ((qi[3] & 0xFF) << 24);
    o.y = (qi[4] & 0xFF) | ((qi[5] & 0xFF) << 8) | ((qi[6] & 0xFF) << 16) | ((qi[7] & 0xFF) << 24);
    dst[i] = o;
  }
}

cudaError_t launch_pack_experts(const uint16_t* A, const uint16_t* B, int E, int r, int K, int N, int8_t* A8, int8_t* B8, float* hp_scales,
                                uint32_t* amax_bits, cudaStream_t st) {
  const long long nA = (long long)r * K / 8, nB = (long long)N * r / 8;
  if (cudaMemsetAsync(amax_bits, 0, sizeof(uint32_t) * 2 * E, st) != cudaSuccess) return cudaGetLastError();
  long long g = ((nA > nB ? nA : nB) + 1023) / 1024;
  const int gx = (int)(g < 1 ? 1 : (g > 296 ? 296 : g));
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)gx, (unsigned)(2 * E), 1); cfg.blockDim = dim3(256, 1, 1); cfg.stream = st;
  cfg.attrs = attr; cfg.numAttrs = 0;     // the first kernel follows a memset: plain stream order
  { LaunchScope ls(KID_PACK_SUMS, st);
    cudaLaunchKernelEx(&cfg, k_expert_amax, reinterpret_cast<const uint4*>(A), reinterpret_cast<const uint4*>(B), nA, nB, amax_bits); }
  cfg.numAttrs = 1;
  { LaunchScope ls(KID_BINARIZE_PACK, st);
    cudaLaunchKernelEx(&cfg, k_expert_quant, reinterpret_cast<const uint4*>(A), reinterpret_cast<const uint4*>(B), nA, nB,
                       static_cast<const uint32_t*>(amax_bits), reinterpret_cast<uint2*>(A8), reinterpret_cast<uint2*>(B8), hp_scales); }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// FFN-level decoupling (Eq. 11): the two small kernels between the projections.
// ---------------------------------------------------------------------------
// Hidden activation of the 1-bit FFN: M = bf16(silu(G) * U), element by element (fp32).
__global__ void __launch_bounds__(256) k_swiglu(const uint4* __restrict__ G, const uint4* __restrict__ U, uint4* __restrict__ M, long long n8) {
  pdl_launch_dependents();
  pdl_wait();
  for (long long i = blockIdx.x * 256LL + threadIdx.x; i < n8; i += gridDim.x * 256LL) {
    const uint4 g = __ldg(G + i), u = __ldg(U + i);
    const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, uw[4] = {u.x, u.y, u.z, u.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float g0 = bf16lo(gw[j]), g1 = bf16hi(gw[j]);
      o[j] = pack_bf16x2(g0 / (1.0f + __expf(-g0)) * bf16lo(uw[j]), g1 / (1.0f + __expf(-g1)) * bf16hi(uw[j]));
    }
    M[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// Hidden activation of the INT8 FFN, one warp per token: from the exact sums g_int = G8 q, u_int = U8 q
//   g = fl(fl(g_int) * fl(1 / fl(gamma_G gamma_t))), u likewise, m = fl(fl(g * s) * u) with the logistic factor s taken
//   in fp64 and rounded once to fp32 (an fp32 exponential would not be reproducible, and m feeds a quantiser),
// then Eq. 7-9 on the row of m: gamma_m = 128 / max(max|m|, 1e-5), codes clamp(rint(m gamma_m)).  r <= 128.
__global__ void __launch_bounds__(256) k_ffn8_act(const int* __restrict__ g_int, const int* __restrict__ u_int, const float* __restrict__ gamma,
                                                  const float* __restrict__ hp_scales, int T, int r, int8_t* __restrict__ qm,
                                                  float* __restrict__ gamma_m) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= T) return;
  const float gt = gamma[t];
  const float deq_g = __fdiv_rn(1.0f, __fmul_rn(hp_scales[0], gt)), deq_u = __fdiv_rn(1.0f, __fmul_rn(hp_scales[1], gt));
  float m[4];
  float amax = 0.f;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int j = lane + 32 * k;
    m[k] = 0.f;
    if (j < r) {
      const float g = __fmul_rn(__int2float_rn(g_int[(long long)t * r + j]), deq_g);
      const float u = __fmul_rn(__int2float_rn(u_int[(long long)t * r + j]), deq_u);
      const float s = (float)(1.0 / (1.0 + exp(-(double)g)));
      m[k] = __fmul_rn(__fmul_rn(g, s), u);
      amax = fmaxf(amax, fabsf(m[k]));
    }
  }
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  const float gm = __fdiv_rn(kActQmax, fmaxf(amax, kActAmaxFloor));
  if (lane == 0) gamma_m[t] = gm;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int j = lane + 32 * k;
    if (j < r) qm[(long long)t * r + j] = (int8_t)max(-128, min(127, __float2int_rn(__fmul_rn(m[k], gm))));
  }
}

cudaError_t launch_swiglu(const uint16_t* G, const uint16_t* U, uint16_t* M, long long n, cudaStream_t st) {
  const long long n8 = n / 8;
  long long g = (n8 + 1023) / 1024;
  launch_pdl(k_swiglu, (int)(g < 1 ? 1 : (g > 148 * 8 ? 148 * 8 : g)), 256, 0, st, reinterpret_cast<const uint4*>(G), reinterpret_cast<const uint4*>(U),
             reinterpret_cast<uint4*>(M), n8);
  ++g_launches;
  return cudaGetLastError();
}

cudaError_t launch_ffn8_act(const int* g_int, const int* u_int, const float* gamma, const float* hp_scales, int T, int r, int8_t* qm,
                            float* gamma_m, cudaStream_t st) {
  launch_pdl(k_ffn8_act, (T + 7) / 8, 256, 0, st, g_int, u_int, gamma, hp_scales, T, r, qm, gamma_m);
  ++g_launches;
  return cudaGetLastError();
}

__global__ void k_fill_zero(uint4* p, long long n16) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  for (long long i = blockIdx.x * 256LL + threadIdx.x; i < n16; i += gridDim.x * 256LL) p[i] = make_uint4(0, 0, 0, 0);
}

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------
static inline int grid_for(long long work, int per_block, int cap) {
  long long g = (work + per_block - 1) / per_block;
  if (g < 1) g = 1;
  return (int)(g > cap ? cap : g);
}

cudaError_t launch_pack(const float* W, int N, int K, uint32_t* bits, int8_t* s8, float* scales, double* partial, cudaStream_t st) {
  const long long n4 = (long long)N * K / 4;
  const int nparts = grid_for(n4, 256 * 8, 6 * 148);   // six blocks per SM, each thread keeps four loads in flight (~14 MB in all)
  static_assert(6 * 148 <= kPackPartials, "partial sums of the weight reduction");
  { LaunchScope ls(KID_PACK_SUMS, st);
  launch_pdl(k_weight_partial_sums, nparts, 256, 0, st, reinterpret_cast<const float4*>(W), n4, partial); }
  const int grid = grid_for(n4, 256 * 4, 148 * 8);
  LaunchScope ls(KID_BINARIZE_PACK, st);
  launch_pdl(k_binarize_pack, grid, 256, 0, st, reinterpret_cast<const float4*>(W), n4, partial, nparts, 1.0 / ((double)N * K), bits,
                                        reinterpret_cast<uint32_t*>(s8), scales);
  return cudaGetLastError();
}

cudaError_t launch_route_and_quant(const uint16_t* X, const uint16_t* Wr, int T, int K, int E, const SavedPtrs& sv, const FwdScratch& sc,
                                   cudaStream_t st, cudaStream_t st_quant, const uint16_t* norm_weight, float norm_eps) {
  if (E > 1) st_quant = st;   // the sorted position of a token comes from the router and the scan
  const uint4* nw = reinterpret_cast<const uint4*>(norm_weight);
  if (nw) {
    st_quant = st;
    LaunchScope ls(KID_ROUTER, st);
    launch_pdl(k_row_rms, (T + 7) / 8, 256, 0, st, reinterpret_cast<const uint4*>(X), T, K, norm_eps, sc.rms);
  }
  const int nblocks = (T + kRouterTokensPerBlock - 1) / kRouterTokensPerBlock;
  if (E > 1) {
    LaunchScope ls(KID_ROUTER, st);
    // two tokens per warp (half the loads and unpacking of Wr per token), 512 threads
    if (E <= 4) launch_pdl(k_router<4, 4>, nblocks, 8 * kRouterTokensPerBlock, 0, st, reinterpret_cast<const uint4*>(X), reinterpret_cast<const uint4*>(Wr), T, K, E,
                           sv.expert, sc.gate_tok, sc.probs_tok, sc.block_counts, nw, sc.rms);
    else if (E <= 8) launch_pdl(k_router<8, 4>, nblocks, 8 * kRouterTokensPerBlock, 0, st, reinterpret_cast<const uint4*>(X), reinterpret_cast<const uint4*>(Wr), T, K, E,
                                sv.expert, sc.gate_tok, sc.probs_tok, sc.block_counts, nw, sc.rms);
    else launch_pdl(k_router<kMaxExperts, 2>, nblocks, 16 * kRouterTokensPerBlock, 0, st, reinterpret_cast<const uint4*>(X), reinterpret_cast<const uint4*>(Wr), T, K, E,
                    sv.expert, sc.gate_tok, sc.probs_tok, sc.block_counts, nw, sc.rms);
  }
  { LaunchScope ls(KID_ROUTE_SCAN, st);
  launch_pdl(k_route_scan, 1, 512, 0, st, T, E, nblocks, sc.block_counts, sc.block_base, sv.offsets, sv.rt); }
  LaunchScope ls(KID_ACT_QUANT, st_quant);
  const int per_lane = (K / 8 + 31) / 32;   // 16-byte pieces of a row per lane if one warp took the whole row
  auto kern = k_act_quant<0, 1>;
  int wpr = 1;
  if (per_lane <= 4) kern = k_act_quant<4, 1>;
  else if (per_lane <= 8) kern = k_act_quant<8, 1>;
  else if (per_lane <= 16) { kern = k_act_quant<8, 2>; wpr = 2; }
  else if (per_lane <= 32) { kern = k_act_quant<8, 4>; wpr = 4; }
  const int rows_per_block = 8 / wpr;
  launch_pdl(kern, (T + rows_per_block - 1) / rows_per_block, 256, 0, st_quant, reinterpret_cast<const uint4*>(X), T, K, E, sv.expert, sc.block_base, sv.offsets, sc.gate_tok,
                                    sc.probs_tok, reinterpret_cast<uint2*>(sv.q), reinterpret_cast<uint4*>(sv.xt),
                                    reinterpret_cast<uint4*>(sv.xs), sv.gamma, sv.gate, sv.probs, sv.perm, sv.pos, nw, sc.rms);
  return cudaGetLastError();
}

cudaError_t launch_scatter_rows(const uint16_t* src, uint16_t* dst, const int* pos, int T, int row_elems, cudaStream_t st) {
  LaunchScope ls(KID_SCATTER_ROWS, st);
  launch_pdl(k_scatter_rows, (T + 7) / 8, 256, 0, st, reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), pos, T, row_elems / 8);
  return cudaGetLastError();
}

cudaError_t launch_scaled_sign(const int8_t* s8, uint16_t* out, const float* beta, int beta_stride, int N, int K, unsigned* arrivals,
                               cudaStream_t st) {
  const long long n16 = (long long)N * K / 16;
  LaunchScope ls(KID_SCALED_SIGN, st);
  launch_pdl(k_scaled_sign, grid_for(n16, 256 * 2, 148 * 8), 256, 0, st, reinterpret_cast<const uint4*>(s8), reinterpret_cast<uint4*>(out), beta,
                                                               beta_stride, N, K, arrivals);
  return cudaGetLastError();
}

cudaError_t launch_scaled_b(const uint16_t* B, uint16_t* out, const float* alpha, int E, int N, int r, cudaStream_t st) {
  const long long n2 = (long long)E * N * r / 2;
  LaunchScope ls(KID_SCALED_B, st);
  launch_pdl(k_scaled_b, grid_for(n2, 256 * 4, 148 * 8), 256, 0, st, reinterpret_cast<const uint32_t*>(B), reinterpret_cast<uint32_t*>(out), alpha, E, N, r);
  return cudaGetLastError();
}

cudaError_t launch_finalize_scales(const float* dbeta_partial, int nslots, const float* dalpha_partial, int E, int N, const float* w_scales,
                                   int vec, float* dbeta, float* dalpha, double* blk_sums, unsigned* arrivals, cudaStream_t st) {
  LaunchScope ls(vec ? KID_SUM_PARTIALS : KID_SUM_SCALAR, st);
  launch_pdl(k_finalize_scales, (N + 127) / 128, 128, 0, st, dbeta_partial, nslots, dalpha_partial, E, N, w_scales, dbeta, dalpha,
             vec ? nullptr : blk_sums, vec ? nullptr : arrivals);
  return cudaGetLastError();
}

cudaError_t launch_fill_zero(void* p, size_t bytes, cudaStream_t st) {
  const long long n16 = (long long)(bytes / 16);
  if (n16 == 0) return cudaSuccess;
  launch_pdl(k_fill_zero, grid_for(n16, 256 * 4, 148 * 4), 256, 0, st, reinterpret_cast<uint4*>(p), n16);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// experts' down-projections side by side: out[n, e r + j] = B[e, n, j] (the all-experts test mode of the forward)
// ---------------------------------------------------------------------------
__global__ void k_concat_experts(const uint4* __restrict__ B, uint4* __restrict__ out, int E, int N, int r8) {
  const long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= (long long)N * E * r8) return;
  const int jc = (int)(o % r8);
  const long long t = o / r8;
  const int e = (int)(t % E);
  const long long n = t / E;
  out[o] = B[((long long)e * N + n) * r8 + jc];
}
cudaError_t launch_concat_experts(const uint16_t* B, int E, int N, int r, uint16_t* out, cudaStream_t st) {
  const long long total = (long long)N * E * (r / 8);
  LaunchScope ls(KID_SCATTER_ROWS, st);
  k_concat_experts<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(reinterpret_cast<const uint4*>(B), reinterpret_cast<uint4*>(out), E, N, r / 8);
  return cudaGetLastError();
}

}  // namespace pq
