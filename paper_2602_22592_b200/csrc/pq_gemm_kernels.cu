// Tensor-core kernels of the pQuant layer, built on the engine in pq_gemm.cuh:
//   forward  : H = X A_e^T (grouped by expert), then the fused output tile
//              Y = alpha g (H B_e^T) + beta (lam/gamma) (q S^T)      (Eq. 10, 11)
//   backward : dH, dX, dW, dB, dA of the straight-through estimator  (App. B.1)
//   debug    : raw accumulators of one contraction, for bit-exact tests
#include <type_traits>

#include "pq_gemm.cuh"
#include "pq_kernels.cuh"

namespace pq {

// ---------------------------------------------------------------------------
// tensor maps
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Row-major tensor of `rank` dims (dims[0] innermost), 128-byte swizzle, zero fill outside.
// box[0] * elem_bytes must be 128.  Returns false on any violated precondition.
static bool make_map(CUtensorMap* m, bool is_i8, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                     const uint32_t* box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const int eb = is_i8 ? 1 : 2;
  if ((reinterpret_cast<uintptr_t>(base) & 15) != 0) return false;
  if (box[0] * eb != 128) return false;
  cuuint64_t gd[4];
  cuuint64_t gs[3];
  cuuint32_t bx[4], es[4];
  for (int i = 0; i < rank; ++i) {
    gd[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    if (box[i] > 256 || dims[i] == 0) return false;
  }
  for (int i = 0; i + 1 < rank; ++i) {
    gs[i] = strides_bytes[i];
    if (gs[i] % 16) return false;
  }
  CUresult r = fn(m, is_i8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd,
                  gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

static bool map2d(CUtensorMap* m, bool is_i8, const void* base, uint64_t inner, uint64_t outer, uint32_t box_inner, uint32_t box_outer) {
  const uint64_t dims[2] = {inner, outer};
  const uint64_t strides[1] = {inner * (is_i8 ? 1 : 2)};
  const uint32_t box[2] = {box_inner, box_outer};
  return make_map(m, is_i8, base, 2, dims, strides, box);
}
static bool map3d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t mid, uint64_t outer, uint32_t box_inner, uint32_t box_mid) {
  const uint64_t dims[3] = {inner, mid, outer};
  const uint64_t strides[2] = {inner * 2, inner * mid * 2};
  const uint32_t box[3] = {box_inner, box_mid, 1};
  return make_map(m, false, base, 3, dims, strides, box);
}

// int8 [outer][mid][inner] with the contraction index innermost: boxes of 128 bytes x box_mid rows of one batch entry;
// `pitch` is the row stride in bytes (a multiple of 16, at least `inner`)
static bool map3d_i8(CUtensorMap* m, const void* base, uint64_t inner, uint64_t pitch, uint64_t mid, uint64_t outer, uint32_t box_mid) {
  const uint64_t dims[3] = {inner, mid, outer};
  const uint64_t strides[2] = {pitch, pitch * mid};
  const uint32_t box[3] = {128, box_mid, 1};
  return make_map(m, true, base, 3, dims, strides, box);
}

// MN-major operand: matrix [batch][k_total][mn_total] with mn contiguous, read in 64 (mn) x 64 (k) boxes.
// When mn_total is a multiple of 64 the map views the 64-wide column blocks as a dimension of their own,
// (64, k_total, mn_total / 64[, batch]) -- base_rank 2 or 3 says whether the operand has the batch dimension --, so that ONE load delivers `nblk` boxes back to back; *blk = nblk.
// Otherwise (a narrower last block would alias the next row) a plain map with one box per load; *blk = 0.
static bool map_mn(CUtensorMap* m, int* blk, const void* base, uint64_t mn_total, uint64_t k_total, int base_rank, uint64_t batch, int nblk) {
  if (mn_total % 64 == 0) {
    *blk = nblk;
    const uint64_t dims[4] = {64, k_total, mn_total / 64, batch};
    const uint64_t strides[3] = {mn_total * 2, 128, mn_total * k_total * 2};
    const uint32_t box[4] = {64, 64, (uint32_t)nblk, 1};
    return make_map(m, false, base, base_rank + 1, dims, strides, box);
  }
  *blk = 0;
  return base_rank == 3 ? map3d(m, base, mn_total, k_total, batch, 64, 64) : map2d(m, false, base, mn_total, k_total, 64, 64);
}

static int g_sm_count = 0;
static int sm_count() {
  if (!g_sm_count) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (g_sm_count <= 0) g_sm_count = 148;
  }
  return g_sm_count;
}

static int grid_for_tiles(int max_tiles) {
  int grid = max_tiles < sm_count() ? max_tiles : sm_count();
  return grid < 1 ? 1 : grid;
}

template <class Params>
static int launch_gemm(int kernel_id, void (*kernel)(Params), const Params& p, int max_tiles, cudaStream_t st) {
  // (cudaFuncSetAttribute is cheap and idempotent; calling it per launch keeps this free of static state per kernel)
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes) != cudaSuccess) return PQ_ERR_CUDA;
  const int grid = grid_for_tiles(max_tiles);
  LaunchScope ls(kernel_id, st);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid, 1, 1); cfg.blockDim = dim3(kGemmThreads, 1, 1); cfg.dynamicSmemBytes = kGemmSmemBytes;
  cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, p) == cudaSuccess ? PQ_OK : PQ_ERR_CUDA;
}

__device__ __forceinline__ int round_up(int x, int m) { return (x + m - 1) / m * m; }
// width actually contracted for a tile that starts at n0: the tile's width, cut at the matrix edge
__device__ __forceinline__ int clip_bn(int bn, int n0, int n_total, int granule) {
  const int left = round_up(n_total - n0, granule);
  return left < bn ? (left > 0 ? left : granule) : bn;
}

// Intermediates that feed a second tensor-core product (H, g H, dH / c) are kept
// as TWO bf16 planes, v ~= hi + lo with hi = bf16(v), lo = bf16(v - hi): about 16
// significand bits, so their rounding does not show in the results.  The planes
// are stacked along the row axis ([2][item_rows][r]); a product against such an
// operand simply runs its contraction over both planes.
__device__ __forceinline__ void split2(float a, float b, uint32_t& hi, uint32_t& lo) {
  hi = pack_bf16x2(a, b);
  lo = pack_bf16x2(a - bf16lo(hi), b - bf16hi(hi));
}
static inline int h_round_up(int x, int m) { return (x + m - 1) / m * m; }

// ---------------------------------------------------------------------------
// debug: D[M,N] = contraction of A and B in one of the four operand forms
// ---------------------------------------------------------------------------
struct DebugProblem {
  using Acc = AccDouble;
  struct Params {
    CUtensorMap ta, tb;
    TileGrid g;
    int mode, M, N, K, a_blk, b_blk;
    void* D;
  };
  struct Tile { TileCoord c; };
  __device__ static int num_tiles(const Params& p) { return p.g.total; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) { t.c = tile_coord(p.g, i); }
  __device__ static int num_segments(const Params&, const Tile&) { return 1; }
  __device__ static void segment(const Params& p, const Tile& t, int, Segment& s) {
    s.mode = p.mode; s.acc = 0; s.ksteps = 4; s.b_box = p.g.bn; s.a_blk = p.a_blk; s.b_blk = p.b_blk;
    s.bn = clip_bn(t.c.bn, t.c.n0, p.N, p.mode >= MODE_BF_KM ? 64 : 32);
    const int bk = p.mode == MODE_I8_KK ? 128 : 64;
    s.nkb = (p.K + bk - 1) / bk;
    s.ta = &p.ta; s.tb = &p.tb; s.a_rank = 2; s.b_rank = 2; s.a_z = 0; s.b_z = 0;
    if (p.mode == MODE_BF_MM) { s.a_x = t.c.m * 128; s.a_y = 0; } else { s.a_x = 0; s.a_y = t.c.m * 128; }
    if (p.mode >= MODE_BF_KM) { s.b_x = t.c.n0; s.b_y = 0; } else { s.b_x = 0; s.b_y = t.c.n0; }
  }
  using Pre = NoPre;
  __device__ static Pre prepare(const Params&, const Tile&, int, int) { return Pre{}; }
  __device__ static void epilogue(const Params& p, const Tile& t, const Pre& pre, uint32_t tacc, uint32_t, int quad, int half, int lane, uint8_t* stage) {
    const int row = t.c.m * 128 + quad * 32 + lane;
    uint32_t* D = reinterpret_cast<uint32_t*>(p.D);
    for (int c = half; c * 32 < t.c.bn; c += 2) {
      const int n0 = t.c.n0 + c * 32;
      if (n0 >= p.N) break;
      uint32_t v[32];
      tmem_ld32(tacc + c * 32, v);
      tmem_ld_wait();
      uint4 o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) o[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      const int valid = min(32, p.N - n0) * 4;   // N is a multiple of 8 -> whole 16-byte pieces
      warp_store_rows(stage, o, row < p.M ? D + (long long)row * p.N + n0 : nullptr, valid, lane);
    }
  }
};
PQ_DEFINE_GEMM_KERNEL(k_gemm_debug, DebugProblem)

int gemm_debug(int mode, int M, int N, int K, const void* A, const void* B, void* D, int tile_n, cudaStream_t st) {
  DebugProblem::Params p;
  p.mode = mode; p.M = M; p.N = N; p.K = K; p.D = D; p.a_blk = 0; p.b_blk = 0;
  const int granule = mode >= MODE_BF_KM ? 64 : 32;
  if (tile_n <= 0) tile_n = 256;
  if (tile_n > 256 || tile_n % granule) return PQ_ERR_SHAPE;
  const int mt = (M + 127) / 128, nt = (N + tile_n - 1) / tile_n;
  p.g = make_tile_grid(mt, nt, tile_n);
  bool ok = true;
  switch (mode) {
    case MODE_I8_KK:
      ok = map2d(&p.ta, true, A, K, M, 128, 128) && map2d(&p.tb, true, B, K, N, 128, tile_n);
      break;
    case MODE_BF_KK:
      ok = map2d(&p.ta, false, A, K, M, 64, 128) && map2d(&p.tb, false, B, K, N, 64, tile_n);
      break;
    case MODE_BF_KM:
      ok = map2d(&p.ta, false, A, K, M, 64, 128) && map_mn(&p.tb, &p.b_blk, B, N, K, 2, 1, tile_n / 64);
      break;
    case MODE_BF_MM:
      ok = map_mn(&p.ta, &p.a_blk, A, M, K, 2, 1, 2) && map_mn(&p.tb, &p.b_blk, B, N, K, 2, 1, tile_n / 64);
      break;
    default:
      return PQ_ERR_UNSUPPORTED;
  }
  if (!ok) return PQ_ERR_CUDA;
  return launch_gemm(KID_DEBUG, k_gemm_debug, p, p.g.total, st);
}

// ---------------------------------------------------------------------------
// F1: hidden activations of the HP branch, H = X_sorted A_e^T, one tile per item
// ---------------------------------------------------------------------------
struct HpUpProblem {
  using Acc = AccDouble;
  struct Params {
    CUtensorMap tx, ta;  // X sorted [T,K]; A [E,r,K]
    RoutingTables rt;
    uint16_t* H;
    int K, r, bn, item_rows;
  };
  struct Tile { int item; int4 it; };
  __device__ static int stage_cols(const Params& p) { return p.bn <= 128 ? 128 : 256; }
  __device__ static int num_tiles(const Params& p) { return p.rt.n_items[0]; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) { t.item = i; t.it = p.rt.items[i]; }
  __device__ static int num_segments(const Params&, const Tile&) { return 1; }
  __device__ static void segment(const Params& p, const Tile& t, int, Segment& s) {
    s.mode = MODE_BF_KK; s.acc = 0; s.bn = p.bn; s.ksteps = 4; s.nkb = (p.K + 63) / 64;
    s.ta = &p.tx; s.a_rank = 2; s.a_x = 0; s.a_y = t.it.x * 128; s.a_z = 0;
    s.tb = &p.ta; s.b_rank = 3; s.b_x = 0; s.b_y = 0; s.b_z = t.it.y;
    s.b_box = p.bn; s.a_blk = 0; s.b_blk = 0;
  }
  using Pre = NoPre;
  __device__ static Pre prepare(const Params&, const Tile&, int, int) { return Pre{}; }
  __device__ static void epilogue(const Params& p, const Tile& t, const Pre& pre, uint32_t taddr, uint32_t, int quad, int half, int lane, uint8_t* stage) {
    const int row = quad * 32 + lane;
    const bool live = row >= t.it.z && row < t.it.w;
    uint4* out_hi = reinterpret_cast<uint4*>(p.H + ((long long)t.item * 128 + row) * p.r);
    uint4* out_lo = reinterpret_cast<uint4*>(p.H + ((long long)p.item_rows + t.item * 128 + row) * p.r);
    for (int c = half; c * 32 < p.r; c += 2) {
      uint32_t v[32];
      tmem_ld32(taddr + c * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (c * 32 + g * 8 < p.r) {
          uint32_t hi[4] = {0, 0, 0, 0}, lo[4] = {0, 0, 0, 0};
          if (live) {
#pragma unroll
            for (int j = 0; j < 4; ++j) split2(__uint_as_float(v[8 * g + 2 * j]), __uint_as_float(v[8 * g + 2 * j + 1]), hi[j], lo[j]);
          }
          out_hi[c * 4 + g] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          out_lo[c * 4 + g] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      }
    }
  }
};

PQ_DEFINE_GEMM_KERNEL(k_gemm_hp_up, HpUpProblem)

// ---------------------------------------------------------------------------
// F1 in INT8 (Sec. 3.2): h_int = q_sorted A8_e^T, exact in int32, one tile per item; the epilogue quantises each
// row of h per token the way activations are (Eq. 7-9, taken from the integers: gamma_h = 128 / max |h_int|) and
// writes the codes qh [items*128, rp] (row pitch rp = r rounded up to 16, padding zero) and gamma_h [items*128].
// ---------------------------------------------------------------------------
struct HpUp8Problem {
  using Acc = AccDouble;
  struct Params {
    CUtensorMap tq, ta;  // q sorted [T,K] s8; A8 [E,r,K] s8
    RoutingTables rt;
    int8_t* qh;
    float* gamma_h;
    int* raw;            // not null: write the exact sums h_int [items*128, r] instead of codes (the caller quantises later)
    int K, r, rp, bn;
  };
  struct Tile { int item; int4 it; };
  __device__ static int stage_cols(const Params& p) { return p.bn <= 128 ? 128 : 256; }
  __device__ static int num_tiles(const Params& p) { return p.rt.n_items[0]; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) { t.item = i; t.it = p.rt.items[i]; }
  __device__ static int num_segments(const Params&, const Tile&) { return 1; }
  __device__ static void segment(const Params& p, const Tile& t, int, Segment& s) {
    s.mode = MODE_I8_KK; s.acc = 0; s.bn = p.bn; s.ksteps = 4; s.nkb = (p.K + 127) / 128;
    s.ta = &p.tq; s.a_rank = 2; s.a_x = 0; s.a_y = t.it.x * 128; s.a_z = 0;
    s.tb = &p.ta; s.b_rank = 3; s.b_x = 0; s.b_y = 0; s.b_z = t.it.y;
    s.b_box = p.bn; s.a_blk = 0; s.b_blk = 0;
  }
  using Pre = NoPre;
  __device__ static Pre prepare(const Params&, const Tile&, int, int) { return Pre{}; }
  __device__ static void epilogue(const Params& p, const Tile& t, const Pre& pre, uint32_t taddr, uint32_t, int quad, int half, int lane, uint8_t* stage) {
    if (p.raw) {
      int* out = p.raw + ((long long)t.item * 128 + quad * 32 + lane) * p.r;
      for (int c = half; c * 32 < p.r; c += 2) {
        uint32_t v[32];
        tmem_ld32(taddr + c * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c * 32 + 4 * j < p.r) reinterpret_cast<uint4*>(out + c * 32)[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      }
      return;
    }
    if (half) return;   // the maximum over a row's r columns stays in one thread
    const int row = quad * 32 + lane;
    const bool live = row >= t.it.z && row < t.it.w;
    int amax = 0;
    for (int c = 0; c * 32 < p.r; ++c) {
      uint32_t v[32];
      tmem_ld32(taddr + c * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (c * 32 + j < p.r) amax = max(amax, abs((int)v[j]));
    }
    const float gamma_h = __fdiv_rn(kActQmax, fmaxf(__int2float_rn(amax), kActAmaxFloor));
    const long long grow = (long long)t.item * 128 + row;
    p.gamma_h[grow] = live ? gamma_h : 0.f;
    uint4* out = reinterpret_cast<uint4*>(p.qh + grow * p.rp);
    for (int c = 0; c * 32 < p.rp; ++c) {
      uint32_t v[32];
      tmem_ld32(taddr + c * 32, v);
      tmem_ld_wait();
      uint32_t w[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        uint32_t word = 0u;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int col = c * 32 + 4 * j + b;
          int code = 0;
          if (live && col < p.r) code = max(-128, min(127, __float2int_rn(__fmul_rn(__int2float_rn((int)v[4 * j + b]), gamma_h))));
          word |= (uint32_t)(code & 0xFF) << (8 * b);
        }
        w[j] = word;
      }
      if (c * 32 < p.rp) out[2 * c] = make_uint4(w[0], w[1], w[2], w[3]);
      if (c * 32 + 16 < p.rp) out[2 * c + 1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
  }
};
PQ_DEFINE_GEMM_KERNEL(k_gemm_hp_up8, HpUp8Problem)

// ---------------------------------------------------------------------------
// F2: fused output tile.  Accumulator 0 (int32): q S^T over K.  Accumulator 1
// (fp32): H B_e^T over r, once per item of the tile (masked H rows are zero).
// Epilogue: Y[token, n] = alpha_n g z + beta_n (lam / gamma) acc, rounded once.
// ---------------------------------------------------------------------------
template <bool HP>
struct FwdProblem {
  // with the HP branch a tile holds an int32 and an fp32 accumulator of 256 columns each: all of TMEM
  using Acc = typename std::conditional<HP, AccPair, AccDouble>::type;
  struct Params {
    CUtensorMap tq, ts, th, tb;  // q [T,K] s8; S [N,K] s8; H [items*128,r]; B [E,N,r]
    RoutingTables rt;
    TileGrid g;
    const int* perm;
    const float* gamma;
    const float* gate;
    const float* w_scales;
    const float* alpha;
    const float* beta;
    uint16_t* Y;
    // INT8 HP branch (Sec. 3.2): th / tb then map the int8 codes of h and of B_e, the second accumulator is int32, and
    // its de-quantisation factor 1 / (gamma_B gamma_h gamma_A gamma_t) is folded into the row's HP factor
    const float* gamma_h;    // [items*128], null for the bf16 branch
    const float* hp_scales;  // [E][2] = {gamma_A, gamma_B}
    int hp_ext;              // the codes of h and gamma_h were written by the caller
    int T, N, K, r, sstride, item_rows;
  };
  struct Tile { TileCoord c; int bn, ib, ie; };
  __device__ static int num_tiles(const Params& p) { return p.g.total; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) {
    t.c = tile_coord(p.g, i);
    t.bn = clip_bn(t.c.bn, t.c.n0, p.N, 32);
    if (HP) { t.ib = p.rt.tile_item_begin[t.c.m]; t.ie = p.rt.tile_item_begin[t.c.m + 1]; } else { t.ib = t.ie = 0; }
  }
  // The HP product uses the leading bf16 plane of H only: its 2^-9 relative rounding is of the size of the
  // output's own rounding to bf16; the second plane serves the backward pass, whose sums are longer.
  __device__ static int num_segments(const Params&, const Tile& t) { return 1 + (t.ie - t.ib); }
  __device__ static void segment(const Params& p, const Tile& t, int i, Segment& s) {
    s.bn = t.bn; s.ksteps = 4; s.a_z = 0; s.b_z = 0; s.b_box = 256; s.a_blk = 0; s.b_blk = 0;
    if (i == 0) {
      s.mode = MODE_I8_KK; s.acc = 0; s.nkb = (p.K + 127) / 128;
      s.ta = &p.tq; s.a_rank = 2; s.a_x = 0; s.a_y = t.c.m * 128;
      s.tb = &p.ts; s.b_rank = 2; s.b_x = 0; s.b_y = t.c.n0;
    } else {
      const int item = t.ib + (i - 1);
      const int e = p.rt.items[item].y;
      if (p.gamma_h) { s.mode = MODE_I8_KK; s.acc = 1; s.nkb = (p.r + 127) / 128; }
      else { s.mode = MODE_BF_KK; s.acc = 1; s.nkb = (p.r + 63) / 64; }
      s.ta = &p.th; s.a_rank = p.gamma_h ? 3 : 2; s.a_x = 0; s.a_y = item * 128;
      s.tb = &p.tb; s.b_rank = 3; s.b_x = 0; s.b_y = t.c.n0; s.b_z = e;
    }
  }
  // y = cb_n * acc + ca_n * z for 32 consecutive columns starting at n, packed to 16 bf16 pairs
  template <bool VEC>
  __device__ static __forceinline__ void combine32(const Params& p, int n, float cb, float ca, const uint32_t (&a)[32], const uint32_t (&z)[32],
                                                  uint4* out, bool z_is_int) {
    uint32_t w[16];
#pragma unroll
    for (int q4 = 0; q4 < 8; ++q4) {
      float b4[4] = {cb, cb, cb, cb}, a4[4] = {ca, ca, ca, ca};
      if (VEC) {
        const float4 bv = __ldg(reinterpret_cast<const float4*>(p.beta + n) + q4);
        b4[0] *= bv.x; b4[1] *= bv.y; b4[2] *= bv.z; b4[3] *= bv.w;
        if (HP) {
          const float4 av = __ldg(reinterpret_cast<const float4*>(p.alpha + n) + q4);
          a4[0] *= av.x; a4[1] *= av.y; a4[2] *= av.z; a4[3] *= av.w;
        }
      }
      float y[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        y[u] = b4[u] * (float)(int)a[4 * q4 + u];
        if (HP) y[u] = fmaf(a4[u], z_is_int ? (float)(int)z[4 * q4 + u] : __uint_as_float(z[4 * q4 + u]), y[u]);
      }
      w[2 * q4] = pack_bf16x2(y[0], y[1]);
      w[2 * q4 + 1] = pack_bf16x2(y[2], y[3]);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) out[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
  }
  // per-row factors: 1-bit branch lam / gamma_t (Eq. 10), HP branch g_t; scalar feature scales folded in
  struct Pre { uint16_t* yrow; float cb, ca; };
  __device__ static Pre prepare(const Params& p, const Tile& t, int quad, int lane) {
    const int pos = t.c.m * 128 + quad * 32 + lane;
    Pre r{nullptr, 0.f, 0.f};
    if (pos < p.T) {
      const int token = p.perm ? p.perm[pos] : pos;
      r.yrow = p.Y + (long long)token * p.N;
      r.cb = __fdiv_rn(p.w_scales[0], p.gamma[pos]);
      if (HP) r.ca = p.gate[pos];
      if (HP && p.gamma_h) {
        // the item of this row: its expert's weight scales and the row's own hidden scale
        const int rel = quad * 32 + lane;
        float deq = 0.f;
        for (int it = t.ib; it < t.ie; ++it) {
          const int4 d = p.rt.items[it];
          if (rel >= d.z && rel < d.w) {
            const float gh = p.gamma_h[(long long)it * 128 + rel];
            // hidden codes made by the library from h_int = A8 q carry gamma_A gamma_t; codes handed in from outside
            // (the FFN-level form, whose hidden activation went through its non-linearity first) carry gamma_h alone
            deq = p.hp_ext ? 1.0f / (p.hp_scales[2 * d.y + 1] * gh) : 1.0f / (p.hp_scales[2 * d.y + 1] * gh * p.hp_scales[2 * d.y] * p.gamma[pos]);
          }
        }
        r.ca *= deq;
      }
      if (!p.sstride) { r.cb *= p.beta[0]; if (HP) r.ca *= p.alpha[0]; }
    }
    return r;
  }
  __device__ static void epilogue(const Params& p, const Tile& t, const Pre& pre, uint32_t tacc, uint32_t tz, int quad, int half, int lane, uint8_t* stage) {
    const bool vec = p.sstride != 0;
    for (int c = half; c * 64 < t.bn; c += 2) {     // 64 output columns = 128 bytes of the row per pass
      const int n0 = t.c.n0 + c * 64;
      if (n0 >= p.N) break;
      uint4 o[8];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int nb = n0 + h * 32;
        if (c * 64 + h * 32 < t.bn && nb < p.N) {
          uint32_t a[32], z[32];
          tmem_ld32(tacc + c * 64 + h * 32, a);
          if (HP) tmem_ld32(tz + c * 64 + h * 32, z);
          tmem_ld_wait();
          if (vec) combine32<true>(p, nb, pre.cb, pre.ca, a, z, o + 4 * h, p.gamma_h != nullptr);
          else combine32<false>(p, nb, pre.cb, pre.ca, a, z, o + 4 * h, p.gamma_h != nullptr);
        }
      }
      warp_store_rows(stage, o, pre.yrow ? pre.yrow + n0 : nullptr, min(64, min(t.bn - c * 64, p.N - n0)) * 2, lane);
    }
  }
};
PQ_DEFINE_GEMM_KERNEL(k_gemm_fwd_hp, FwdProblem<true>)
PQ_DEFINE_GEMM_KERNEL(k_gemm_fwd_1bit, FwdProblem<false>)

// INT8 branch: the saved h region holds the codes qh [items*128, r] and, behind them, gamma_h [items*128]
static inline float* hp8_gamma_h(const SavedPtrs& sv, int r) {
  const size_t codes = ((size_t)sv.max_items * 128 * r + 255) / 256 * 256;
  return reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(sv.h) + codes);
}

template <bool HP>
static int fill_forward_params(const LayerArgs& a, const int8_t* w_s8, const SavedPtrs& sv, uint16_t* Y, typename FwdProblem<HP>::Params& f) {
  using P = FwdProblem<HP>;
  const int mtiles = (a.T + 127) / 128;
  if (!map2d(&f.tq, true, sv.q, a.K, a.T, 128, 128)) return PQ_ERR_CUDA;
  if (!map2d(&f.ts, true, w_s8, a.K, a.N, 128, 256)) return PQ_ERR_CUDA;
  f.th = f.tq; f.tb = f.tq;
  f.gamma_h = nullptr; f.hp_scales = a.hp_scales; f.hp_ext = a.hp_ext ? 1 : 0;
  if (HP && a.hp_scales) {
    // INT8 branch: codes of h [items*128, r] and of B_e [E, N, r], one byte per value
    const uint64_t rows = (uint64_t)sv.max_items * 128;
    if (!map3d_i8(&f.th, sv.h, a.r, a.r, rows, 1, 128)) return PQ_ERR_CUDA;
    if (!map3d_i8(&f.tb, a.B, a.r, a.r, a.N, a.E, 256)) return PQ_ERR_CUDA;
    f.gamma_h = hp8_gamma_h(sv, a.r);
  } else if (HP) {
    if (!map2d(&f.th, false, sv.h, a.r, (uint64_t)sv.max_items * 256, 64, 128)) return PQ_ERR_CUDA;
    if (!map3d(&f.tb, a.B, a.r, a.N, a.E, 64, 256)) return PQ_ERR_CUDA;
  }
  f.rt = sv.rt; f.perm = (HP && a.E > 1) ? sv.perm : nullptr; f.gamma = sv.gamma; f.gate = sv.gate; f.w_scales = a.w_scales;
  f.alpha = a.alpha; f.beta = a.beta; f.Y = Y; f.T = a.T; f.N = a.N; f.K = a.K; f.r = a.r; f.sstride = a.scale_stride;
  f.item_rows = sv.max_items * 128;
  f.g = make_tile_grid(mtiles, (a.N + 255) / 256, 256);
  return PQ_OK;
}

// h_int = q A8_e^T per item.  raw == nullptr: codes and scales of h into the saved h region; otherwise the exact sums
// [items*128, r] into `raw` (A8 [E, r, K] int8).
int gemm_hp_up8(const LayerArgs& a, const SavedPtrs& sv, const void* A8, int* raw, cudaStream_t st) {
  HpUp8Problem::Params p;
  p.rt = sv.rt; p.qh = reinterpret_cast<int8_t*>(sv.h); p.gamma_h = raw ? nullptr : hp8_gamma_h(sv, a.r); p.raw = raw;
  p.K = a.K; p.r = a.r; p.rp = a.r; p.bn = h_round_up(a.r, 16);
  if (!map2d(&p.tq, true, sv.q, a.K, a.T, 128, 128)) return PQ_ERR_CUDA;
  if (!map3d_i8(&p.ta, A8, a.K, a.K, a.r, a.E, p.bn)) return PQ_ERR_CUDA;
  return launch_gemm(KID_HP_UP, k_gemm_hp_up8, p, sv.max_items, st);
}

int gemm_forward(const LayerArgs& a, const int8_t* w_s8, const SavedPtrs& sv, const uint16_t* xs, uint16_t* Y, cudaStream_t st,
                 cudaEvent_t before_main) {
  if (a.r > 0 && a.hp_scales) {
    int rc = PQ_OK;
    if (!a.hp_ext) {
      rc = gemm_hp_up8(a, sv, a.A, nullptr, st);
      if (rc) return rc;
    }
    FwdProblem<true>::Params f;
    rc = fill_forward_params<true>(a, w_s8, sv, Y, f);
    if (rc) return rc;
    if (before_main && cudaStreamWaitEvent(st, before_main, 0) != cudaSuccess) return PQ_ERR_CUDA;
    return launch_gemm(KID_FWD, k_gemm_fwd_hp, f, f.g.total, st);
  }
  if (a.r > 0) {
    HpUpProblem::Params p;
    p.rt = sv.rt; p.H = sv.h; p.K = a.K; p.r = a.r; p.bn = h_round_up(a.r, 16); p.item_rows = sv.max_items * 128;
    if (!map2d(&p.tx, false, xs, a.K, a.T, 64, 128)) return PQ_ERR_CUDA;
    if (!map3d(&p.ta, a.A, a.K, a.r, a.E, 64, p.bn)) return PQ_ERR_CUDA;
    int rc = launch_gemm(KID_HP_UP, k_gemm_hp_up, p, sv.max_items, st);
    if (rc) return rc;
    FwdProblem<true>::Params f;
    rc = fill_forward_params<true>(a, w_s8, sv, Y, f);
    if (rc) return rc;
    if (before_main && cudaStreamWaitEvent(st, before_main, 0) != cudaSuccess) return PQ_ERR_CUDA;
    return launch_gemm(KID_FWD, k_gemm_fwd_hp, f, f.g.total, st);
  }
  FwdProblem<false>::Params f;
  int rc = fill_forward_params<false>(a, w_s8, sv, Y, f);
  if (rc) return rc;
  if (before_main && cudaStreamWaitEvent(st, before_main, 0) != cudaSuccess) return PQ_ERR_CUDA;
  return launch_gemm(KID_FWD, k_gemm_fwd_1bit, f, f.g.total, st);
}


// ===========================================================================
// backward (straight-through estimator, App. B.1)
// ===========================================================================
// The scale of the 1-bit input gradient: dX1 = c * (dYs . Sb) with
//   scalar beta:  Sb = S,            c = lam * beta
//   vector beta:  Sb = bf16(beta_n) S, c = lam
// The HP and router contributions are accumulated in the same tile, so they
// are pre-divided by c (and the whole tile multiplied by c in the epilogue).
// c == 0 switches the 1-bit term off instead.
__device__ __forceinline__ float dx_scale(const float* w_scales, const float* beta, int sstride) {
  return sstride ? w_scales[0] : w_scales[0] * beta[0];
}

// ---------------------------------------------------------------------------
// B1: dHraw = dYs . (alpha B_e) per item; epilogue forms
//   dg_t = alpha * sum_j H dHraw,  dH = g dHraw  ->  dhc = dH / c  (bf16, masked)
//   gh = g H (bf16, masked),  dl[t,j] = dg g (delta_je - p_tj),  dlc = dl / c
// ---------------------------------------------------------------------------
struct HpDhProblem {
  using Acc = AccDouble;
  struct Params {
    CUtensorMap tdy, tba;  // dYs [T,N]; (alpha) B [E,N,r]
    RoutingTables rt;
    const uint16_t* H;
    const float* gate;
    const float* probs;
    const float* w_scales;
    const float* alpha;
    const float* beta;
    uint16_t* dhc;
    uint16_t* gh;
    float* dl;
    uint16_t* dlc;
    int T, N, r, E, bn, sstride, item_rows, ba_blk;
  };
  struct Tile { int item; int4 it; };
  __device__ static int stage_cols(const Params& p) { return p.bn <= 128 ? 128 : 256; }
  __device__ static int num_tiles(const Params& p) { return p.rt.n_items[0]; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) { t.item = i; t.it = p.rt.items[i]; }
  __device__ static int num_segments(const Params&, const Tile&) { return 1; }
  __device__ static void segment(const Params& p, const Tile& t, int, Segment& s) {
    s.a_blk = 0; s.b_blk = p.ba_blk;
    s.mode = MODE_BF_KM; s.acc = 0; s.bn = p.bn; s.ksteps = 4; s.nkb = (p.N + 63) / 64;
    s.ta = &p.tdy; s.a_rank = 2; s.a_x = 0; s.a_y = t.it.x * 128; s.a_z = 0;
    s.tb = &p.tba; s.b_rank = 3; s.b_x = 0; s.b_y = 0; s.b_z = t.it.y;
    s.b_box = 0;
  }
  using Pre = NoPre;
  __device__ static Pre prepare(const Params&, const Tile&, int, int) { return Pre{}; }
  __device__ static void epilogue(const Params& p, const Tile& t, const Pre& pre, uint32_t taddr, uint32_t, int quad, int half, int lane, uint8_t* stage) {
    if (half) return;   // each row's sum over all r columns stays in one thread
    const int row = quad * 32 + lane;
    const bool live = row >= t.it.z && row < t.it.w;
    const int pos = t.it.x * 128 + row;
    const float c = dx_scale(p.w_scales, p.beta, p.sstride);
    const float inv_cc = c != 0.f ? 1.0f / c : 1.0f;
    const float ca = p.sstride ? 1.0f : p.alpha[0];
    const float g = live ? p.gate[pos] : 0.f;
    const long long hrow = ((long long)t.item * 128 + row) * p.r;
    const long long plane = (long long)p.item_rows * p.r;
    const uint4* hin = reinterpret_cast<const uint4*>(p.H + hrow);
    const uint4* hin_lo = reinterpret_cast<const uint4*>(p.H + plane + hrow);
    uint4* dhc = reinterpret_cast<uint4*>(p.dhc + hrow);
    uint4* dhc_lo = reinterpret_cast<uint4*>(p.dhc + plane + hrow);
    uint4* gh = reinterpret_cast<uint4*>(p.gh + hrow);
    uint4* gh_lo = reinterpret_cast<uint4*>(p.gh + plane + hrow);
    float dg = 0.f;
    for (int c32 = 0; c32 * 32 < p.r; ++c32) {
      uint32_t v[32];
      tmem_ld32(taddr + c32 * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int q8 = 0; q8 < 4; ++q8) {
        if (c32 * 32 + q8 * 8 < p.r) {
          uint32_t w1[4] = {0, 0, 0, 0}, w1l[4] = {0, 0, 0, 0}, w2[4] = {0, 0, 0, 0}, w2l[4] = {0, 0, 0, 0};
          if (live) {
            const uint4 hv = hin[c32 * 4 + q8], hl = hin_lo[c32 * 4 + q8];
            const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w}, hlw[4] = {hl.x, hl.y, hl.z, hl.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float h0 = bf16lo(hw[j]) + bf16lo(hlw[j]), h1 = bf16hi(hw[j]) + bf16hi(hlw[j]);
              const float d0 = __uint_as_float(v[q8 * 8 + 2 * j]), d1 = __uint_as_float(v[q8 * 8 + 2 * j + 1]);
              dg = fmaf(h0, d0, dg);
              dg = fmaf(h1, d1, dg);
              const float sc = ca * g * inv_cc;
              split2(sc * d0, sc * d1, w1[j], w1l[j]);
              split2(g * h0, g * h1, w2[j], w2l[j]);
            }
          }
          dhc[c32 * 4 + q8] = make_uint4(w1[0], w1[1], w1[2], w1[3]);
          dhc_lo[c32 * 4 + q8] = make_uint4(w1l[0], w1l[1], w1l[2], w1l[3]);
          gh[c32 * 4 + q8] = make_uint4(w2[0], w2[1], w2[2], w2[3]);
          gh_lo[c32 * 4 + q8] = make_uint4(w2l[0], w2l[1], w2l[2], w2l[3]);
        }
      }
    }
    if (p.E > 1 && live) {
      dg *= ca;
      uint32_t packed[8];
      float prev = 0.f;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        float d = 0.f;
        if (e < p.E) {
          d = dg * g * ((e == t.it.y ? 1.0f : 0.0f) - p.probs[(long long)pos * p.E + e]);
          p.dl[(long long)pos * p.E + e] = d;
        }
        if (e & 1) packed[e >> 1] = pack_bf16x2(prev * inv_cc, d * inv_cc);
        prev = d;
      }
      uint4* o = reinterpret_cast<uint4*>(p.dlc + (long long)pos * 16);
      o[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
      o[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
    }
  }
};

PQ_DEFINE_GEMM_KERNEL(k_gemm_hp_dh, HpDhProblem)

// ---------------------------------------------------------------------------
// B2: dX tile = c * ( dYs . Sb  +  sum_items dhc . A_e  +  dlc . Wr ), rows
// scattered back to token order.
// ---------------------------------------------------------------------------
struct BwdDxProblem {
  using Acc = AccDouble;
  struct Params {
    CUtensorMap tdy, tsb, tdh, ta3, tdl, twr;
    RoutingTables rt;
    const int* perm;
    const float* w_scales;
    const float* beta;
    uint16_t* dX;
    TileGrid g;
    int T, N, K, r, E, sstride, item_rows, sb_blk, a3_blk, wr_blk;
  };
  struct Tile { TileCoord c; int m, bn, ib, ie, skip1; };
  __device__ static int num_tiles(const Params& p) { return p.g.total; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) {
    t.c = tile_coord(p.g, i);
    t.m = t.c.m;
    t.bn = clip_bn(t.c.bn, t.c.n0, p.K, 64);
    if (p.r > 0) { t.ib = p.rt.tile_item_begin[t.m]; t.ie = p.rt.tile_item_begin[t.m + 1]; } else { t.ib = t.ie = 0; }
    t.skip1 = dx_scale(p.w_scales, p.beta, p.sstride) == 0.f;
  }
  __device__ static int num_segments(const Params& p, const Tile& t) { return (t.skip1 ? 0 : 1) + 2 * (t.ie - t.ib) + (p.E > 1 ? 1 : 0); }
  __device__ static void segment(const Params& p, const Tile& t, int i, Segment& s) {
    s.mode = MODE_BF_KM; s.acc = 0; s.bn = t.bn; s.ksteps = 4; s.a_rank = 2; s.a_x = 0; s.a_z = 0;
    s.b_x = t.c.n0; s.b_y = 0; s.b_z = 0; s.b_box = 0; s.a_blk = 0;
    if (!t.skip1) {
      if (i == 0) {
        s.nkb = (p.N + 63) / 64;
        s.ta = &p.tdy; s.a_y = t.m * 128;
        s.tb = &p.tsb; s.b_rank = 2; s.b_blk = p.sb_blk;
        return;
      }
      --i;
    }
    if (i < 2 * (t.ie - t.ib)) {
      const int item = t.ib + (i >> 1), plane = i & 1;
      s.nkb = (p.r + 63) / 64;
      s.ta = &p.tdh; s.a_y = plane * p.item_rows + item * 128;
      s.tb = &p.ta3; s.b_rank = 3; s.b_z = p.rt.items[item].y; s.b_blk = p.a3_blk;
      return;
    }
    s.nkb = 1; s.ksteps = 1;
    s.ta = &p.tdl; s.a_y = t.m * 128;
    s.tb = &p.twr; s.b_rank = 2; s.b_blk = p.wr_blk;
  }
  struct Pre { uint16_t* xrow; float cc; };
  __device__ static Pre prepare(const Params& p, const Tile& t, int quad, int lane) {
    const int pos = t.m * 128 + quad * 32 + lane;
    const float c = dx_scale(p.w_scales, p.beta, p.sstride);
    Pre r{nullptr, c != 0.f ? c : 1.0f};
    if (pos < p.T) r.xrow = p.dX + (long long)(p.perm ? p.perm[pos] : pos) * p.K;
    return r;
  }
  __device__ static void epilogue(const Params& p, const Tile& t, const Pre& pre, uint32_t taddr, uint32_t, int quad, int half, int lane, uint8_t* stage) {
    const float cc = pre.cc;
    const bool has = num_segments(p, t) > 0;
    for (int c64 = half; c64 * 64 < t.bn; c64 += 2) {
      const int k0 = t.c.n0 + c64 * 64;
      if (k0 >= p.K) break;
      uint32_t v0[32], v1[32];
      tmem_ld32(taddr + c64 * 64, v0);
      tmem_ld32(taddr + c64 * 64 + 32, v1);
      tmem_ld_wait();
      uint4 o[8];
      uint32_t w[32];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        w[j] = has ? pack_bf16x2(cc * __uint_as_float(v0[2 * j]), cc * __uint_as_float(v0[2 * j + 1])) : 0u;
        w[16 + j] = has ? pack_bf16x2(cc * __uint_as_float(v1[2 * j]), cc * __uint_as_float(v1[2 * j + 1])) : 0u;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) o[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
      warp_store_rows(stage, o, pre.xrow ? pre.xrow + k0 : nullptr, min(64, p.K - k0) * 2, lane);
    }
  }
};
PQ_DEFINE_GEMM_KERNEL(k_gemm_bwd_dx, BwdDxProblem)

// ---------------------------------------------------------------------------
// B3: the two products that contract dYs^T over tokens, in one launch.
//   dW tiles: G = dYs^T . xt; dW = beta_n G; per-tile partial of dbeta_n = lam * sum_k S[n,k] G[n,k].
//   dB tiles (one per expert and 128 output features, after the dW tiles): dBraw_e = dYs^T . (g H) over
//     the expert's items, the hi and lo planes of g H side by side as the two halves of the tile's
//     columns; dB = alpha_n dBraw, and the partial of dalpha_n = sum_j B[e,n,j] dBraw[n,j].
//   router tiles (one per 256 columns of K): dWr = c * (dl / c)^T . Xs, the logit gradient in the
//     bf16 form the dX tile also uses, rows >= E of the tile unused (Sec. 3.3, "trained end-to-end").
//   dA tiles (one per expert and 256 columns of K): dA_e = c * (dH / c)^T . Xs over the expert's items, with the
//     leading bf16 plane of dH / c (its 2^-9 rounding averages out over the tokens of the sum).
// ---------------------------------------------------------------------------
struct BwdDwProblem {
  using Acc = AccDouble;
  enum Kind : int { KIND_DW = 0, KIND_DB = 1, KIND_DWR = 2, KIND_DA = 3 };
  struct Params {
    CUtensorMap tdyT, txt, tgh, tdlT, txs, tdhT;
    RoutingTables rt;
    const int8_t* s8;
    const float* beta;
    const float* alpha;
    const float* w_scales;
    float* dWr;              // [E, K]
    float* dA;               // [E, r, K]
    const uint16_t* B;       // [E, N, r]
    float* dW;
    float* dB;               // [E, N, r]
    float* dbeta_partial;    // [2 * ceil(K/256), N]
    float* dalpha_partial;   // [2 * E, N]
    TileGrid g;
    int T, N, K, r, r64, E, sstride, dy_blk, xt_blk, gh_blk, xs_blk, dh_blk, item_rows, ntn, ntk, db_tiles, wr_tiles, da_tiles;
  };
  struct Tile { TileCoord c; int kind, nt, bn, e, ib, ie; };
  __device__ static int num_tiles(const Params& p) { return p.wr_tiles + p.da_tiles + p.g.total + p.db_tiles; }
  // order: the tiles whose contraction runs over all tokens first (router, dA with one expert, dW), the short ones last
  __device__ static void tile_init(const Params& p, int i, Tile& t) {
    t.ib = t.ie = 0; t.e = 0; t.nt = 0;
    if (i < p.wr_tiles) {
      t.kind = KIND_DWR;
      t.c.m = 0; t.c.n0 = i * 256; t.c.bn = 256;
      t.bn = clip_bn(256, t.c.n0, p.K, 64);
      return;
    }
    i -= p.wr_tiles;
    if (i < p.da_tiles) {
      t.kind = KIND_DA;
      t.e = i / p.ntk;
      t.ib = p.rt.expert_item_begin[t.e]; t.ie = p.rt.expert_item_begin[t.e + 1];
      t.c.m = 0; t.c.n0 = (i % p.ntk) * 256; t.c.bn = 256;
      t.bn = clip_bn(256, t.c.n0, p.K, 64);
      return;
    }
    i -= p.da_tiles;
    if (i < p.g.total) {
      t.kind = KIND_DW;
      t.c = tile_coord(p.g, i);
      t.nt = t.c.m;
      t.bn = clip_bn(t.c.bn, t.c.n0, p.K, 64);
      return;
    }
    i -= p.g.total;
    t.kind = KIND_DB;
    t.e = i / p.ntn; t.nt = i % p.ntn;
    t.ib = p.rt.expert_item_begin[t.e]; t.ie = p.rt.expert_item_begin[t.e + 1];
    t.bn = 2 * p.r64;
    t.c.m = t.nt; t.c.n0 = 0; t.c.bn = t.bn;
  }
  __device__ static int num_segments(const Params&, const Tile& t) { return (t.kind == KIND_DW || t.kind == KIND_DWR) ? 1 : t.ie - t.ib; }
  __device__ static void segment(const Params& p, const Tile& t, int i, Segment& s) {
    s.mode = MODE_BF_MM; s.acc = 0; s.bn = t.bn; s.ksteps = 4; s.b_box = 0;
    s.a_rank = 2; s.a_z = 0; s.b_rank = 2; s.b_z = 0;
    switch (t.kind) {
      case KIND_DW:
        s.nkb = (p.T + 63) / 64;
        s.ta = &p.tdyT; s.a_x = t.nt * 128; s.a_y = 0; s.a_blk = p.dy_blk;
        s.tb = &p.txt; s.b_x = t.c.n0; s.b_y = 0; s.b_blk = p.xt_blk;
        break;
      case KIND_DWR:
        s.nkb = (p.T + 63) / 64;
        s.ta = &p.tdlT; s.a_x = 0; s.a_y = 0; s.a_blk = 0;          // 16 columns: plain boxes, zero beyond
        s.tb = &p.txs; s.b_x = t.c.n0; s.b_y = 0; s.b_blk = p.xs_blk;
        break;
      case KIND_DB: {
        const int item = t.ib + i;
        s.nkb = 2;                                        // the 128 tokens of the item's tile (rows outside the item are zero in g H)
        s.ta = &p.tdyT; s.a_x = t.nt * 128; s.a_y = p.rt.items[item].x * 128; s.a_blk = p.dy_blk;
        s.tb = &p.tgh; s.b_x = 0; s.b_y = item * 128; s.b2_y = p.item_rows + item * 128; s.b_blk = p.gh_blk;
        break;
      }
      default: {                                          // KIND_DA: (dH / c)^T . Xs over the expert's items, leading plane of dH / c
        const int item = t.ib + i;
        s.nkb = 2;
        s.ta = &p.tdhT; s.a_x = 0; s.a_y = item * 128; s.a_blk = p.dh_blk;
        s.tb = &p.txs; s.b_x = t.c.n0; s.b_y = p.rt.items[item].x * 128; s.b_blk = p.xs_blk;
        break;
      }
    }
  }
  using Pre = NoPre;
  __device__ static Pre prepare(const Params&, const Tile&, int, int) { return Pre{}; }
  __device__ static void epilogue(const Params& p, const Tile& t, const Pre& pre, uint32_t taddr, uint32_t, int quad, int half, int lane, uint8_t* stage) {
    if (t.kind == KIND_DWR || t.kind == KIND_DA) {
      // ---- router tile: row j < E of the accumulator is dWr[j, :] / c;  dA tile: row j < r is dA[e, j, :] / c
      const int j = quad * 32 + lane;
      const float c = dx_scale(p.w_scales, p.beta, p.sstride);
      const float cc = c != 0.f ? c : 1.0f;
      const bool any = t.kind == KIND_DWR || t.ie > t.ib;    // an expert without tokens: exact zeros
      float* out = nullptr;
      if (t.kind == KIND_DWR) { if (j < p.E) out = p.dWr + (long long)j * p.K; }
      else if (j < p.r) out = p.dA + ((long long)t.e * p.r + j) * p.K;
      for (int c32 = half; c32 * 32 < t.bn; c32 += 2) {
        const int k0 = t.c.n0 + c32 * 32;
        if (k0 >= p.K) break;
        uint32_t v[32];
        if (any) {
          tmem_ld32(taddr + c32 * 32, v);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int u = 0; u < 32; ++u) v[u] = 0u;
        }
        uint4 o[8];
#pragma unroll
        for (int q4 = 0; q4 < 8; ++q4)
          o[q4] = make_uint4(__float_as_uint(cc * __uint_as_float(v[4 * q4])), __float_as_uint(cc * __uint_as_float(v[4 * q4 + 1])),
                             __float_as_uint(cc * __uint_as_float(v[4 * q4 + 2])), __float_as_uint(cc * __uint_as_float(v[4 * q4 + 3])));
        warp_store_rows(stage, o, out ? out + k0 : nullptr, min(32, p.K - k0) * 4, lane);
      }
      return;
    }
    const int n = t.nt * 128 + quad * 32 + lane;
    const bool live = n < p.N;
    if (t.kind == KIND_DB) {
      // ---- dB tile: columns [0, r64) hold the hi-plane product, [r64, 2 r64) the lo-plane product
      const bool any = t.ie > t.ib;                     // an expert without tokens: exact zeros
      const float al = live ? p.alpha[n * p.sstride] : 0.f;
      const long long row = ((long long)t.e * p.N + (live ? n : 0)) * p.r;
      float part = 0.f;
      for (int c32 = half; c32 * 32 < p.r; c32 += 2) {
        uint32_t vh[32], vl[32];
        if (any) {
          tmem_ld32(taddr + c32 * 32, vh);
          tmem_ld32(taddr + p.r64 + c32 * 32, vl);
          tmem_ld_wait();
        }
        uint4 o[8];
#pragma unroll
        for (int q4 = 0; q4 < 8; ++q4) {
          float gsum[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) gsum[u] = any ? __uint_as_float(vh[4 * q4 + u]) + __uint_as_float(vl[4 * q4 + u]) : 0.f;
          const int j = c32 * 32 + q4 * 4;
          if (live && j < p.r) {
            const uint2 bv = *reinterpret_cast<const uint2*>(p.B + row + j);
            part = fmaf(bf16lo(bv.x), gsum[0], part); part = fmaf(bf16hi(bv.x), gsum[1], part);
            part = fmaf(bf16lo(bv.y), gsum[2], part); part = fmaf(bf16hi(bv.y), gsum[3], part);
          }
          o[q4] = make_uint4(__float_as_uint(al * gsum[0]), __float_as_uint(al * gsum[1]), __float_as_uint(al * gsum[2]),
                             __float_as_uint(al * gsum[3]));
        }
        warp_store_rows(stage, o, live ? p.dB + row + c32 * 32 : nullptr, min(32, p.r - c32 * 32) * 4, lane);
      }
      if (live) p.dalpha_partial[(long long)(2 * t.e + half) * p.N + n] = part;
      return;
    }
    const float be = live ? p.beta[n * p.sstride] : 0.f;
    float* wrow = live ? p.dW + (long long)n * p.K : nullptr;
    const uint4* srow = reinterpret_cast<const uint4*>(p.s8 + (long long)(live ? n : 0) * p.K);
    float part = 0.f;
    for (int c32 = half; c32 * 32 < t.bn; c32 += 2) {
      const int k0 = t.c.n0 + c32 * 32;
      if (k0 >= p.K) break;
      uint32_t v[32];
      tmem_ld32(taddr + c32 * 32, v);
      tmem_ld_wait();
      uint4 o[8];
      uint32_t sw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      if (live) {
        const uint4 s0 = __ldg(srow + (k0 >> 4)), s1 = __ldg(srow + (k0 >> 4) + 1);
        sw[0] = s0.x; sw[1] = s0.y; sw[2] = s0.z; sw[3] = s0.w; sw[4] = s1.x; sw[5] = s1.y; sw[6] = s1.z; sw[7] = s1.w;
      }
#pragma unroll
      for (int q4 = 0; q4 < 8; ++q4) {
        const float g0 = __uint_as_float(v[q4 * 4]), g1 = __uint_as_float(v[q4 * 4 + 1]);
        const float g2 = __uint_as_float(v[q4 * 4 + 2]), g3 = __uint_as_float(v[q4 * 4 + 3]);
        const uint32_t sb = sw[q4];  // four +-1 bytes: bit 7 set <-> -1
        part += (sb & 0x80u) ? -g0 : g0;
        part += (sb & 0x8000u) ? -g1 : g1;
        part += (sb & 0x800000u) ? -g2 : g2;
        part += (sb & 0x80000000u) ? -g3 : g3;
        o[q4] = make_uint4(__float_as_uint(be * g0), __float_as_uint(be * g1), __float_as_uint(be * g2), __float_as_uint(be * g3));
      }
      warp_store_rows(stage, o, wrow ? wrow + k0 : nullptr, 128, lane);
    }
    // one slot per (column tile, warp of the row pair)
    if (live) p.dbeta_partial[(long long)(2 * (t.c.n0 / 256) + half) * p.N + n] = part;
  }
};
PQ_DEFINE_GEMM_KERNEL(k_gemm_bwd_dw, BwdDwProblem)

int gemm_backward(const LayerArgs& a, const int8_t* w_s8, const SavedPtrs& sv, const BwdBuffers& b, uint16_t* dX, float* dW, float* dA,
                  float* dB, float* dWr, cudaStream_t st, const BwdStreams& bs) {
  const int mtiles = (a.T + 127) / 128;
  const int ntk = (a.K + 255) / 256, ntn128 = (a.N + 127) / 128;
  const bool hp = a.r > 0;
  const int r64 = h_round_up(a.r, 64);
  const uint64_t item_rows = (uint64_t)sv.max_items * 128;  // rows of one plane; buffers hold two
  cudaStream_t sx = bs.side ? bs.side : st;                 // stream of the HP gradient GEMM and dX
  int rc;

  BwdDwProblem::Params w;
  {
    if (!map_mn(&w.tdyT, &w.dy_blk, b.dys, a.N, a.T, 2, 1, 2)) return PQ_ERR_CUDA;
    if (!map_mn(&w.txt, &w.xt_blk, sv.xt, a.K, a.T, 2, 1, 4)) return PQ_ERR_CUDA;
    w.tgh = w.txt; w.gh_blk = 0;
    if (hp && !map_mn(&w.tgh, &w.gh_blk, b.gh, a.r, 2 * item_rows, 2, 1, r64 / 64)) return PQ_ERR_CUDA;
    w.rt = sv.rt; w.s8 = w_s8; w.beta = a.beta; w.alpha = a.alpha; w.B = a.B; w.dW = dW; w.dB = dB;
    w.dbeta_partial = b.dbeta_partial; w.dalpha_partial = b.dalpha_partial;
    w.T = a.T; w.N = a.N; w.K = a.K; w.r = a.r; w.r64 = r64; w.E = a.E; w.sstride = a.scale_stride; w.item_rows = (int)item_rows;
    w.ntn = ntn128; w.ntk = ntk; w.db_tiles = hp ? a.E * ntn128 : 0; w.da_tiles = hp ? a.E * ntk : 0;
    w.tdlT = w.txt; w.txs = w.txt; w.tdhT = w.txt; w.xs_blk = 0; w.dh_blk = 0; w.wr_tiles = 0;
    w.w_scales = a.w_scales; w.dWr = dWr; w.dA = dA;
    if (hp) {
      if (!map_mn(&w.txs, &w.xs_blk, b.xs, a.K, a.T, 2, 1, 4)) return PQ_ERR_CUDA;
      if (!map_mn(&w.tdhT, &w.dh_blk, b.dhc, a.r, 2 * item_rows, 2, 1, 2)) return PQ_ERR_CUDA;
    }
    if (hp && a.E > 1) {
      int unused = 0;
      if (!map_mn(&w.tdlT, &unused, b.dlc, 16, a.T, 2, 1, 2)) return PQ_ERR_CUDA;
      w.wr_tiles = ntk;
    }
    w.g = make_tile_grid(ntn128, ntk, 256);
  }
  if (bs.side) {
    // the dW tiles proper need dY and q / gamma only: they start at once and take every SM; what follows on the
    // other stream moves into their last wave
    BwdDwProblem::Params m = w;
    m.wr_tiles = 0; m.da_tiles = 0; m.db_tiles = 0;
    rc = launch_gemm(KID_BWD_DW, k_gemm_bwd_dw, m, m.g.total, st);
    if (rc) return rc;
  }
  if (hp) {
    HpDhProblem::Params p;
    if (!map2d(&p.tdy, false, b.dys, a.N, a.T, 64, 128)) return PQ_ERR_CUDA;
    if (!map_mn(&p.tba, &p.ba_blk, b.ba, a.r, a.N, 3, a.E, r64 / 64)) return PQ_ERR_CUDA;
    p.rt = sv.rt; p.H = sv.h; p.gate = sv.gate; p.probs = sv.probs; p.w_scales = a.w_scales; p.alpha = a.alpha; p.beta = a.beta;
    p.dhc = b.dhc; p.gh = b.gh; p.dl = b.dl; p.dlc = b.dlc;
    p.T = a.T; p.N = a.N; p.r = a.r; p.E = a.E; p.bn = r64; p.sstride = a.scale_stride; p.item_rows = (int)item_rows;
    rc = launch_gemm(KID_HP_DH, k_gemm_hp_dh, p, sv.max_items, sx);
    if (rc) return rc;
    if (bs.side && cudaEventRecord(bs.dh_done, sx) != cudaSuccess) return PQ_ERR_CUDA;
  }
  {
    BwdDxProblem::Params p;
    if (!map2d(&p.tdy, false, b.dys, a.N, a.T, 64, 128)) return PQ_ERR_CUDA;
    if (!map_mn(&p.tsb, &p.sb_blk, b.sb, a.K, a.N, 2, 1, 4)) return PQ_ERR_CUDA;
    p.tdh = p.tdy; p.ta3 = p.tdy; p.tdl = p.tdy; p.twr = p.tdy; p.a3_blk = 0; p.wr_blk = 0;
    if (hp) {
      if (!map2d(&p.tdh, false, b.dhc, a.r, 2 * item_rows, 64, 128)) return PQ_ERR_CUDA;
      if (!map_mn(&p.ta3, &p.a3_blk, a.A, a.K, a.r, 3, a.E, 4)) return PQ_ERR_CUDA;
    }
    if (hp && a.E > 1) {
      if (!map2d(&p.tdl, false, b.dlc, 16, a.T, 64, 128)) return PQ_ERR_CUDA;
      if (!map_mn(&p.twr, &p.wr_blk, a.Wr, a.K, a.E, 2, 1, 4)) return PQ_ERR_CUDA;
    }
    p.rt = sv.rt; p.perm = (hp && a.E > 1) ? sv.perm : nullptr; p.w_scales = a.w_scales; p.beta = a.beta; p.dX = dX;
    p.T = a.T; p.N = a.N; p.K = a.K; p.r = a.r; p.E = hp ? a.E : 1; p.sstride = a.scale_stride; p.item_rows = (int)item_rows;
    p.g = make_tile_grid(mtiles, ntk, 256);
    rc = launch_gemm(KID_BWD_DX, k_gemm_bwd_dx, p, p.g.total, sx);
    if (rc) return rc;
    if (bs.side && cudaEventRecord(bs.side_done, sx) != cudaSuccess) return PQ_ERR_CUDA;
  }
  if (!bs.side) {
    rc = launch_gemm(KID_BWD_DW, k_gemm_bwd_dw, w, w.wr_tiles + w.da_tiles + w.g.total + w.db_tiles, st);
    if (rc) return rc;
  } else {
    if (hp) {
      // dB, dA and the router gradient read what the HP gradient GEMM wrote
      BwdDwProblem::Params x = w;
      x.g.total = 0;
      if (cudaStreamWaitEvent(st, bs.dh_done, 0) != cudaSuccess) return PQ_ERR_CUDA;
      rc = launch_gemm(KID_HP_DB, k_gemm_bwd_dw, x, x.wr_tiles + x.da_tiles + x.db_tiles, st);
      if (rc) return rc;
    }
    if (cudaStreamWaitEvent(st, bs.side_done, 0) != cudaSuccess) return PQ_ERR_CUDA;
  }
  return PQ_OK;
}

}  // namespace pq
