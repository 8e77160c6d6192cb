// Tensor-core kernels of the pQuant layer, built on the engine in pq_gemm.cuh:
//   forward  : H = X A_e^T (grouped by expert), then the fused output tile
//              Y = alpha g (H B_e^T) + beta (lam/gamma) (q S^T)      (Eq. 10, 11)
//   backward : dH, dX, dW, dB, dA of the straight-through estimator  (App. B.1)
//   debug    : raw accumulators of one contraction, for bit-exact tests
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
  cuuint64_t gd[3];
  cuuint64_t gs[2];
  cuuint32_t bx[3], es[3];
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

template <class P>
static int launch_gemm(const typename P::Params& p, int max_tiles, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(gemm_kernel<P>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes) != cudaSuccess) return PQ_ERR_CUDA;
    configured = true;
  }
  int grid = max_tiles < sm_count() ? max_tiles : sm_count();
  if (grid < 1) grid = 1;
  gemm_kernel<P><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? PQ_OK : PQ_ERR_CUDA;
}

__device__ __forceinline__ int round_up(int x, int m) { return (x + m - 1) / m * m; }
static inline int h_round_up(int x, int m) { return (x + m - 1) / m * m; }

// ---------------------------------------------------------------------------
// debug: D[M,N] = contraction of A and B in one of the four operand forms
// ---------------------------------------------------------------------------
struct DebugProblem {
  static constexpr int kAccPerTile = 1;
  struct Params {
    CUtensorMap ta, tb;
    int mode, M, N, K, ntn;
    void* D;
  };
  struct Tile { int m, n; };
  __device__ static int num_tiles(const Params& p) { return ((p.M + 127) / 128) * p.ntn; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) { t.m = i / p.ntn; t.n = i % p.ntn; }
  __device__ static int num_segments(const Params&, const Tile&) { return 1; }
  __device__ static void segment(const Params& p, const Tile& t, int, Segment& s) {
    s.mode = p.mode; s.acc = 0; s.bn = 256; s.ksteps = 4;
    const int bk = p.mode == MODE_I8_KK ? 128 : 64;
    s.nkb = (p.K + bk - 1) / bk;
    s.ta = &p.ta; s.tb = &p.tb; s.a_rank = 2; s.b_rank = 2; s.a_z = 0; s.b_z = 0;
    if (p.mode == MODE_BF_MM) { s.a_x = t.m * 128; s.a_y = 0; } else { s.a_x = 0; s.a_y = t.m * 128; }
    if (p.mode >= MODE_BF_KM) { s.b_x = t.n * 256; s.b_y = 0; } else { s.b_x = 0; s.b_y = t.n * 256; }
    s.b_bytes = kStageBBytes;
  }
  __device__ static void epilogue(const Params& p, const Tile& t, uint32_t taddr, int quad, int lane) {
    const int row = t.m * 128 + quad * 32 + lane;
    uint32_t* D = reinterpret_cast<uint32_t*>(p.D);
    for (int c = 0; c < 8; ++c) {
      const int n0 = t.n * 256 + c * 32;
      if (n0 >= p.N) break;
      uint32_t v[32];
      tmem_ld32(taddr + c * 32, v);
      tmem_ld_wait();
      if (row < p.M) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (n0 + j < p.N) D[(long long)row * p.N + n0 + j] = v[j];
      }
    }
  }
};

int gemm_debug(int mode, int M, int N, int K, const void* A, const void* B, void* D, cudaStream_t st) {
  DebugProblem::Params p;
  p.mode = mode; p.M = M; p.N = N; p.K = K; p.D = D; p.ntn = (N + 255) / 256;
  bool ok = true;
  switch (mode) {
    case MODE_I8_KK:
      ok = map2d(&p.ta, true, A, K, M, 128, 128) && map2d(&p.tb, true, B, K, N, 128, 256);
      break;
    case MODE_BF_KK:
      ok = map2d(&p.ta, false, A, K, M, 64, 128) && map2d(&p.tb, false, B, K, N, 64, 256);
      break;
    case MODE_BF_KM:
      ok = map2d(&p.ta, false, A, K, M, 64, 128) && map2d(&p.tb, false, B, N, K, 64, 64);
      break;
    case MODE_BF_MM:
      ok = map2d(&p.ta, false, A, M, K, 64, 64) && map2d(&p.tb, false, B, N, K, 64, 64);
      break;
    default:
      return PQ_ERR_UNSUPPORTED;
  }
  if (!ok) return PQ_ERR_CUDA;
  return launch_gemm<DebugProblem>(p, ((M + 127) / 128) * p.ntn, st);
}

// ---------------------------------------------------------------------------
// F1: hidden activations of the HP branch, H = X_sorted A_e^T, one tile per item
// ---------------------------------------------------------------------------
struct HpUpProblem {
  static constexpr int kAccPerTile = 1;
  struct Params {
    CUtensorMap tx, ta;  // X sorted [T,K]; A [E,r,K]
    RoutingTables rt;
    uint16_t* H;
    int K, r, bn;
  };
  struct Tile { int item; int4 it; };
  __device__ static int num_tiles(const Params& p) { return p.rt.n_items[0]; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) { t.item = i; t.it = p.rt.items[i]; }
  __device__ static int num_segments(const Params&, const Tile&) { return 1; }
  __device__ static void segment(const Params& p, const Tile& t, int, Segment& s) {
    s.mode = MODE_BF_KK; s.acc = 0; s.bn = p.bn; s.ksteps = 4; s.nkb = (p.K + 63) / 64;
    s.ta = &p.tx; s.a_rank = 2; s.a_x = 0; s.a_y = t.it.x * 128; s.a_z = 0;
    s.tb = &p.ta; s.b_rank = 3; s.b_x = 0; s.b_y = 0; s.b_z = t.it.y;
    s.b_bytes = p.bn * 128;
  }
  __device__ static void epilogue(const Params& p, const Tile& t, uint32_t taddr, int quad, int lane) {
    const int row = quad * 32 + lane;
    const bool live = row >= t.it.z && row < t.it.w;
    uint4* out = reinterpret_cast<uint4*>(p.H + ((long long)t.item * 128 + row) * p.r);
    for (int c = 0; c * 32 < p.r; ++c) {
      uint32_t v[32];
      tmem_ld32(taddr + c * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (c * 32 + g * 8 < p.r) {
          uint4 o = make_uint4(0, 0, 0, 0);
          if (live) {
            o.x = pack_bf16x2(__uint_as_float(v[8 * g + 0]), __uint_as_float(v[8 * g + 1]));
            o.y = pack_bf16x2(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]));
            o.z = pack_bf16x2(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]));
            o.w = pack_bf16x2(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]));
          }
          out[c * 4 + g] = o;
        }
      }
    }
  }
};

// ---------------------------------------------------------------------------
// F2: fused output tile.  Accumulator 0 (int32): q S^T over K.  Accumulator 1
// (fp32): H B_e^T over r, once per item of the tile (masked H rows are zero).
// Epilogue: Y[token, n] = alpha_n g z + beta_n (lam / gamma) acc, rounded once.
// ---------------------------------------------------------------------------
template <bool HP>
struct FwdProblem {
  static constexpr int kAccPerTile = HP ? 2 : 1;
  struct Params {
    CUtensorMap tq, ts, th, tb;  // q [T,K] s8; S [N,K] s8; H [items*128,r]; B [E,N,r]
    RoutingTables rt;
    const int* perm;
    const float* gamma;
    const float* gate;
    const float* w_scales;
    const float* alpha;
    const float* beta;
    uint16_t* Y;
    int T, N, K, r, sstride, ntn;
  };
  struct Tile { int m, n, ib, ie; };
  __device__ static int num_tiles(const Params& p) { return ((p.T + 127) / 128) * p.ntn; }
  __device__ static void tile_init(const Params& p, int i, Tile& t) {
    t.m = i / p.ntn; t.n = i % p.ntn;
    if (HP) { t.ib = p.rt.tile_item_begin[t.m]; t.ie = p.rt.tile_item_begin[t.m + 1]; } else { t.ib = t.ie = 0; }
  }
  __device__ static int num_segments(const Params&, const Tile& t) { return 1 + (t.ie - t.ib); }
  __device__ static void segment(const Params& p, const Tile& t, int i, Segment& s) {
    s.bn = 256; s.ksteps = 4; s.a_z = 0; s.b_z = 0; s.b_bytes = kStageBBytes;
    if (i == 0) {
      s.mode = MODE_I8_KK; s.acc = 0; s.nkb = (p.K + 127) / 128;
      s.ta = &p.tq; s.a_rank = 2; s.a_x = 0; s.a_y = t.m * 128;
      s.tb = &p.ts; s.b_rank = 2; s.b_x = 0; s.b_y = t.n * 256;
    } else {
      const int item = t.ib + i - 1;
      const int e = p.rt.items[item].y;
      s.mode = MODE_BF_KK; s.acc = 1; s.nkb = (p.r + 63) / 64;
      s.ta = &p.th; s.a_rank = 2; s.a_x = 0; s.a_y = item * 128;
      s.tb = &p.tb; s.b_rank = 3; s.b_x = 0; s.b_y = t.n * 256; s.b_z = e;
    }
  }
  __device__ static void epilogue(const Params& p, const Tile& t, uint32_t taddr, int quad, int lane) {
    const int pos = t.m * 128 + quad * 32 + lane;
    const bool live = pos < p.T;
    const int token = live ? (p.perm ? p.perm[pos] : pos) : 0;
    const float s1 = live ? __fdiv_rn(p.w_scales[0], p.gamma[pos]) : 0.f;
    const float g = (HP && live) ? p.gate[pos] : 0.f;
    uint4* yrow = reinterpret_cast<uint4*>(p.Y + (long long)token * p.N);
    for (int c = 0; c < 8; ++c) {
      const int n0 = t.n * 256 + c * 32;
      if (n0 >= p.N) break;
      uint32_t a[32], z[32];
      tmem_ld32(taddr + c * 32, a);
      if (HP) tmem_ld32(taddr + kAccCols + c * 32, z);
      tmem_ld_wait();
      if (live) {
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) {
          float y[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int n = n0 + gq * 8 + j;
            const float be = __ldg(p.beta + n * p.sstride);
            float v = be * s1 * (float)(int)a[gq * 8 + j];
            if (HP) v += __ldg(p.alpha + n * p.sstride) * g * __uint_as_float(z[gq * 8 + j]);
            y[j] = v;
          }
          yrow[(n0 >> 3) + gq] = make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
        }
      }
    }
  }
};

int gemm_forward(const LayerArgs& a, const int8_t* w_s8, const SavedPtrs& sv, const uint16_t* xs, uint16_t* Y, cudaStream_t st) {
  const int mtiles = (a.T + 127) / 128;
  const bool hp = a.r > 0;
  if (hp) {
    HpUpProblem::Params p;
    p.rt = sv.rt; p.H = sv.h; p.K = a.K; p.r = a.r; p.bn = h_round_up(a.r, 16);
    if (!map2d(&p.tx, false, xs, a.K, a.T, 64, 128)) return PQ_ERR_CUDA;
    if (!map3d(&p.ta, a.A, a.K, a.r, a.E, 64, p.bn)) return PQ_ERR_CUDA;
    int rc = launch_gemm<HpUpProblem>(p, sv.max_items, st);
    if (rc) return rc;
    FwdProblem<true>::Params f;
    if (!map2d(&f.tq, true, sv.q, a.K, a.T, 128, 128)) return PQ_ERR_CUDA;
    if (!map2d(&f.ts, true, w_s8, a.K, a.N, 128, 256)) return PQ_ERR_CUDA;
    if (!map2d(&f.th, false, sv.h, a.r, (uint64_t)sv.max_items * 128, 64, 128)) return PQ_ERR_CUDA;
    if (!map3d(&f.tb, a.B, a.r, a.N, a.E, 64, 256)) return PQ_ERR_CUDA;
    f.rt = sv.rt; f.perm = a.E > 1 ? sv.perm : nullptr; f.gamma = sv.gamma; f.gate = sv.gate; f.w_scales = a.w_scales;
    f.alpha = a.alpha; f.beta = a.beta; f.Y = Y; f.T = a.T; f.N = a.N; f.K = a.K; f.r = a.r; f.sstride = a.scale_stride;
    f.ntn = (a.N + 255) / 256;
    return launch_gemm<FwdProblem<true>>(f, mtiles * f.ntn, st);
  }
  FwdProblem<false>::Params f;
  if (!map2d(&f.tq, true, sv.q, a.K, a.T, 128, 128)) return PQ_ERR_CUDA;
  if (!map2d(&f.ts, true, w_s8, a.K, a.N, 128, 256)) return PQ_ERR_CUDA;
  f.th = f.tq; f.tb = f.tq;
  f.rt = sv.rt; f.perm = nullptr; f.gamma = sv.gamma; f.gate = sv.gate; f.w_scales = a.w_scales;
  f.alpha = a.alpha; f.beta = a.beta; f.Y = Y; f.T = a.T; f.N = a.N; f.K = a.K; f.r = 0; f.sstride = a.scale_stride;
  f.ntn = (a.N + 255) / 256;
  return launch_gemm<FwdProblem<false>>(f, mtiles * f.ntn, st);
}

}  // namespace pq
