// Persistent, warp-specialised tcgen05 GEMM engine for sm_100a.
//
// One CTA per SM, 320 threads: warp 0 = TMA producer, warp 1 = MMA issuer
// (also owns the TMEM allocation), warps 2-9 = epilogue (two per TMEM lane
// quadrant, which take alternate column chunks of the tile).  Operands travel global -> shared by TMA into a ring (4 stages of 48 KB; more, smaller ones for narrow tiles) of
// 128-byte-swizzled tiles; tcgen05.mma accumulates 128 x (<=256) tiles in
// TMEM; the epilogue reads them back with tcgen05.ld.
//
// A tile's contraction is a list of SEGMENTS.  Each segment names its operand
// form (int8 or bf16; each operand either contraction-contiguous "K" or
// output-dimension-contiguous "MN"), its tensor maps and start coordinates,
// the number of 128-byte k-blocks, and which of the tile's accumulators it
// adds into.  This lets one kernel chain, e.g., the int8 1-bit product, the
// bf16 expert product and the router product of one output tile.
//
// A "Problem" type supplies the tile list, the segments and the epilogue.
#pragma once
#include <cuda.h>

#include <type_traits>

#include "pq_common.cuh"

namespace pq {

constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr int kMaxStages = 8;             // barrier pairs reserved for the operand ring
constexpr int kTileM = 128;
constexpr int kStageABytes = 128 * 128;  // 128 rows x 128 B, or two 64x64 bf16 MN boxes
constexpr int kStageBBytes = 256 * 128;  // up to 256 rows x 128 B, or four MN boxes
constexpr int kRingBytes = 4 * (kStageABytes + kStageBBytes);   // operand ring: four stages of a 256-column tile
constexpr int kMnBoxBytes = 64 * 128;    // one MN-major box: 64 k-rows of 64 bf16
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;            // TMEM columns of one accumulator stage in the default layout
constexpr int kEpiWarpBytes = 32 * 128;                // per epilogue warp: 32 rows of one 128-byte chunk (xor-swizzled)
constexpr int kGemmSmemBytes = kRingBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kEpiWarps * kEpiWarpBytes;
static_assert(kGemmSmemBytes <= 227 * 1024, "shared memory of one CTA");

enum OpMode : int {
  MODE_I8_KK = 0,  // int8, A[M,K] and B[N,K] K-contiguous
  MODE_BF_KK = 1,  // bf16, both K-contiguous
  MODE_BF_KM = 2,  // bf16, A K-contiguous, B N-contiguous
  MODE_BF_MM = 3   // bf16, A M-contiguous, B N-contiguous
};

struct Segment {
  int mode;                 // OpMode
  int acc;                  // accumulator of the tile this segment adds into
  int nkb;                  // k-blocks (128 bytes of K each: 128 int8 / 64 bf16)
  int bn;                   // UMMA N for this segment (multiple of 16, <= 256; MN-major B: multiple of 64)
  int ksteps;               // UMMA k-steps issued per k-block (1..4)
  const CUtensorMap* ta;
  const CUtensorMap* tb;
  int a_x, a_y, a_z;        // K operand: (k0, row0, z);  MN operand: (mn0, k0, z)
  int b_x, b_y, b_z;
  int a_rank, b_rank;       // tensor-map rank (2 or 3)
  int b_box;                // K-major B: rows one TMA load delivers (box height of tb); bn is covered by
                            // ceil(bn / b_box) loads.  Per k-block B always occupies bn * 128 bytes.
  int b2_y;                 // MN-major B only, -1 = unused: the columns [bn/2, bn) of B come from a second row range of
                            // tb starting at k row b2_y (same columns b_x), e.g. the second bf16 plane of an operand
  int a_blk, b_blk;         // MN-major operand read through a "blocked" tensor map (64-wide column blocks as an
                            // extra dimension): number of blocks one load delivers; 0 = one 64 x 64 box per load
};

// Output tiles are 128 rows x `bn` columns, the cells of an (mt x nt) grid walked row by row.
struct TileGrid {
  int mt, nt, bn, total;
};
__host__ inline TileGrid make_tile_grid(int mt, int nt, int bn) { return TileGrid{mt, nt, bn, mt * nt}; }
struct TileCoord { int m, n0, bn; };
__device__ __forceinline__ TileCoord tile_coord(const TileGrid& g, int i) {
  return TileCoord{i / g.nt, (i % g.nt) * g.bn, g.bn};
}

__device__ __forceinline__ bool a_is_mn(int mode) { return mode == MODE_BF_MM; }
__device__ __forceinline__ bool b_is_mn(int mode) { return mode >= MODE_BF_KM; }


__device__ __forceinline__ void tma_fetch(uint32_t dst, const CUtensorMap* t, uint32_t bar, int rank, int x, int y, int z) {
  if (rank == 3) tma_load_3d(dst, t, bar, x, y, z);
  else tma_load_2d(dst, t, bar, x, y);
}
// Blocked view of an MN-major operand: dimensions (64 columns of a block, k row, block index[, batch]).
__device__ __forceinline__ void tma_fetch_blocked(uint32_t dst, const CUtensorMap* t, uint32_t bar, int base_rank, int k, int blk, int z) {
  if (base_rank == 3) tma_load_4d(dst, t, bar, 0, k, blk, z);
  else tma_load_3d(dst, t, bar, 0, k, blk);
}

struct PipeState {
  int stage = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void advance(int n) {
    if (++stage == n) { stage = 0; phase ^= 1; }
  }
};

// Bounded wait that also gives up when another role of this CTA has failed.
__device__ __forceinline__ bool pipe_wait(uint32_t bar, uint32_t parity, int where, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > c_spin_cycles) {
      report_timeout(where);
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}

// Coalescing store for epilogues.  Each lane holds 128 contiguous bytes (8 x 16 B) of ITS OWN output
// row, and rows may live anywhere in global memory (row_ptr = 0 skips the row).  The warp transposes
// through its staging buffer so that every store instruction writes 4 rows x 128 contiguous bytes
// instead of 32 rows x 16 bytes.  Only the first valid_bytes of each row are written.  The 16-byte
// piece j of row r sits at position j ^ (r & 7) of the row, which keeps both passes free of bank conflicts.
__device__ __forceinline__ void warp_store_rows(uint8_t* stage, const uint4 (&v)[8], void* row_ptr, int valid_bytes, int lane) {
  uint4* mine = reinterpret_cast<uint4*>(stage + lane * 128);
#pragma unroll
  for (int j = 0; j < 8; ++j) mine[j ^ (lane & 7)] = v[j];
  __syncwarp();
  const unsigned long long my = reinterpret_cast<unsigned long long>(row_ptr);
  const int c = lane & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = 4 * i + (lane >> 3);
    const unsigned long long dst = __shfl_sync(0xffffffffu, my, row);
    const uint4 val = *reinterpret_cast<const uint4*>(stage + row * 128 + ((c ^ (row & 7)) << 4));
    if (dst != 0ull && c * 16 < valid_bytes) *reinterpret_cast<uint4*>(dst + c * 16) = val;
  }
  __syncwarp();
}

// Problems whose epilogue needs nothing fetched ahead of the accumulator
struct NoPre {};

// Widest B operand of a launch, in tile columns (B takes that many x 128 bytes of a stage): the ring holds as many
// stages as fit, so a launch of narrow tiles keeps more k-blocks in flight.  Problems without `stage_cols` use 256.
template <class P, class = void>
struct stage_cols_of {
  __device__ static int get(const typename P::Params&) { return 256; }
};
template <class P>
struct stage_cols_of<P, std::void_t<decltype(&P::stage_cols)>> {
  __device__ static int get(const typename P::Params& p) { return P::stage_cols(p); }
};

// Accumulator layouts in TMEM (column of accumulator `acc` of pipeline stage `stage`).
//   AccDouble     : one accumulator per tile, two stages of 256 columns.
//   AccPair       : two accumulators of 256 columns per tile (all of TMEM), one stage: the epilogue of
//                   a tile does not overlap the next tile's contraction.
struct AccDouble {
  static constexpr int kStages = 2;
  __device__ static uint32_t col(int stage, int /*acc*/) { return stage * kAccCols; }
};
struct AccPair {
  static constexpr int kStages = 1;
  __device__ static uint32_t col(int /*stage*/, int acc) { return acc * kAccCols; }
};

template <class P>
__device__ __forceinline__ void gemm_body(const typename P::Params& p) {
  extern __shared__ uint8_t smem_raw[];
  using Acc = typename P::Acc;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t kStageBytes = kStageABytes + (uint32_t)stage_cols_of<P>::get(p) * 128u;   // a multiple of 1024
  const int kStages = min(kMaxStages, (int)(kRingBytes / kStageBytes));
  const uint32_t bar_base = smem_base + kRingBytes;
  // barrier block: full[8] empty[8] tfull[2] tempty[2] (8 B each), then tmem ptr, abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + s); };
  auto tempty_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 2 + s); };
  uint8_t* bar_generic = smem_raw + (bar_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(bar_generic + 8 * (2 * kMaxStages + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_generic + 8 * (2 * kMaxStages + 5) + 8);
  uint8_t* epi_stage = bar_generic + 256;  // kEpiWarps x kEpiWarpBytes

  constexpr int kAccStages = Acc::kStages;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(tfull_bar(s), 1); mbar_init(tempty_bar(s), kEpiWarps); }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_holder)), kTmemCols);
    tmem_relinquish();
  }
  // Launched with programmatic stream serialisation: the next kernel's CTAs may start (and do their own set-up)
  // while this one's last tiles run; nothing of global memory is touched before the previous kernel has finished.
  pdl_launch_dependents();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  const uint32_t tmem_base = *tmem_holder;
  const int ntiles = P::num_tiles(p);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      PipeState st;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
        typename P::Tile t;
        P::tile_init(p, tile, t);
        const int nseg = P::num_segments(p, t);
        for (int s = 0; ok && s < nseg; ++s) {
          Segment sg;
          sg.b2_y = -1;
          P::segment(p, t, s, sg);
          const int a_step = (sg.mode == MODE_I8_KK) ? 128 : 64;
          // both operands of k-block kb into the stage at sa
          auto fetch = [&](int kb, uint32_t sa, uint32_t bar) {
            const uint32_t sb = sa + kStageABytes;
            if (a_is_mn(sg.mode)) {
              if (sg.a_blk) {
                tma_fetch_blocked(sa, sg.ta, bar, sg.a_rank, sg.a_y + kb * 64, sg.a_x >> 6, sg.a_z);
              } else {
                tma_fetch(sa, sg.ta, bar, sg.a_rank, sg.a_x, sg.a_y + kb * 64, sg.a_z);
                tma_fetch(sa + kMnBoxBytes, sg.ta, bar, sg.a_rank, sg.a_x + 64, sg.a_y + kb * 64, sg.a_z);
              }
            } else {
              tma_fetch(sa, sg.ta, bar, sg.a_rank, sg.a_x + kb * a_step, sg.a_y, sg.a_z);
            }
            if (b_is_mn(sg.mode)) {
              const int parts = sg.b2_y >= 0 ? 2 : 1;
              for (int part = 0; part < parts; ++part) {
                const int krow = (part ? sg.b2_y : sg.b_y) + kb * 64;
                if (sg.b_blk) {
                  tma_fetch_blocked(sb + part * sg.b_blk * kMnBoxBytes, sg.tb, bar, sg.b_rank, krow, sg.b_x >> 6, sg.b_z);
                } else {
                  const int nbox = sg.bn / (64 * parts);
                  for (int b = 0; b < nbox; ++b)
                    tma_fetch(sb + (part * nbox + b) * kMnBoxBytes, sg.tb, bar, sg.b_rank, sg.b_x + 64 * b, krow, sg.b_z);
                }
              }
            } else {
              for (int row = 0; row < sg.bn; row += sg.b_box)
                tma_fetch(sb + row * 128, sg.tb, bar, sg.b_rank, sg.b_x + kb * a_step, sg.b_y + row, sg.b_z);
            }
          };
          for (int kb = 0; kb < sg.nkb; ++kb) {
            if (!pipe_wait(empty_bar(st.stage), st.phase ^ 1, WHERE_PRODUCER, abort_flag)) { ok = false; break; }
            const uint32_t bar = full_bar(st.stage);
            const uint32_t sa = smem_base + st.stage * kStageBytes;
            if (b_is_mn(sg.mode)) {
              mbar_expect_tx(bar, kStageABytes + (sg.b_blk ? (sg.b2_y >= 0 ? 2 : 1) * sg.b_blk * kMnBoxBytes : sg.bn * 128));
            } else {
              const int nload = (sg.bn + sg.b_box - 1) / sg.b_box;
              mbar_expect_tx(bar, kStageABytes + nload * sg.b_box * 128);
            }
            fetch(kb, sa, bar);
            st.advance(kStages);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      PipeState st, ac;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
        typename P::Tile t;
        P::tile_init(p, tile, t);
        const int nseg = P::num_segments(p, t);
        if (!pipe_wait(tempty_bar(ac.stage), ac.phase ^ 1, WHERE_MMA, abort_flag)) { ok = false; break; }
        tc_fence_after();
        uint32_t started[2] = {0u, 0u};
        for (int s = 0; ok && s < nseg; ++s) {
          Segment sg;
          sg.b2_y = -1;
          P::segment(p, t, s, sg);
          const uint32_t d_tmem = tmem_base + Acc::col(ac.stage, sg.acc);
          const bool amn = a_is_mn(sg.mode), bmn = b_is_mn(sg.mode);
          const uint32_t idesc = (sg.mode == MODE_I8_KK) ? umma_idesc(2, 1, 0, 0, sg.bn)
                                                          : umma_idesc(1, 1, amn ? 1 : 0, bmn ? 1 : 0, sg.bn);
          for (int kb = 0; kb < sg.nkb; ++kb) {
            if (!pipe_wait(full_bar(st.stage), st.phase, WHERE_MMA, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = smem_base + st.stage * kStageBytes;
            const uint32_t sb = sa + kStageABytes;
            for (int k = 0; k < sg.ksteps; ++k) {
              const uint64_t ad = amn ? umma_smem_desc(sa + k * 2048, kMnBoxBytes, 1024) : umma_smem_desc(sa + k * 32, 16, 1024);
              const uint64_t bd = bmn ? umma_smem_desc(sb + k * 2048, kMnBoxBytes, 1024) : umma_smem_desc(sb + k * 32, 16, 1024);
              if (sg.mode == MODE_I8_KK) umma_i8(d_tmem, ad, bd, idesc, started[sg.acc]);
              else umma_f16(d_tmem, ad, bd, idesc, started[sg.acc]);
              started[sg.acc] = 1u;
            }
            umma_commit(empty_bar(st.stage));  // frees the smem stage once these MMAs retire
            st.advance(kStages);
          }
        }
        if (ok) umma_commit(tfull_bar(ac.stage));
        ac.advance(kAccStages);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    PipeState ac;
    const int quad = warp & 3;          // TMEM lanes [32*quad, 32*quad+32) are this warp's
    const int half = (warp - 2) >> 2;   // which of the two warps of the quadrant: it takes column chunks half, half+2, ...
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
      typename P::Tile t;
      P::tile_init(p, tile, t);
      // per-row factors and addresses are fetched while the contraction is still running
      const typename P::Pre pre = P::prepare(p, t, quad, lane);
      // Every lane watches the barrier itself, but the warp takes ONE decision: what follows is full of
      // warp-collective instructions (tcgen05.ld, shuffles), so a lane that gave up must take the others along.
      ok = __all_sync(0xffffffffu, pipe_wait(tfull_bar(ac.stage), ac.phase, WHERE_EPILOGUE, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const uint32_t tlane = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
      P::epilogue(p, t, pre, tlane + Acc::col(ac.stage, 0), tlane + Acc::col(ac.stage, 1), quad, half, lane, epi_stage + (warp - 2) * kEpiWarpBytes);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(ac.stage));
      ac.advance(kAccStages);
    }
  }

  __syncthreads();
  if (*abort_flag) {
    // a wait ran out: give copies and MMAs already in flight time to land before the
    // shared memory and TMEM of this CTA are released
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// One named kernel per problem, so that profiler listings show which product ran.
#define PQ_DEFINE_GEMM_KERNEL(name, Problem)                                                      \
  __global__ void __launch_bounds__(kGemmThreads, 1) name(const __grid_constant__ typename Problem::Params p) { \
    gemm_body<Problem>(p);                                                                        \
  }

}  // namespace pq
