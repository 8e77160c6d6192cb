// Decode path of the pQuant layer (App. A), streaming form: one cooperative kernel per batch of independent
// linears, M <= 16 tokens each, reading weights that were laid out for it once (pq_pack_decode):
//
//   sign bits   [row group g of 128 features][chunk c of 128 contraction values][4][32 lanes][16 bytes]:
//               lane l of a warp owns the features 128 g + 32 f + l, f = 0..3, and a warp reads a chunk as four
//               fully coalesced 512-byte loads; no lane ever needs another lane's weights.
//   expert B_e  [expert][group of 32 features][r / 8][32 lanes][8 bf16]: the same idea for the rows of B_e.
//
// The kernel has two phases with one grid-wide barrier between them (hence the cooperative launch: every CTA
// is resident, one per SM):
//   phase 1  the CTAs whose share of the weight stream touches a linear split that linear's token work:
//            RMSNorm (optional), absmax quantisation (Eq. 7-9), router (Sec. 3.3) and the rows of h = A_e x
//            (every row cut into sixteen pieces, one per warp, so that a CTA with one row still has all its
//            loads in flight at once).  The int8 codes go to global memory in the order the bit product
//            reads them, h in fp32.
//   phase 2  two lists of work items, each cut into equal contiguous shares, one per CTA and then one per warp:
//            (a) the expert product z = B_e h for (token, group of 32 features): twenty coalesced loads in
//                flight per lane, fp32 multiply-adds, z to global memory;
//            (b) the chunks of sign bits: dp4a of 0/1 byte masks with the int8 codes
//                (sum_k q S = 2 * sum_{bit set} q - sum q), partial sums added to an int32 accumulator in
//                global memory.
//            Every item reports to the counter of its row group (128 features x 8 tokens); the warp whose
//            report completes the count reads the sums and z back and writes Y (Eq. 10-11).
// Nothing is staged through shared memory but the activations and the router rows: the weight loads in flight
// live in registers, so the stream needs no producer, no barriers between warps and no polling.
#include <algorithm>
#include <mutex>

#include "pq_kernels.cuh"

namespace pq {

constexpr int kStreamThreads = 512;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kStreamMaxBatch = 96;      // linears per launch: their records travel as kernel parameters (32 KB limit)
constexpr int kStreamTokenGroup = 8;     // tokens whose codes sit in shared memory at once
constexpr int kStreamBarSlots = 64;

// Grid barrier words, one pair per caller stream slot: {arrivals, departures}.  Zero between launches: the last
// CTA to leave a kernel clears its pair.  (decode_stream_reset clears all of them after an error.)
__device__ unsigned g_stream_bar[kStreamBarSlots][2];

struct StreamLinear {
  const uint16_t* X;        // [M, K] bf16
  const uint16_t* Wr;       // [E, K] bf16 or null
  const uint16_t* A;        // [E, r, K] bf16
  const uint4* B_il;        // interleaved rows of B_e (bf16), or of the int8 codes B8_e when A8 is set
  const int8_t* A8;         // [E, r, K] int8 codes of A_e: the INT8 high-precision branch (Sec. 3.2), or null
  const float* hp_scales;   // [E][2] {gamma_A, gamma_B} of the INT8 branch
  const uint4* bits_il;     // interleaved sign bits
  const float* w_scales;
  const float* alpha;
  const float* beta;
  uint16_t* Y;              // [M, N]
  const uint16_t* norm_w;   // [K] bf16 or null
  DecodeTokInfo* info;      // [16] expert, gate, gamma, code sum per token
  const DecodeTokInfo* info_q;  // where gamma and the code sum come from: `info`, or the record of an earlier linear of the
                            // launch that reads the same activations (then `qg` is that linear's too and nothing is quantised here)
  uint32_t* qg;             // [M][C * 32] words of int8 codes in bit-product order
  float* h;                 // [M][r] (INT8 branch: the exact integers h_int = A8_e q, as int32)
  float* z;                 // [M][G * 128] expert product
  int* acc;                 // [M][G * 128] partial sums over the set bits
  unsigned* cnt;            // [token groups][G] items reported
  int* acc_dump;            // [M, N] or null
  int* zint_dump;           // [M, N] exact sums of the INT8 branch's second product (test hook) or null
  float norm_eps;
  int M, K, N, r, E, sstride;
  int G, C;                 // row groups; chunks per row group
  int chunk0;               // position of this linear's first chunk in the launch-wide list of chunks
  int z0;                   // position of its first item in the launch-wide list of expert-product items (M * 4 G each)
  int share;                // 1: codes, gamma and code sum are another linear's (see info_q)
  int zero_words;           // int32 words from `acc` on that phase 1 clears (acc and cnt are adjacent)
};
// The descriptor travels as kernel parameters (constant memory).  What every CTA needs to find its work sits in a few
// compact tables in front, so that a CTA touches the records of its own one or two linears only: a first touch of a
// cold parameter line costs a trip to memory, and a loop over sixteen records paid sixteen of them in a row.
struct StreamBatch {
  int n;
  int total_chunks, total_z;
  int bar_slot;
  int prefetch;             // chunks ahead of the bit product for which L2 prefetches are issued (0 = none)
  int mma_from;             // token groups of at least this many tokens take the tensor-core bit product
  int interleave;           // the two halves of a CTA walk the two work lists of phase 2 side by side
  int router_rows;          // router rows that fit in shared memory beside the token
  int off_rows, off_part;   // phase 1 carve-up: [token][router rows][partial sums of h][the token's codes in natural order]
  int off_qn;
  int off_h, off_info;      // phase 2 carve-up: [codes][h][token info][INT8 branch: codes of h, their scales]
  int off_qh;
  int chunk0[kStreamMaxBatch + 1];   // first chunk of every linear in the launch-wide list (and the total)
  int z0[kStreamMaxBatch + 1];       // first expert-product item of every linear
  int cost0[kStreamMaxBatch + 1];    // token work before every linear, in units of K / 32 per (token, row of A_e)
  int duty0[161];                    // where in that list the share of CTA b begins (and, one further, ends)
  StreamLinear lin[kStreamMaxBatch];
};

// ---------------------------------------------------------------------------
// one-time layout of the weights for this path
// ---------------------------------------------------------------------------
__global__ void k_pack_decode_bits(const uint32_t* __restrict__ bits, uint4* __restrict__ out, int N, int KW, int G, int C) {
  const long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= (long long)G * C * 128) return;
  const int lane = (int)(o & 31), f = (int)((o >> 5) & 3);
  const long long gc = o >> 7;
  const int c = (int)(gc % C), g = (int)(gc / C);
  const int n = g * 128 + f * 32 + lane;
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  if (n < N) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (4 * c + i < KW) w[i] = bits[(long long)n * KW + 4 * c + i];
  }
  out[o] = make_uint4(w[0], w[1], w[2], w[3]);
}

__global__ void k_pack_decode_b(const uint4* __restrict__ B, uint4* __restrict__ out, int E, int N, int r8, int G32) {
  const long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= (long long)E * G32 * r8 * 32) return;
  const int lane = (int)(o & 31);
  long long t = o >> 5;
  const int jc = (int)(t % r8); t /= r8;
  const int g32 = (int)(t % G32);
  const int e = (int)(t / G32);
  const int n = g32 * 32 + lane;
  out[o] = n < N ? B[((long long)e * N + n) * r8 + jc] : make_uint4(0u, 0u, 0u, 0u);
}

// the same for the int8 codes B8 of the INT8 branch: lane l holds 16 consecutive hidden values of row 32 group + l
__global__ void k_pack_decode_b8(const uint4* __restrict__ B8, uint4* __restrict__ out, int E, int N, int r16, int G32) {
  const long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= (long long)E * G32 * r16 * 32) return;
  const int lane = (int)(o & 31);
  long long t = o >> 5;
  const int jc = (int)(t % r16); t /= r16;
  const int g32 = (int)(t % G32);
  const int e = (int)(t / G32);
  const int n = g32 * 32 + lane;
  out[o] = n < N ? B8[((long long)e * N + n) * r16 + jc] : make_uint4(0u, 0u, 0u, 0u);
}

size_t decode_pack_b8_bytes(int N, int r, int E) { return (size_t)std::max(E, 1) * ((N + 127) / 128) * 4 * (size_t)(r / 16) * 512; }

int decode_pack_b8(int N, int r, int E, const int8_t* B8, int8_t* B8_il, cudaStream_t st) {
  const int G = (N + 127) / 128, Ee = std::max(E, 1);
  const long long total = (long long)Ee * G * 4 * (r / 16) * 32;
  LaunchScope ls(KID_DECODE_PACK, st);
  k_pack_decode_b8<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(reinterpret_cast<const uint4*>(B8), reinterpret_cast<uint4*>(B8_il), Ee, N, r / 16, G * 4);
  return cudaGetLastError() == cudaSuccess ? PQ_OK : PQ_ERR_CUDA;
}

void decode_pack_sizes(int K, int N, int r, int E, size_t* bits_bytes, size_t* b_bytes) {
  const size_t G = (N + 127) / 128, C = (K + 127) / 128;
  *bits_bytes = G * C * 2048;
  *b_bytes = r > 0 ? (size_t)std::max(E, 1) * G * 4 * (size_t)(r / 8) * 512 : 0;
}

int decode_pack(int K, int N, int r, int E, const uint32_t* bits, const uint16_t* B, uint32_t* bits_il, uint16_t* B_il, cudaStream_t st) {
  const int G = (N + 127) / 128, C = (K + 127) / 128;
  {
    const long long total = (long long)G * C * 128;
    LaunchScope ls(KID_DECODE_PACK, st);
    k_pack_decode_bits<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(bits, reinterpret_cast<uint4*>(bits_il), N, K / 32, G, C);
    if (cudaGetLastError() != cudaSuccess) return PQ_ERR_CUDA;
  }
  if (r > 0) {
    const int Ee = std::max(E, 1);
    const long long total = (long long)Ee * G * 4 * (r / 8) * 32;
    LaunchScope ls(KID_DECODE_PACK, st);
    k_pack_decode_b<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(reinterpret_cast<const uint4*>(B), reinterpret_cast<uint4*>(B_il), Ee, N, r / 8, G * 4);
    if (cudaGetLastError() != cudaSuccess) return PQ_ERR_CUDA;
  }
  return PQ_OK;
}

// ---------------------------------------------------------------------------
// grid barrier with a bound on the wait (every CTA is resident: cooperative launch)
// ---------------------------------------------------------------------------
__device__ __forceinline__ void stream_bar_arrive(unsigned* bar) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(&bar[0], 1u);
  }
}
// Called by one thread right after the CTA's wait: once every CTA has got past the wait nobody reads the pair any more, and
// the last one through leaves it clear for the next launch (nothing is left to do at the end of the kernel).
__device__ __forceinline__ void stream_bar_depart(unsigned* bar) {
  const unsigned old = atomicAdd(&bar[1], 1u);
  if (old == gridDim.x - 1) {
    bar[0] = 0u;
    bar[1] = 0u;
    __threadfence();
  }
}

// returns false (for every thread of the CTA) when the wait ran out
__device__ __forceinline__ bool stream_bar_wait(unsigned* bar, int* ok_sh) {
  if (threadIdx.x == 0) {
    int ok = 1;
    const long long t0 = clock64();
    while (*reinterpret_cast<volatile unsigned*>(&bar[0]) < gridDim.x) {
      if (clock64() - t0 > c_spin_cycles) {
        report_timeout(WHERE_OTHER);
        ok = 0;
        break;
      }
    }
    __threadfence();
    *ok_sh = ok;
  }
  __syncthreads();
  if (threadIdx.x == kStreamThreads - 32) stream_bar_depart(bar);   // its warp alone waits for the returned count
  return *ok_sh != 0;
}
// ---------------------------------------------------------------------------
// phase 1: one token of one linear, rows [j_lo, j_hi) of h; `owner` also quantises and publishes the token
// ---------------------------------------------------------------------------
struct StreamShared {
  double red_d[kStreamWarps];
  float red_f[kStreamWarps];
  int red_i[kStreamWarps];
  float logit[kMaxExperts];
  int ok;
};

// copies `total` 16-byte pieces, eight loads in flight per thread: piece i goes from src(i) to dst(i)
template <class Dst, class Src>
__device__ __forceinline__ void stream_stage(int total, Dst dst, Src src) {
  for (int base = threadIdx.x; base < total; base += kStreamThreads * 8) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = base + u * kStreamThreads;
      v[u] = i < total ? __ldg(src(i)) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = base + u * kStreamThreads;
      if (i < total) *dst(i) = v[u];
    }
  }
}

// Partial dot products of `nrows` rows (a4: first row, `chunks` 16-byte pieces each) with the token in shared memory
// over this warp's pieces [s_lo, s_hi): 16 / UPL rows at a time, UPL loads per lane and row (more pieces: further rounds).
template <int UPL>
__device__ __forceinline__ void stream_h_rows(const uint4* a4, const uint4* xs4, float* part, int nrows, int chunks, int s_lo, int s_hi,
                                              int warp, int lane) {
  constexpr int RB = 16 / UPL;
  for (int jb = 0; jb < nrows; jb += RB) {
    float acc[RB];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb) acc[rb] = 0.f;
    for (int c0 = s_lo + lane; c0 < s_hi; c0 += 32 * UPL) {
      uint4 wv[RB][UPL];
#pragma unroll
      for (int rb = 0; rb < RB; ++rb)
#pragma unroll
        for (int u = 0; u < UPL; ++u)
          wv[rb][u] = (jb + rb < nrows && c0 + 32 * u < s_hi) ? __ldg(a4 + (long long)(jb + rb) * chunks + c0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int u = 0; u < UPL; ++u) {
        if (c0 + 32 * u < s_hi) {
          const uint4 xv = xs4[c0 + 32 * u];
#pragma unroll
          for (int rb = 0; rb < RB; ++rb) {
            float a = acc[rb];
            a = fmaf(bf16lo(xv.x), bf16lo(wv[rb][u].x), a); a = fmaf(bf16hi(xv.x), bf16hi(wv[rb][u].x), a);
            a = fmaf(bf16lo(xv.y), bf16lo(wv[rb][u].y), a); a = fmaf(bf16hi(xv.y), bf16hi(wv[rb][u].y), a);
            a = fmaf(bf16lo(xv.z), bf16lo(wv[rb][u].z), a); a = fmaf(bf16hi(xv.z), bf16hi(wv[rb][u].z), a);
            a = fmaf(bf16lo(xv.w), bf16lo(wv[rb][u].w), a); a = fmaf(bf16hi(xv.w), bf16hi(wv[rb][u].w), a);
            acc[rb] = a;
          }
        }
      }
    }
#pragma unroll
    for (int rb = 0; rb < RB; ++rb) {
      float a = acc[rb];
      for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
      if (lane == 0 && jb + rb < nrows) part[(jb + rb) * kStreamWarps + warp] = a;
    }
  }
}

// The INT8 branch's first product (Sec. 3.2): rows of int8 codes A8_e against the token's int8 codes, exact in int32.
// Same cutting as above with 16 codes per piece; the partial sums are integers, so their order does not matter.
template <int UPL>
__device__ __forceinline__ void stream_h_rows8(const uint4* a16, const uint4* q16, int* part, int nrows, int pieces, int s_lo, int s_hi,
                                               int warp, int lane) {
  constexpr int RB = 16 / UPL;
  for (int jb = 0; jb < nrows; jb += RB) {
    int acc[RB];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb) acc[rb] = 0;
    for (int c0 = s_lo + lane; c0 < s_hi; c0 += 32 * UPL) {
      uint4 wv[RB][UPL];
#pragma unroll
      for (int rb = 0; rb < RB; ++rb)
#pragma unroll
        for (int u = 0; u < UPL; ++u)
          wv[rb][u] = (jb + rb < nrows && c0 + 32 * u < s_hi) ? __ldg(a16 + (long long)(jb + rb) * pieces + c0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int u = 0; u < UPL; ++u) {
        if (c0 + 32 * u < s_hi) {
          const uint4 qv = q16[c0 + 32 * u];
#pragma unroll
          for (int rb = 0; rb < RB; ++rb) {
            int a = acc[rb];
            a = __dp4a((int)wv[rb][u].x, (int)qv.x, a); a = __dp4a((int)wv[rb][u].y, (int)qv.y, a);
            a = __dp4a((int)wv[rb][u].z, (int)qv.z, a); a = __dp4a((int)wv[rb][u].w, (int)qv.w, a);
            acc[rb] = a;
          }
        }
      }
    }
#pragma unroll
    for (int rb = 0; rb < RB; ++rb) {
      int a = acc[rb];
      for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
      if (lane == 0 && jb + rb < nrows) part[(jb + rb) * kStreamWarps + warp] = a;
    }
  }
}

template <bool HP8>
__device__ void stream_token(const StreamBatch& bp, const StreamLinear& L, int t, int j_lo, int j_hi, bool owner, bool first, uint8_t* smem, StreamShared& sh) {
  const int K = L.K, E = L.E, r = L.r;
  const int chunks = K >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint4* xs4 = reinterpret_cast<uint4*>(smem);
  uint4* rows4 = reinterpret_cast<uint4*>(smem + bp.off_rows);
  float* part = reinterpret_cast<float*>(smem + bp.off_part);
  const uint4* x4 = reinterpret_cast<const uint4*>(L.X) + (long long)t * chunks;
  const uint4* wr4 = reinterpret_cast<const uint4*>(L.Wr);
  const int R = bp.router_rows;
  __syncthreads();   // the previous token's values are no longer read
  // the token and the first round of router rows travel together; when all rows fit they stay for the CTA's later tokens
  const int first_rows = (E > 1 && (first || R < E)) ? min(R, E) : 0;
  stream_stage(chunks * (1 + first_rows), [&](int i) { return i < chunks ? xs4 + i : rows4 + (i - chunks); },
               [&](int i) { return i < chunks ? x4 + i : wr4 + (i - chunks); });
  __syncthreads();
  if (L.norm_w) {
    // RMSNorm in front of the quantiser (App. A): mean of squares and reciprocal root in fp64, the factor rounded
    // once to fp32; the token in shared memory becomes bf16(fp32(fp32(x s) w)), which every later step reads
    double ss = 0.0;
    for (int c = threadIdx.x; c < chunks; c += kStreamThreads) {
      const uint4 v = xs4[c];
      const double d0 = bf16lo(v.x), d1 = bf16hi(v.x), d2 = bf16lo(v.y), d3 = bf16hi(v.y);
      const double d4 = bf16lo(v.z), d5 = bf16hi(v.z), d6 = bf16lo(v.w), d7 = bf16hi(v.w);
      ss += ((d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3)) + ((d4 * d4 + d5 * d5) + (d6 * d6 + d7 * d7));
    }
    for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
    if (lane == 0) sh.red_d[warp] = ss;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kStreamWarps; ++w) tot += sh.red_d[w];
    const float s = (float)(1.0 / sqrt(tot / (double)K + (double)L.norm_eps));
    const uint4* g4 = reinterpret_cast<const uint4*>(L.norm_w);
    for (int c = threadIdx.x; c < chunks; c += kStreamThreads) {
      const uint4 v = xs4[c], g = __ldg(g4 + c);
      uint4 o;
      o.x = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.x), s), bf16lo(g.x)), __fmul_rn(__fmul_rn(bf16hi(v.x), s), bf16hi(g.x)));
      o.y = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.y), s), bf16lo(g.y)), __fmul_rn(__fmul_rn(bf16hi(v.y), s), bf16hi(g.y)));
      o.z = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.z), s), bf16lo(g.z)), __fmul_rn(__fmul_rn(bf16hi(v.z), s), bf16hi(g.z)));
      o.w = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.w), s), bf16lo(g.w)), __fmul_rn(__fmul_rn(bf16hi(v.w), s), bf16hi(g.w)));
      xs4[c] = o;
    }
    // a thread reads back only its own chunks in the pass below; the barrier after it publishes them
  }
  float amax = 0.f;
  for (int c = threadIdx.x; c < chunks; c += kStreamThreads) {
    const uint4 v = xs4[c];
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.x)), fabsf(bf16hi(v.x))), fmaxf(fabsf(bf16lo(v.y)), fabsf(bf16hi(v.y)))));
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.z)), fabsf(bf16hi(v.z))), fmaxf(fabsf(bf16lo(v.w)), fabsf(bf16hi(v.w)))));
  }
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  if (lane == 0) sh.red_f[warp] = amax;
  __syncthreads();
  amax = sh.red_f[0];
#pragma unroll
  for (int w = 1; w < kStreamWarps; ++w) amax = fmaxf(amax, sh.red_f[w]);
  const float gamma = __fdiv_rn(kActQmax, fmaxf(amax, kActAmaxFloor));

  // router in the pinned fp32 order of the training path: lane j owns the chunks c = j mod 32, ascending, fused
  // multiply-add; butterfly 16, 8, 4, 2, 1.  One warp per expert row of the round, out of shared memory.
  int best = 0;
  float gate = 1.0f;
  if (E > 1) {
    for (int e0 = 0; e0 < E; e0 += R) {
      const int n = min(R, E - e0);
      if (e0 > 0) {
        __syncthreads();   // the previous round's rows have been used
        stream_stage(chunks * n, [&](int i) { return rows4 + i; }, [&](int i) { return wr4 + (long long)e0 * chunks + i; });
        __syncthreads();
      }
      for (int k = warp; k < n; k += kStreamWarps) {
        const uint4* wrow = rows4 + (size_t)k * chunks;
        float acc = 0.f;
        for (int c = lane; c < chunks; c += 32) {
          const uint4 xv = xs4[c], wv = wrow[c];
          acc = fmaf(bf16lo(xv.x), bf16lo(wv.x), acc); acc = fmaf(bf16hi(xv.x), bf16hi(wv.x), acc);
          acc = fmaf(bf16lo(xv.y), bf16lo(wv.y), acc); acc = fmaf(bf16hi(xv.y), bf16hi(wv.y), acc);
          acc = fmaf(bf16lo(xv.z), bf16lo(wv.z), acc); acc = fmaf(bf16hi(xv.z), bf16hi(wv.z), acc);
          acc = fmaf(bf16lo(xv.w), bf16lo(wv.w), acc); acc = fmaf(bf16hi(xv.w), bf16hi(wv.w), acc);
        }
        for (int d = 16; d > 0; d >>= 1) acc = acc + __shfl_xor_sync(0xffffffffu, acc, d);
        if (lane == 0) sh.logit[e0 + k] = acc;
      }
    }
    __syncthreads();
    float lmax = sh.logit[0];
    for (int e = 1; e < E; ++e)
      if (sh.logit[e] > lmax) { lmax = sh.logit[e]; best = e; }
    float den = 0.f, pbest = 0.f;
    for (int e = 0; e < E; ++e) {
      const float pe = expf(sh.logit[e] - lmax);
      den += pe;
      if (e == best) pbest = pe;
    }
    gate = pbest * (1.0f / den);
  }

  // rows [j_lo, j_hi) of h = A_e x: warp w takes the w-th sixteenth of every row (whole 16-byte pieces), sixteen
  // loads per lane issued before the first use; the sixteen partial sums of a row are added in warp order afterwards
  const int nrows = r > 0 ? j_hi - j_lo : 0;
  if (HP8 && nrows > 0 && L.A8) {
    // INT8 branch: the token's codes in natural order (Eq. 7-9, the values the owner also writes out below)
    uint2* qn = reinterpret_cast<uint2*>(smem + bp.off_qn);
    for (int c = threadIdx.x; c < chunks; c += kStreamThreads) {
      const uint4 v = xs4[c];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      uint32_t o[2] = {0u, 0u};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int q0 = max(-128, min(127, __float2int_rn(__fmul_rn(bf16lo(w[u]), gamma))));
        const int q1 = max(-128, min(127, __float2int_rn(__fmul_rn(bf16hi(w[u]), gamma))));
        o[u >> 1] |= ((uint32_t)(q0 & 0xFF) | ((uint32_t)(q1 & 0xFF) << 8)) << (16 * (u & 1));
      }
      qn[c] = make_uint2(o[0], o[1]);
    }
    __syncthreads();
    const int pieces = K >> 4;
    const int s_lo = (int)((long long)pieces * warp / kStreamWarps), s_hi = (int)((long long)pieces * (warp + 1) / kStreamWarps);
    const uint4* a16 = reinterpret_cast<const uint4*>(L.A8) + ((long long)best * r + j_lo) * pieces;
    const int upl = ((pieces + kStreamWarps - 1) / kStreamWarps + 31) / 32;
    int* parti = reinterpret_cast<int*>(part);
    const uint4* q16 = reinterpret_cast<const uint4*>(qn);
    if (upl == 1) stream_h_rows8<1>(a16, q16, parti, nrows, pieces, s_lo, s_hi, warp, lane);
    else if (upl == 2) stream_h_rows8<2>(a16, q16, parti, nrows, pieces, s_lo, s_hi, warp, lane);
    else stream_h_rows8<4>(a16, q16, parti, nrows, pieces, s_lo, s_hi, warp, lane);
  } else if (nrows > 0) {
    const int s_lo = (int)((long long)chunks * warp / kStreamWarps), s_hi = (int)((long long)chunks * (warp + 1) / kStreamWarps);
    const uint4* a4 = reinterpret_cast<const uint4*>(L.A) + ((long long)best * r + j_lo) * chunks;
    const int upl = ((chunks + kStreamWarps - 1) / kStreamWarps + 31) / 32;   // loads per lane and row
    if (upl == 1) stream_h_rows<1>(a4, xs4, part, nrows, chunks, s_lo, s_hi, warp, lane);
    else if (upl == 2) stream_h_rows<2>(a4, xs4, part, nrows, chunks, s_lo, s_hi, warp, lane);
    else stream_h_rows<4>(a4, xs4, part, nrows, chunks, s_lo, s_hi, warp, lane);
  }

  if (owner && !L.share) {
    // Eq. 7-9; a thread turns 32 values of k into the 8 words the bit product reads: word b holds the codes of
    // k = b, b + 8, b + 16, b + 24 (the bytes that the mask 0x01010101 << b selects from a weight word)
    const int ngroups = L.C * 4;
    uint32_t* qrow = L.qg + (long long)t * L.C * 32;
    int rowsum = 0;
    for (int grp = threadIdx.x; grp < ngroups; grp += kStreamThreads) {
      uint32_t words[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
      if (grp * 32 < K) {
        int qv[32];
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          const uint4 v = xs4[grp * 4 + ch];
          const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int q0 = max(-128, min(127, __float2int_rn(__fmul_rn(bf16lo(w[u]), gamma))));
            const int q1 = max(-128, min(127, __float2int_rn(__fmul_rn(bf16hi(w[u]), gamma))));
            qv[8 * ch + 2 * u] = q0;
            qv[8 * ch + 2 * u + 1] = q1;
            rowsum += q0 + q1;
          }
        }
#pragma unroll
        for (int b = 0; b < 8; ++b)
          words[b] = (qv[b] & 0xFF) | ((qv[b + 8] & 0xFF) << 8) | ((qv[b + 16] & 0xFF) << 16) | ((qv[b + 24] & 0xFF) << 24);
      }
      uint4* dst = reinterpret_cast<uint4*>(qrow + grp * 8);
      dst[0] = make_uint4(words[0], words[1], words[2], words[3]);
      dst[1] = make_uint4(words[4], words[5], words[6], words[7]);
    }
    for (int d = 16; d > 0; d >>= 1) rowsum += __shfl_xor_sync(0xffffffffu, rowsum, d);
    if (lane == 0) sh.red_i[warp] = rowsum;
  }
  __syncthreads();   // partial sums of h and of the codes are visible
  if (owner && threadIdx.x == 0) {
    int tot = 0;
    if (!L.share)
      for (int w = 0; w < kStreamWarps; ++w) tot += sh.red_i[w];
    L.info[t] = DecodeTokInfo{best, gate, gamma, tot};   // (shared codes: the code sum is filled in from info_q in phase 2)
  }
  for (int i = threadIdx.x; i < nrows; i += kStreamThreads) {
    if (HP8 && L.A8) {
      int a = 0;
#pragma unroll
      for (int w = 0; w < kStreamWarps; ++w) a += reinterpret_cast<const int*>(part)[i * kStreamWarps + w];
      reinterpret_cast<int*>(L.h)[(long long)t * r + j_lo + i] = a;
    } else {
      float a = 0.f;
#pragma unroll
      for (int w = 0; w < kStreamWarps; ++w) a += part[i * kStreamWarps + w];
      L.h[(long long)t * r + j_lo + i] = a;
    }
  }
}

// ---------------------------------------------------------------------------
// phase 2.  Every work item reports to the counter of its row group (128 features x the tokens of one group of
// eight); the report that completes the count (C chunks of sign bits, plus four expert-product items per token
// when there is an HP branch) finishes the row group.
// ---------------------------------------------------------------------------
// four signed codes times four unsigned mask bytes (a mask byte can be 0x80)
__device__ __forceinline__ int dp4a_s8u8(uint32_t q, uint32_t m, int c) {
  int d;
  asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(q), "r"(m), "r"(c));
  return d;
}

__device__ __forceinline__ unsigned stream_target(const StreamLinear& L, int tg) {
  const int mg = min(kStreamTokenGroup, L.M - tg * kStreamTokenGroup);
  return (unsigned)(2 * L.C + (L.r > 0 ? 4 * mg : 0));   // two units per chunk, one per expert-product item
}

// Eq. 10-11 for row group g and the tokens of group tg: everything it needs is complete in global memory
__device__ void stream_finish(const StreamLinear& L, int tg, int g, const DecodeTokInfo* toks, int lane) {
  __threadfence();
  const float lam = __ldg(L.w_scales);
  const int Np = L.G * 128;
  const int mg = min(kStreamTokenGroup, L.M - tg * kStreamTokenGroup);
  float be[4], al[4];
#pragma unroll
  for (int f = 0; f < 4; ++f) {
    const int n = g * 128 + f * 32 + lane;
    be[f] = n < L.N ? __ldg(L.beta + (long long)n * L.sstride) : 0.f;
    al[f] = (n < L.N && L.r > 0) ? __ldg(L.alpha + (long long)n * L.sstride) : 0.f;
  }
  for (int t = 0; t < mg; ++t) {
    const int tok = tg * kStreamTokenGroup + t;
    const DecodeTokInfo tk = toks[tok];
    const float deq = __fdiv_rn(lam, tk.gamma);
    int m[4];
    float z[4];
#pragma unroll
    for (int f = 0; f < 4; ++f) {
      const long long at = (long long)tok * Np + g * 128 + f * 32 + lane;
      m[f] = __ldcg(L.acc + at);
      z[f] = L.r > 0 ? __ldcg(L.z + at) : 0.f;
    }
#pragma unroll
    for (int f = 0; f < 4; ++f) {
      const int n = g * 128 + f * 32 + lane;
      if (n < L.N) {
        const int acc = 2 * m[f] - tk.rowsum;
        float y = be[f] * deq * (float)acc;
        if (L.r > 0) y = fmaf(al[f] * tk.gate, z[f], y);
        L.Y[(long long)tok * L.N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
        if (L.acc_dump) L.acc_dump[(long long)tok * L.N + n] = acc;
      }
    }
  }
}

// reports `units` finished items of row group (tg, g); true for the whole warp when that completes the count
__device__ __forceinline__ bool stream_report(const StreamLinear& L, int tg, int g, unsigned units, int lane) {
  __threadfence();
  __syncwarp();
  unsigned old = 0u;
  if (lane == 0) old = atomicAdd(L.cnt + tg * L.G + g, units);
  old = __shfl_sync(0xffffffffu, old, 0);
  return old + units == stream_target(L, tg);
}

// (a) expert-product items [i_lo, i_hi) of one linear: item = token * 4G + group of 32 features; hs = h of all its tokens.
// Consecutive items of one row group are reported together.
template <bool HP8>
__device__ void stream_expert(const StreamLinear& L, int i_lo, int i_hi, const float* hs, const DecodeTokInfo* toks, const int8_t* qh8,
                              const float* gh) {
  const int lane = threadIdx.x & 31;
  const int G32 = L.G * 4, r = L.r, r8 = r >> 3;
  const int Np = L.G * 128;
  unsigned run = 0u;
  for (int i = i_lo; i < i_hi; ++i) {
    const int tok = i / G32, g32 = i - tok * G32;
    if (HP8 && g32 * 32 < L.N && L.A8) {
      // INT8 branch: z_int = B8_e qh (exact), z = z_int / (gamma_B gamma_h gamma_A gamma_t)
      const int e = toks[tok].expert, r16 = r >> 4;
      const uint4* bp = L.B_il + ((long long)e * G32 + g32) * r16 * 32 + lane;
      const uint4* qv = reinterpret_cast<const uint4*>(qh8 + tok * r);
      int zi = 0;
      uint4 b[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) b[u] = u < r16 ? __ldg(bp + (long long)u * 32) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        if (u < r16) {
          const uint4 q = qv[u];
          zi = __dp4a((int)b[u].x, (int)q.x, zi); zi = __dp4a((int)b[u].y, (int)q.y, zi);
          zi = __dp4a((int)b[u].z, (int)q.z, zi); zi = __dp4a((int)b[u].w, (int)q.w, zi);
        }
      }
      const float den = __fmul_rn(__fmul_rn(__fmul_rn(__ldg(L.hp_scales + 2 * e + 1), gh[tok]), __ldg(L.hp_scales + 2 * e)), toks[tok].gamma);
      const int n = g32 * 32 + lane;
      L.z[(long long)tok * Np + n] = __fdiv_rn((float)zi, den);
      if (L.zint_dump && n < L.N) L.zint_dump[(long long)tok * L.N + n] = zi;
    } else if (g32 * 32 < L.N) {
      const uint4* bp = L.B_il + ((long long)toks[tok].expert * G32 + g32) * r8 * 32 + lane;
      const float* hv = hs + tok * r;
      float z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;
      for (int j0 = 0; j0 < r8; j0 += 20) {
        uint4 b[20];
#pragma unroll
        for (int u = 0; u < 20; ++u) b[u] = j0 + u < r8 ? __ldg(bp + (long long)(j0 + u) * 32) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < 20; ++u) {
          if (j0 + u < r8) {
            const float4 h0 = *reinterpret_cast<const float4*>(hv + (j0 + u) * 8);
            const float4 h1 = *reinterpret_cast<const float4*>(hv + (j0 + u) * 8 + 4);
            z0 = fmaf(bf16lo(b[u].x), h0.x, z0); z1 = fmaf(bf16hi(b[u].x), h0.y, z1);
            z2 = fmaf(bf16lo(b[u].y), h0.z, z2); z3 = fmaf(bf16hi(b[u].y), h0.w, z3);
            z0 = fmaf(bf16lo(b[u].z), h1.x, z0); z1 = fmaf(bf16hi(b[u].z), h1.y, z1);
            z2 = fmaf(bf16lo(b[u].w), h1.z, z2); z3 = fmaf(bf16hi(b[u].w), h1.w, z3);
          }
        }
      }
      L.z[(long long)tok * Np + g32 * 32 + lane] = (z0 + z1) + (z2 + z3);
    }
    ++run;
    const bool last_of_group = (g32 & 3) == 3 || i + 1 == i_hi;   // the next item belongs to another row group (or token)
    if (last_of_group) {
      const int tg = tok / kStreamTokenGroup, g = g32 >> 2;
      if (stream_report(L, tg, g, run, lane)) stream_finish(L, tg, g, toks, lane);
      run = 0u;
    }
  }
}

// (b) chunks [p_lo, p_hi) of one linear for the tokens of group tg.  MT = tokens of the group rounded up to 1, 2, 4
// or 8; with one token the masks need no shift (eight accumulators per feature, weighted 1 << b, exact in int32:
// 127 * 128 * K < 2^31 for every K the library accepts).
template <int MT>
__device__ void stream_bits(const StreamLinear& L, int tg, int mg, int p_lo, int p_hi, const uint32_t* qs, int qstride, const DecodeTokInfo* toks,
                            int ahead) {
  constexpr bool NS = MT == 1;
  constexpr int NA = NS ? 8 : 1;
  const int lane = threadIdx.x & 31;
  const int C = L.C;
  const int Np = L.G * 128;
  int acc[4][MT][NA];
#pragma unroll
  for (int f = 0; f < 4; ++f)
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int a = 0; a < NA; ++a) acc[f][t][a] = 0;
  int p = p_lo;
  if (p >= p_hi) return;
  int g = p / C, c = p - g * C;
  int delivered = 0;                                         // chunks of row group g in the accumulators
  const uint4* src = L.bits_il + (long long)p * 128 + lane;
  uint4 w[4];
#pragma unroll
  for (int f = 0; f < 4; ++f) w[f] = __ldg(src + f * 32);
  // the first chunks of the range on their way to L2 (a chunk is sixteen 128-byte lines: lanes 0..15 ask for one each)
  const char* line = reinterpret_cast<const char*>(L.bits_il + (long long)p * 128) + (lane & 15) * 128;
  if (lane < 16)
    for (int a = 2; a < ahead && p + a < p_hi; ++a) asm volatile("prefetch.global.L2 [%0];" ::"l"(line + (long long)a * 2048));
  while (p < p_hi) {
    if (lane < 16 && ahead > 0 && p + ahead < p_hi) asm volatile("prefetch.global.L2 [%0];" ::"l"(line + (long long)ahead * 2048));
    line += 2048;
    uint4 wn[4];
    const uint4* nxt = src + (p + 1 < p_hi ? 128 : 0);
#pragma unroll
    for (int f = 0; f < 4; ++f) wn[f] = __ldg(nxt + f * 32);
    const uint32_t* qc = qs + c * 32;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint4 qq[MT];
#pragma unroll
        for (int t = 0; t < MT; ++t) qq[t] = *reinterpret_cast<const uint4*>(qc + t * qstride + i * 8 + hh * 4);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
          for (int f = 0; f < 4; ++f) {
            const uint32_t wi = i == 0 ? w[f].x : i == 1 ? w[f].y : i == 2 ? w[f].z : w[f].w;
            const uint32_t m = NS ? (wi & (0x01010101u << (hh * 4 + j))) : ((wi >> (hh * 4 + j)) & 0x01010101u);
#pragma unroll
            for (int t = 0; t < MT; ++t) {
              const uint32_t qv = j == 0 ? qq[t].x : j == 1 ? qq[t].y : j == 2 ? qq[t].z : qq[t].w;
              acc[f][t][NS ? hh * 4 + j : 0] = dp4a_s8u8(qv, m, acc[f][t][NS ? hh * 4 + j : 0]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int f = 0; f < 4; ++f) w[f] = wn[f];
    src = nxt;
    ++p; ++c; ++delivered;
    if (c == C || p == p_hi) {
      // hand the row group's partial sums over
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        if (t < mg) {
          int* dst = L.acc + (long long)(tg * kStreamTokenGroup + t) * Np + g * 128 + lane;
#pragma unroll
          for (int f = 0; f < 4; ++f) {
            int v = 0;
#pragma unroll
            for (int a = 0; a < NA; ++a) v += NS ? (acc[f][t][a] >> a) : acc[f][t][a];
            atomicAdd(dst + f * 32, v);
          }
        }
      }
#pragma unroll
      for (int f = 0; f < 4; ++f)
#pragma unroll
        for (int t = 0; t < MT; ++t)
#pragma unroll
          for (int a = 0; a < NA; ++a) acc[f][t][a] = 0;
      if (stream_report(L, tg, g, 2u * (unsigned)delivered, lane)) stream_finish(L, tg, g, toks, lane);
      if (c == C) { c = 0; ++g; }
      delivered = 0;
    }
  }
}

// (b') the same chunks on the tensor cores (mma.sync m16n8k32, u8 masks x s8 codes, exact in int32), for five to eight
// tokens: sixteen features x 32 contraction values x eight tokens per instruction, where dp4a pays once per token.
// A block of a chunk is 128 rows of 16 bytes in feature order, so thread (g = lane / 4, c = lane % 4) finds the
// four bit words of features 16 T + g and 16 T + g + 8 at rows of their own; like every thread of its quad it loads
// them whole and takes the bits c + 8 j (mask 0x01010101 of w >> c) and c + 4 + 8 j (mask 0x10101010: the value 16,
// summed in a second accumulator that stays an exact multiple of 16) -- the codes in shared memory are already in
// that order (word b of a group of 32 holds k = b + 8 j).  A row group is walked in two halves of 64 features so
// that the accumulators (4 tiles x 2 x 4) and a prefetched half block fit in registers.
__device__ void stream_bits_mma(const StreamLinear& L, int tg, int mg, int p_lo, int p_hi, const uint32_t* qs, int qstride,
                                const DecodeTokInfo* toks, int ahead) {
  const int lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
  const int C = L.C;
  const int Np = L.G * 128;
  const uint32_t* qtok = qs + min(g, mg - 1) * qstride + c;   // token g of the group (surplus lanes read the last one)
  int p = p_lo;
  while (p < p_hi) {
    const int rg = p / C, c0 = p - rg * C, n = min(C - c0, p_hi - p);
    for (int half = 0; half < 2; ++half) {
      int a1[4][4], a16[4][4];
#pragma unroll
      for (int T = 0; T < 4; ++T)
#pragma unroll
        for (int u = 0; u < 4; ++u) { a1[T][u] = 0; a16[T][u] = 0; }
      const uint4* blk = L.bits_il + (long long)p * 128 + half * 64 + g;
      const char* line = reinterpret_cast<const char*>(L.bits_il + (long long)p * 128 + half * 64) + (lane & 7) * 128;
      if (lane < 8)
        for (int a = 1; a < ahead && a < n; ++a) asm volatile("prefetch.global.L2 [%0];" ::"l"(line + (long long)a * 2048));
      uint4 w[4][2];
#pragma unroll
      for (int T = 0; T < 4; ++T) { w[T][0] = __ldg(blk + T * 16); w[T][1] = __ldg(blk + T * 16 + 8); }
      for (int i = 0; i < n; ++i) {
        if (lane < 8 && ahead > 0 && i + ahead < n) asm volatile("prefetch.global.L2 [%0];" ::"l"(line + (long long)(i + ahead) * 2048));
        uint4 wn[4][2];
        const uint4* nb = blk + (i + 1 < n ? 128 : 0);
#pragma unroll
        for (int T = 0; T < 4; ++T) { wn[T][0] = __ldg(nb + T * 16); wn[T][1] = __ldg(nb + T * 16 + 8); }
        const uint32_t* qc = qtok + (c0 + i) * 32;
#pragma unroll
        for (int pr = 0; pr < 2; ++pr) {
          const uint32_t q1a = qc[(2 * pr) * 8], q1b = qc[(2 * pr + 1) * 8], q16a = qc[(2 * pr) * 8 + 4], q16b = qc[(2 * pr + 1) * 8 + 4];
#pragma unroll
          for (int T = 0; T < 4; ++T) {
            const uint32_t x00 = pr == 0 ? w[T][0].x : w[T][0].z, x01 = pr == 0 ? w[T][0].y : w[T][0].w;
            const uint32_t x10 = pr == 0 ? w[T][1].x : w[T][1].z, x11 = pr == 0 ? w[T][1].y : w[T][1].w;
            const uint32_t t00 = x00 >> c, t01 = x01 >> c, t10 = x10 >> c, t11 = x11 >> c;
            const uint32_t m1[4] = {t00 & 0x01010101u, t10 & 0x01010101u, t01 & 0x01010101u, t11 & 0x01010101u};
            const uint32_t m16[4] = {t00 & 0x10101010u, t10 & 0x10101010u, t01 & 0x10101010u, t11 & 0x10101010u};
            mma_u8s8(a1[T], m1, q1a, q1b);
            mma_u8s8(a16[T], m16, q16a, q16b);
          }
        }
#pragma unroll
        for (int T = 0; T < 4; ++T) { w[T][0] = wn[T][0]; w[T][1] = wn[T][1]; }
        blk = nb;
      }
      // accumulator u of tile T: feature 16 T + g (u < 2) or + 8, token 2 c + (u & 1)
#pragma unroll
      for (int T = 0; T < 4; ++T)
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int t = 2 * c + (u & 1);
          if (t < mg) {
            const int row = rg * 128 + half * 64 + T * 16 + g + (u >> 1) * 8;
            atomicAdd(L.acc + (long long)(tg * kStreamTokenGroup + t) * Np + row, a1[T][u] + (a16[T][u] >> 4));
          }
        }
      if (stream_report(L, tg, rg, (unsigned)n, lane)) stream_finish(L, tg, rg, toks, lane);
    }
    p += n;
  }
}

// ---------------------------------------------------------------------------
// the kernel: grid = one CTA per SM (cooperative launch), 512 threads
// ---------------------------------------------------------------------------
// A token's record as phase 2 uses it: routing from the linear's own record, gamma and code sum from the linear whose
// codes it multiplies (itself unless it shares another's activations).  Written by other CTAs: read through L2.
__device__ __forceinline__ DecodeTokInfo stream_record(const StreamLinear& L, int t) {
  const int4 a = __ldcg(reinterpret_cast<const int4*>(L.info) + t);
  DecodeTokInfo r{a.x, __int_as_float(a.y), __int_as_float(a.z), a.w};
  if (L.share) {
    const int4 b = __ldcg(reinterpret_cast<const int4*>(L.info_q) + t);
    r.gamma = __int_as_float(b.z);
    r.rowsum = b.w;
  }
  return r;
}

// barrier of one group of warps of the CTA (ids 1 and 2; 0 is __syncthreads)
__device__ __forceinline__ void stream_group_sync(int bid, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(bid), "r"(nthreads) : "memory"); }

// HP8: some linear of the launch uses the INT8 high-precision branch; MMA: some token group is large enough for the
// tensor-core bit product.  Separate instantiations, so that the common case carries neither's registers nor code.
template <bool HP8, bool MMA>
__global__ void __launch_bounds__(kStreamThreads, 1) k_decode_stream(const __grid_constant__ StreamBatch bp) {
  extern __shared__ __align__(128) uint8_t stream_smem[];
  __shared__ StreamShared sh;
  unsigned* bar = g_stream_bar[bp.bar_slot];
  const int nC = (int)gridDim.x, cta = (int)blockIdx.x;
  const int warp = threadIdx.x >> 5;
  const long long T = bp.total_chunks, Z = bp.total_z;
  const int span_lo = (int)(T * cta / nC), span_hi = (int)(T * (cta + 1) / nC);
  const int zspan_lo = (int)(Z * cta / nC), zspan_hi = (int)(Z * (cta + 1) / nC);

  // the linears whose chunks / expert-product items this CTA's spans touch
  int l_lo = 0, l_hi = 0, zl_lo = 0, zl_hi = 0;
  for (int l = 0; l < bp.n; ++l) {
    if (bp.chunk0[l + 1] <= span_lo) l_lo = l + 1;
    if (bp.chunk0[l] < span_hi) l_hi = l + 1;
    if (bp.z0[l + 1] <= zspan_lo) zl_lo = l + 1;
    if (bp.z0[l] < zspan_hi) zl_hi = l + 1;
  }

  // phase 0: accumulators and counters start at zero.  A linear's words are shared out in proportion to its chunks:
  // the CTA that owns chunks [lo, hi) of its GC chunks clears words [ceil(lo W / GC), ceil(hi W / GC)).
  for (int l = l_lo; l < l_hi; ++l) {
    const StreamLinear& L = bp.lin[l];
    const long long gc = (long long)L.G * L.C;
    const int lo = max(span_lo, L.chunk0) - L.chunk0, hi = min(span_hi, L.chunk0 + (int)gc) - L.chunk0;
    if (lo >= hi) continue;
    const long long w_lo = ((long long)lo * L.zero_words + gc - 1) / gc, w_hi = ((long long)hi * L.zero_words + gc - 1) / gc;
    for (long long i = w_lo + threadIdx.x; i < w_hi; i += kStreamThreads) L.acc[i] = 0;
  }

  // phase 1: this CTA's share of the token work, a launch-wide list of (token, row of A_e) units weighted by the length
  // of a row and cut into contiguous shares by the host; a unit belongs to the CTA in whose share it begins
  {
    const long long d_lo = bp.duty0[cta], d_hi = bp.duty0[cta + 1];
    for (int l = 0; l < bp.n; ++l) {
      if (bp.cost0[l + 1] <= d_lo || bp.cost0[l] >= d_hi) continue;
      const StreamLinear& L = bp.lin[l];
      const long long w = L.K >> 5, base = bp.cost0[l];
      const int rp = max(L.r, 1);
      const long long U = (long long)L.M * rp;
      const int u_lo = (int)min(U, (max(d_lo - base, 0LL) + w - 1) / w), u_hi = (int)min(U, (max(d_hi - base, 0LL) + w - 1) / w);
      if (u_lo >= u_hi) continue;
      for (int t = u_lo / rp; t <= (u_hi - 1) / rp; ++t) {
        const int j_lo = max(u_lo, t * rp) - t * rp, j_hi = min(u_hi, (t + 1) * rp) - t * rp;
        stream_token<HP8>(bp, L, t, j_lo, j_hi, j_lo == 0, t == u_lo / rp, stream_smem, sh);
      }
    }
  }
  stream_bar_arrive(bar);
  const bool ok = stream_bar_wait(bar, &sh.ok);

  if (ok) {
    // phase 2: two steps.  Alone, the whole CTA walks its chunks of sign bits, then its expert-product items.  With
    // `interleave` the two halves of the CTA (eight warps and a named barrier each) do one of each at a time -- half 0
    // the first half of the chunks, then the second half of the items, half 1 the other way round -- so that a list
    // bound by instruction issue and a list bound by memory run side by side; the host turns it on where it measured faster (up to eight tokens per linear).
    uint32_t* qs = reinterpret_cast<uint32_t*>(stream_smem);
    float* hs = reinterpret_cast<float*>(stream_smem + bp.off_h);
    const int ngroups = bp.interleave ? 2 : 1;
    const int gthreads = kStreamThreads / ngroups, gwarps = gthreads / 32;
    const int grp = threadIdx.x / gthreads, gtid = threadIdx.x - grp * gthreads, gw = gtid >> 5;
    const int bid = 1 + grp;
    DecodeTokInfo* toks = reinterpret_cast<DecodeTokInfo*>(stream_smem + bp.off_info) + grp * kDecodeMaxTokens;
    const int span_mid = span_lo + (span_hi - span_lo) / 2, zspan_mid = zspan_lo + (zspan_hi - zspan_lo) / 2;
    for (int step = 0; step < 2; ++step) {
      const bool bits_now = ngroups == 1 ? step == 0 : (grp ^ step) == 0;
      if (bits_now) {
        const int lo = ngroups == 1 ? span_lo : (grp == 0 ? span_lo : span_mid), hi = ngroups == 1 ? span_hi : (grp == 0 ? span_mid : span_hi);
        for (int l = 0; l < bp.n; ++l) {
          if (bp.chunk0[l + 1] <= lo || bp.chunk0[l] >= hi) continue;
          const StreamLinear& L = bp.lin[l];
          const int seg_lo = max(lo, L.chunk0) - L.chunk0, seg_hi = min(hi, bp.chunk0[l + 1]) - L.chunk0;
          const int qwords = L.C * 32, qstride = qwords + 4;   // the pad spreads the tokens' rows over the banks (mma variant)
          const int len = seg_hi - seg_lo;
          const int p_lo = seg_lo + (int)((long long)len * gw / gwarps), p_hi = seg_lo + (int)((long long)len * (gw + 1) / gwarps);
          for (int tg = 0; tg * kStreamTokenGroup < L.M; ++tg) {
            const int mg = min(kStreamTokenGroup, L.M - tg * kStreamTokenGroup);
            stream_group_sync(bid, gthreads);   // the previous codes and token records are no longer read
            {
              // written by other CTAs in phase 1: read through L2
              const int row4 = qwords >> 2;
              const uint4* from = reinterpret_cast<const uint4*>(L.qg + (long long)tg * kStreamTokenGroup * qwords);
              for (int i = gtid; i < mg * row4; i += gthreads) {
                const int t = i / row4, j = i - t * row4;
                reinterpret_cast<uint4*>(qs + t * qstride)[j] = __ldcg(from + i);
              }
              if (gtid < L.M) {
                toks[gtid] = stream_record(L, gtid);
                if (L.share && seg_lo == 0 && tg == 0) L.info[gtid] = toks[gtid];   // complete the record for the decode view
              }
            }
            stream_group_sync(bid, gthreads);
            if (MMA && mg >= bp.mma_from) stream_bits_mma(L, tg, mg, p_lo, p_hi, qs, qstride, toks, bp.prefetch);
            else if (mg == 1) stream_bits<1>(L, tg, mg, p_lo, p_hi, qs, qstride, toks, bp.prefetch);
            else if (mg == 2) stream_bits<2>(L, tg, mg, p_lo, p_hi, qs, qstride, toks, bp.prefetch);
            else if (mg <= 4) stream_bits<4>(L, tg, mg, p_lo, p_hi, qs, qstride, toks, bp.prefetch);
            else stream_bits<8>(L, tg, mg, p_lo, p_hi, qs, qstride, toks, bp.prefetch);
          }
        }
      } else {
        const int lo = ngroups == 1 ? zspan_lo : (grp == 1 ? zspan_lo : zspan_mid), hi = ngroups == 1 ? zspan_hi : (grp == 1 ? zspan_mid : zspan_hi);
        for (int l = 0; l < bp.n; ++l) {
          if (bp.z0[l + 1] <= lo || bp.z0[l] >= hi || bp.z0[l + 1] == bp.z0[l]) continue;
          const StreamLinear& L = bp.lin[l];
          const int seg_lo = max(lo, L.z0) - L.z0, seg_hi = min(hi, bp.z0[l + 1]) - L.z0;
          stream_group_sync(bid, gthreads);
          for (int i = gtid; i < L.M * L.r; i += gthreads) hs[i] = __ldcg(L.h + i);
          if (gtid < L.M) toks[gtid] = stream_record(L, gtid);
          stream_group_sync(bid, gthreads);
          int8_t* qh8 = reinterpret_cast<int8_t*>(stream_smem + bp.off_qh);
          float* gh = reinterpret_cast<float*>(stream_smem + bp.off_qh + kDecodeMaxTokens * 256);
          if (HP8 && L.A8) {
            // the hidden activation enters the second 8-bit product quantised per token from its exact integers (Eq. 7-9):
            // gamma_h = 128 / max(max_j |fl32(h_int)|, 1e-5), code = clamp(rint(fl32(h_int) * gamma_h)); a warp per token
            for (int t = gw; t < L.M; t += gwarps) {
              const int* hi32 = reinterpret_cast<const int*>(hs) + t * L.r;
              const int lane = threadIdx.x & 31;
              float amax = 0.f;
              for (int j = lane; j < L.r; j += 32) amax = fmaxf(amax, fabsf((float)hi32[j]));
              for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
              const float g = __fdiv_rn(kActQmax, fmaxf(amax, kActAmaxFloor));
              for (int j = lane; j < L.r; j += 32) qh8[t * L.r + j] = (int8_t)max(-128, min(127, __float2int_rn(__fmul_rn((float)hi32[j], g))));
              if (lane == 0) gh[t] = g;
            }
            stream_group_sync(bid, gthreads);
          }
          const int len = seg_hi - seg_lo;
          stream_expert<HP8>(L, seg_lo + (int)((long long)len * gw / gwarps), seg_lo + (int)((long long)len * (gw + 1) / gwarps), hs, toks, qh8, gh);
        }
      }
      __syncthreads();   // the halves swap the code and h buffers (alone: the bit product's buffers are free)
    }
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static inline size_t s_up256(size_t x) { return (x + 255) / 256 * 256; }

// bytes this path needs in an item's workspace beyond what decode_workspace_bytes() counts:
// codes | h | z | accumulators and counters
size_t decode_stream_extra_bytes(int M, int K, int N, int r, bool dump) {
  const size_t G = (N + 127) / 128, C = (K + 127) / 128;
  const size_t groups = (M + kStreamTokenGroup - 1) / kStreamTokenGroup;
  return s_up256((size_t)M * C * 128) + s_up256((size_t)M * std::max(r, 1) * 4) + s_up256((size_t)M * G * 128 * 4) +
         s_up256(((size_t)M * G * 128 + groups * G) * 4) + (dump ? s_up256((size_t)M * N * 4) : 0);
}
// where the INT8 branch leaves its exact integers (h_int always, z_int with the dump flag), for the decode view
void decode_stream_view(int M, int K, int N, int r, void* ws, bool dump, int** h_int, int** z_int) {
  const size_t G = (N + 127) / 128, C = (K + 127) / 128;
  const size_t groups = (M + kStreamTokenGroup - 1) / kStreamTokenGroup;
  uint8_t* w = static_cast<uint8_t*>(ws) + decode_workspace_bytes(M, K, N, r, dump) + s_up256((size_t)M * C * 128);
  *h_int = reinterpret_cast<int*>(w);
  w += s_up256((size_t)M * std::max(r, 1) * 4) + s_up256((size_t)M * G * 128 * 4) + s_up256(((size_t)M * G * 128 + groups * G) * 4);
  *z_int = dump ? reinterpret_cast<int*>(w) : nullptr;
}

static int g_decode_stream_on = 1;
static int g_decode_stream_prefetch = 1;
static int g_decode_stream_interleave = 1;
void decode_stream_interleave(int mode) { g_decode_stream_interleave = mode < 0 ? 0 : mode > 2 ? 2 : mode; }
static int g_decode_stream_mma_from = 5;   // measured on the 3B shapes: dp4a is ahead up to four tokens, level at four
void decode_stream_mma_from(int m) { g_decode_stream_mma_from = m < 1 ? 1 : m; }
void decode_stream_enable(int mode) { g_decode_stream_on = mode < 0 ? 0 : mode > 2 ? 2 : mode; }
void decode_stream_prefetch(int on) { g_decode_stream_prefetch = on ? 1 : 0; }
int decode_stream_mode() { return g_decode_stream_on; }
int decode_stream_max_batch() { return kStreamMaxBatch; }

void decode_stream_reset() {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_stream_bar) == cudaSuccess) cudaMemset(p, 0, sizeof(unsigned) * kStreamBarSlots * 2);
}

// one barrier pair per caller stream: launches on one stream are ordered, launches on different streams may overlap
static int stream_bar_slot(cudaStream_t st) {
  static std::mutex mu;
  static cudaStream_t table[kStreamBarSlots];
  static int used = 0;
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < used; ++i)
    if (table[i] == st) return i;
  if (used == kStreamBarSlots) return -1;
  table[used] = st;
  return used++;
}

constexpr size_t kStreamSmemLimit = 200 * 1024;

int decode_stream_launch(const DecodeItemArgs* items, int n, cudaStream_t st) {
  static int sms = [] {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    return v;
  }();
  if (n < 1 || n > kStreamMaxBatch) return PQ_ERR_UNSUPPORTED;
  StreamBatch bp{};
  bp.n = n;
  long long total = 0, total_z = 0;
  size_t codes = 0, hbytes = 0, xbytes = 0, part = 0;
  int max_e = 1;
  for (int i = 0; i < n; ++i) {
    const DecodeItemArgs& it = items[i];
    const int M = it.a.T, K = it.a.K, N = it.a.N, r = it.a.r;
    if (!it.bits_il || (r > 0 && !it.B_il) || (r & 7) || M > 16) return PQ_ERR_UNSUPPORTED;
    if (it.A8 && (r <= 0 || (r & 15) || !it.hp_scales)) return PQ_ERR_UNSUPPORTED;
    StreamLinear& L = bp.lin[i];
    L.X = it.X; L.Wr = it.a.Wr; L.A = it.a.A; L.B_il = reinterpret_cast<const uint4*>(it.B_il);
    L.bits_il = reinterpret_cast<const uint4*>(it.bits_il);
    L.w_scales = it.a.w_scales; L.alpha = it.a.alpha; L.beta = it.a.beta; L.Y = it.Y;
    L.norm_w = it.norm_weight; L.norm_eps = it.norm_eps;
    L.A8 = it.A8; L.hp_scales = it.hp_scales;
    L.M = M; L.K = K; L.N = N; L.r = r; L.E = (r > 0 && it.a.E > 1) ? it.a.E : 1; L.sstride = it.a.scale_stride;
    L.G = (N + 127) / 128; L.C = (K + 127) / 128;
    uint8_t* w = static_cast<uint8_t*>(it.ws);
    L.info = reinterpret_cast<DecodeTokInfo*>(w);
    L.acc_dump = it.dump ? decode_view(M, K, N, r, it.ws, true).acc : nullptr;
    w += decode_workspace_bytes(M, K, N, r, it.dump);
    L.qg = reinterpret_cast<uint32_t*>(w); w += s_up256((size_t)M * L.C * 128);
    L.h = reinterpret_cast<float*>(w); w += s_up256((size_t)M * std::max(r, 1) * 4);
    L.z = reinterpret_cast<float*>(w); w += s_up256((size_t)M * L.G * 128 * 4);
    L.acc = reinterpret_cast<int*>(w);
    const int groups = (M + kStreamTokenGroup - 1) / kStreamTokenGroup;
    L.cnt = reinterpret_cast<unsigned*>(L.acc + (size_t)M * L.G * 128);
    L.zero_words = M * L.G * 128 + groups * L.G;
    w += s_up256((size_t)L.zero_words * 4);
    L.zint_dump = (it.dump && it.A8) ? reinterpret_cast<int*>(w) : nullptr;
    // N1 (App. A, "without redundant data reads"): a linear that reads the same activations as an earlier one of the
    // launch (gate and up of a block, q / k / v) multiplies that linear's codes instead of quantising again
    L.info_q = L.info; L.share = 0;
    for (int j = 0; j < i; ++j) {
      const DecodeItemArgs& o = items[j];
      if (o.X == it.X && o.a.T == M && o.a.K == K && o.norm_weight == it.norm_weight && o.norm_eps == it.norm_eps && !bp.lin[j].share) {
        L.qg = bp.lin[j].qg; L.info_q = bp.lin[j].info; L.share = 1;
        break;
      }
    }
    L.chunk0 = (int)total;
    total += (long long)L.G * L.C;
    L.z0 = (int)total_z;
    if (r > 0) total_z += (long long)M * L.G * 4;
    if (total > (1ll << 30) || total_z > (1ll << 30)) return PQ_ERR_UNSUPPORTED;
    // the bit product is instantiated for 1, 2, 4 or 8 tokens and reads that many rows of codes (the surplus rows are
    // never used, but they must lie inside the allocation)
    const int mt = M >= 5 ? 8 : M >= 3 ? 4 : M;
    codes = std::max(codes, (size_t)mt * (L.C * 128 + 16));
    hbytes = std::max(hbytes, (size_t)M * std::max(r, 1) * 4);
    xbytes = std::max(xbytes, (size_t)K * 2);
    part = std::max(part, (size_t)std::max(r, 1) * kStreamWarps * 4);
    max_e = std::max(max_e, L.E);
  }
  bp.total_chunks = (int)total;
  bp.total_z = (int)total_z;
  for (int i = 0; i <= kStreamMaxBatch; ++i) {
    bp.chunk0[i] = i < n ? bp.lin[i].chunk0 : (int)total;
    bp.z0[i] = i < n ? bp.lin[i].z0 : (int)total_z;
  }
  const int nC = sms;
  {
    long long run = 0;
    for (int i = 0; i < n; ++i) {
      bp.cost0[i] = (int)run;
      run += (long long)bp.lin[i].M * std::max(bp.lin[i].r, 1) * (bp.lin[i].K >> 5);
      if (run > (1ll << 30)) return PQ_ERR_UNSUPPORTED;
    }
    for (int i = n; i <= kStreamMaxBatch; ++i) bp.cost0[i] = (int)run;
    if (nC > 160) return PQ_ERR_UNSUPPORTED;
    if (4 * n <= nC) {
      // few linears: every linear gets CTAs of its own, as many as its share of the work (at least one), so that no CTA
      // prepares tokens of two linears (the token, the router rows and the routing are a fixed cost per CTA and linear)
      int next = 0;
      for (int i = 0; i < n; ++i) {
        int end = i + 1 == n ? nC : (int)((double)bp.cost0[i + 1] / (double)run * (nC - n) + 0.5) + (i + 1);
        end = std::min(std::max(end, next + 1), nC - (n - 1 - i));
        const long long c0 = bp.cost0[i], c1 = bp.cost0[i + 1];
        for (int c = next; c < end; ++c) bp.duty0[c] = (int)(c0 + (c1 - c0) * (c - next) / (end - next));
        next = end;
      }
      bp.duty0[nC] = (int)run;
    } else {
      // many linears: equal shares of the list, whatever linears they fall on
      for (int c = 0; c <= nC; ++c) bp.duty0[c] = (int)(run * c / nC);
    }
  }
  // shared memory: phase 1 [token][router rows][partial sums], phase 2 [codes][h][token records]
  xbytes = s_up256(xbytes);
  const size_t avail = kStreamSmemLimit - xbytes - s_up256(part) - xbytes / 2;
  bp.router_rows = max_e > 1 ? (int)std::min<size_t>(max_e, avail / xbytes) : 0;
  if (max_e > 1 && bp.router_rows < 1) return PQ_ERR_UNSUPPORTED;
  bp.off_rows = (int)xbytes;
  bp.off_part = (int)(xbytes + (size_t)bp.router_rows * xbytes);
  bp.off_qn = (int)(bp.off_part + s_up256(part));
  const size_t smem1 = bp.off_qn + xbytes / 2;          // the token's int8 codes: half the bytes of its bf16 values
  bp.off_h = (int)s_up256(codes);
  bp.off_info = (int)(bp.off_h + s_up256(hbytes));
  bp.off_qh = bp.off_info + 2 * kDecodeMaxTokens * (int)sizeof(DecodeTokInfo);   // one set of token records per half
  const size_t smem2 = bp.off_qh + kDecodeMaxTokens * 256 + 256;
  const size_t smem = std::max(smem1, smem2);
  if (smem > kStreamSmemLimit) return PQ_ERR_UNSUPPORTED;
  bp.bar_slot = stream_bar_slot(st);
  if (bp.bar_slot < 0) return PQ_ERR_UNSUPPORTED;
  bp.prefetch = g_decode_stream_prefetch ? 4 : 0;
  bp.mma_from = g_decode_stream_mma_from;
  {
    // measured on the 3B shapes: ahead by 1-4 % at one token, 6-16 % at four, behind by 2-4 % at sixteen (two token groups
    // walk the chunks twice, and half a CTA restages the codes for each)
    int max_m = 1;
    for (int i = 0; i < n; ++i) max_m = std::max(max_m, bp.lin[i].M);
    bp.interleave = g_decode_stream_interleave > 1 || (g_decode_stream_interleave == 1 && max_m <= kStreamTokenGroup);
  }
  bool hp8 = false, mma = false;
  for (int i = 0; i < n; ++i) {
    hp8 = hp8 || bp.lin[i].A8 != nullptr;
    const int M = bp.lin[i].M;
    mma = mma || std::min(M, kStreamTokenGroup) >= bp.mma_from || (M > kStreamTokenGroup && M - kStreamTokenGroup >= bp.mma_from);
  }
  using Kern = void (*)(StreamBatch);
  const Kern kern = hp8 ? (mma ? (Kern)k_decode_stream<true, true> : (Kern)k_decode_stream<true, false>)
                        : (mma ? (Kern)k_decode_stream<false, true> : (Kern)k_decode_stream<false, false>);
  static const bool limit_set =
      cudaFuncSetAttribute(k_decode_stream<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit) == cudaSuccess &&
      cudaFuncSetAttribute(k_decode_stream<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit) == cudaSuccess &&
      cudaFuncSetAttribute(k_decode_stream<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit) == cudaSuccess &&
      cudaFuncSetAttribute(k_decode_stream<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit) == cudaSuccess;
  if (!limit_set) return PQ_ERR_CUDA;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cudaLaunchConfig_t cfg{};
  cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
  cfg.gridDim = dim3(nC, 1, 1); cfg.blockDim = dim3(kStreamThreads, 1, 1); cfg.dynamicSmemBytes = smem;
  LaunchScope ls(KID_DECODE_STREAM, st);
  if (cudaLaunchKernelEx(&cfg, kern, bp) != cudaSuccess) return PQ_ERR_CUDA;
  return PQ_OK;
}

}  // namespace pq
