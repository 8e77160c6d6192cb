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
//            RMSNorm (optional), absmax quantisation (Eq. 7-9), router (Sec. 3.3) and the rows of h = A_e x.
//            The int8 codes go to global memory in the order the bit product reads them, h in fp32.
//   phase 2  the chunks of all linears form one list that is cut into equal contiguous spans, one per CTA and
//            then one per warp.  A warp multiplies its chunks (dp4a of 0/1 byte masks with the int8 codes:
//            sum_k q S = 2 * sum_{bit set} q - sum q), adds its partial sums to an int32 accumulator in global
//            memory and counts the chunks of the row group it has delivered; the warp that completes a row group
//            reads the sums back, adds the expert product and writes Y (Eq. 10-11).
// Nothing is staged through shared memory but the activations: the loads in flight live in registers, so the
// stream needs no producer, no barriers between warps and no polling.
#include <algorithm>
#include <mutex>

#include "pq_kernels.cuh"

namespace pq {

constexpr int kStreamThreads = 512;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kStreamMaxBatch = 16;
constexpr int kStreamTokenGroup = 8;     // tokens whose codes sit in shared memory at once
constexpr int kStreamBarSlots = 64;

// Grid barrier words, one pair per caller stream slot: {arrivals, departures}.  Zero between launches: the last
// CTA to leave a kernel clears its pair.  (decode_stream_reset clears all of them after an error.)
__device__ unsigned g_stream_bar[kStreamBarSlots][2];

struct StreamLinear {
  const uint16_t* X;        // [M, K] bf16
  const uint16_t* Wr;       // [E, K] bf16 or null
  const uint16_t* A;        // [E, r, K] bf16
  const uint4* B_il;        // interleaved rows of B_e
  const uint4* bits_il;     // interleaved sign bits
  const float* w_scales;
  const float* alpha;
  const float* beta;
  uint16_t* Y;              // [M, N]
  const uint16_t* norm_w;   // [K] bf16 or null
  DecodeTokInfo* info;      // [16] expert, gate, gamma, code sum per token
  uint32_t* qg;             // [M][C * 32] words of int8 codes in bit-product order
  float* h;                 // [M][r]
  int* acc;                 // [M][G * 128] partial sums over the set bits
  unsigned* cnt;            // [token groups][G] chunks delivered
  int* acc_dump;            // [M, N] or null
  float norm_eps;
  int M, K, N, r, E, sstride;
  int G, C;                 // row groups; chunks per row group
  int chunk0;               // position of this linear's first chunk in the launch-wide list
  int cta_first, cta_count; // the CTAs whose span touches this linear
  int zero_words;           // int32 words from `acc` on that phase 1 clears (acc and cnt are adjacent)
};
struct StreamBatch {
  StreamLinear lin[kStreamMaxBatch];
  int n;
  int total_chunks;
  int bar_slot;
  int prefetch;             // issue L2 prefetches for the span's sign bits before phase 1
  int off_h, off_info;      // shared-memory carve-up: [x or q region][h][info]
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
  return *ok_sh != 0;
}
__device__ __forceinline__ void stream_bar_depart(unsigned* bar) {
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned old = atomicAdd(&bar[1], 1u);
    if (old == gridDim.x - 1) {   // everybody has passed the wait: leave the pair clear for the next launch
      bar[0] = 0u;
      bar[1] = 0u;
      __threadfence();
    }
  }
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

__device__ void stream_token(const StreamLinear& L, int t, int j_lo, int j_hi, bool owner, uint4* xs4, StreamShared& sh) {
  const int K = L.K, E = L.E, r = L.r;
  const int chunks = K >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();   // the previous token's values are no longer read
  {
    const uint4* x4 = reinterpret_cast<const uint4*>(L.X) + (long long)t * chunks;
    for (int c = threadIdx.x; c < chunks; c += kStreamThreads) xs4[c] = x4[c];
  }
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
  // multiply-add; butterfly 16, 8, 4, 2, 1.  One warp per expert row, the row read straight from global memory.
  int best = 0;
  float gate = 1.0f;
  if (E > 1) {
    for (int e = warp; e < E; e += kStreamWarps) {
      const uint4* wrow = reinterpret_cast<const uint4*>(L.Wr) + (long long)e * chunks;
      float acc = 0.f;
      for (int c0 = lane; c0 < chunks; c0 += 128) {
        uint4 wv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) wv[u] = c0 + 32 * u < chunks ? __ldg(wrow + c0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (c0 + 32 * u < chunks) {
            const uint4 xv = xs4[c0 + 32 * u];
            acc = fmaf(bf16lo(xv.x), bf16lo(wv[u].x), acc); acc = fmaf(bf16hi(xv.x), bf16hi(wv[u].x), acc);
            acc = fmaf(bf16lo(xv.y), bf16lo(wv[u].y), acc); acc = fmaf(bf16hi(xv.y), bf16hi(wv[u].y), acc);
            acc = fmaf(bf16lo(xv.z), bf16lo(wv[u].z), acc); acc = fmaf(bf16hi(xv.z), bf16hi(wv[u].z), acc);
            acc = fmaf(bf16lo(xv.w), bf16lo(wv[u].w), acc); acc = fmaf(bf16hi(xv.w), bf16hi(wv[u].w), acc);
          }
        }
      }
      for (int d = 16; d > 0; d >>= 1) acc = acc + __shfl_xor_sync(0xffffffffu, acc, d);
      if (lane == 0) sh.logit[e] = acc;
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

  if (owner) {
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
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int w = 0; w < kStreamWarps; ++w) tot += sh.red_i[w];
      L.info[t] = DecodeTokInfo{best, gate, gamma, tot};
    }
  }

  // rows [j_lo, j_hi) of h = A_e x (fp32 accumulation over the bf16 operands), one warp per row
  if (r > 0) {
    for (int j = j_lo + warp; j < j_hi; j += kStreamWarps) {
      const uint4* arow = reinterpret_cast<const uint4*>(L.A) + ((long long)best * r + j) * chunks;
      float a0 = 0.f, a1 = 0.f;
      for (int c0 = lane; c0 < chunks; c0 += 256) {
        uint4 wv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) wv[u] = c0 + 32 * u < chunks ? __ldg(arow + c0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          if (c0 + 32 * u < chunks) {
            const uint4 xv = xs4[c0 + 32 * u];
            a0 = fmaf(bf16lo(xv.x), bf16lo(wv[u].x), a0); a1 = fmaf(bf16hi(xv.x), bf16hi(wv[u].x), a1);
            a0 = fmaf(bf16lo(xv.y), bf16lo(wv[u].y), a0); a1 = fmaf(bf16hi(xv.y), bf16hi(wv[u].y), a1);
            a0 = fmaf(bf16lo(xv.z), bf16lo(wv[u].z), a0); a1 = fmaf(bf16hi(xv.z), bf16hi(wv[u].z), a1);
            a0 = fmaf(bf16lo(xv.w), bf16lo(wv[u].w), a0); a1 = fmaf(bf16hi(xv.w), bf16hi(wv[u].w), a1);
          }
        }
      }
      float a = a0 + a1;
      for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
      if (lane == 0) L.h[(long long)t * r + j] = a;
    }
  }
}

// ---------------------------------------------------------------------------
// phase 2: the bit product of a warp's chunks [p_lo, p_hi) of one linear for the tokens of one group, and the
// epilogue of every row group this warp completes.  MT = tokens of the group rounded up to a power of two;
// with one token the masks need no shift (eight accumulators per feature, weighted 1 << b, exact in int32:
// 127 * 128 * K < 2^31 for every K the library accepts).
// ---------------------------------------------------------------------------
// four signed codes times four unsigned mask bytes (a mask byte can be 0x80)
__device__ __forceinline__ int dp4a_s8u8(uint32_t q, uint32_t m, int c) {
  int d;
  asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(q), "r"(m), "r"(c));
  return d;
}

template <int MT>
__device__ __forceinline__ void stream_epilogue(const StreamLinear& L, int tg, int mg, int g, int (&vals)[4][MT], const float* hs,
                                                const DecodeTokInfo* toks, int lane) {
  const float lam = __ldg(L.w_scales);
  const int r = L.r, r8 = r >> 3;
  const int G32 = L.G * 4;
#pragma unroll
  for (int t = 0; t < MT; ++t) {
    if (t >= mg) break;
    const DecodeTokInfo tk = toks[t];
    const int tok = tg * kStreamTokenGroup + t;
    float z[4] = {0.f, 0.f, 0.f, 0.f};
    if (r > 0) {
      const uint4* bp = L.B_il + ((long long)tk.expert * G32 + g * 4) * r8 * 32 + lane;
      const float* hv = hs + t * r;
      for (int jc = 0; jc < r8; jc += 2) {
        uint4 b[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int f = 0; f < 4; ++f) b[u][f] = jc + u < r8 ? __ldg(bp + ((long long)f * r8 + jc + u) * 32) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          if (jc + u < r8) {
            const float4 h0 = *reinterpret_cast<const float4*>(hv + (jc + u) * 8);
            const float4 h1 = *reinterpret_cast<const float4*>(hv + (jc + u) * 8 + 4);
#pragma unroll
            for (int f = 0; f < 4; ++f) {
              float a = z[f];
              a = fmaf(bf16lo(b[u][f].x), h0.x, a); a = fmaf(bf16hi(b[u][f].x), h0.y, a);
              a = fmaf(bf16lo(b[u][f].y), h0.z, a); a = fmaf(bf16hi(b[u][f].y), h0.w, a);
              a = fmaf(bf16lo(b[u][f].z), h1.x, a); a = fmaf(bf16hi(b[u][f].z), h1.y, a);
              a = fmaf(bf16lo(b[u][f].w), h1.z, a); a = fmaf(bf16hi(b[u][f].w), h1.w, a);
              z[f] = a;
            }
          }
        }
      }
    }
    const float deq = __fdiv_rn(lam, tk.gamma);
#pragma unroll
    for (int f = 0; f < 4; ++f) {
      const int n = g * 128 + f * 32 + lane;
      if (n < L.N) {
        const int acc = 2 * vals[f][t] - tk.rowsum;
        float y = __ldg(L.beta + (long long)n * L.sstride) * deq * (float)acc;
        if (r > 0) y = fmaf(__ldg(L.alpha + (long long)n * L.sstride) * tk.gate, z[f], y);
        L.Y[(long long)tok * L.N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
        if (L.acc_dump) L.acc_dump[(long long)tok * L.N + n] = acc;
      }
    }
  }
}

template <int MT>
__device__ void stream_bits(const StreamLinear& L, int tg, int mg, int p_lo, int p_hi, const uint32_t* qs, int qwords, const float* hs,
                            const DecodeTokInfo* toks) {
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
  while (p < p_hi) {
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
        for (int t = 0; t < MT; ++t) qq[t] = *reinterpret_cast<const uint4*>(qc + t * qwords + i * 8 + hh * 4);
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
      // hand the row group's partial sums over; the warp that delivers its last chunk finishes it
      int vals[4][MT];
#pragma unroll
      for (int f = 0; f < 4; ++f)
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          int v = 0;
#pragma unroll
          for (int a = 0; a < NA; ++a) { v += NS ? (acc[f][t][a] >> a) : acc[f][t][a]; acc[f][t][a] = 0; }
          vals[f][t] = v;
        }
      bool finish = delivered == C;
      if (!finish) {
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          if (t < mg) {
            int* dst = L.acc + (long long)(tg * kStreamTokenGroup + t) * Np + g * 128 + lane;
#pragma unroll
            for (int f = 0; f < 4; ++f) atomicAdd(dst + f * 32, vals[f][t]);
          }
        }
        __threadfence();
        __syncwarp();
        unsigned old = 0u;
        if (lane == 0) old = atomicAdd(L.cnt + tg * L.G + g, (unsigned)delivered);
        old = __shfl_sync(0xffffffffu, old, 0);
        finish = old + (unsigned)delivered == (unsigned)C;
        if (finish) {
          __threadfence();
#pragma unroll
          for (int t = 0; t < MT; ++t) {
            if (t < mg) {
              const int* from = L.acc + (long long)(tg * kStreamTokenGroup + t) * Np + g * 128 + lane;
#pragma unroll
              for (int f = 0; f < 4; ++f) vals[f][t] = __ldcg(from + f * 32);
            }
          }
        }
      }
      if (finish) stream_epilogue<MT>(L, tg, mg, g, vals, hs, toks, lane);
      if (c == C) { c = 0; ++g; }
      delivered = 0;
    }
  }
}

// ---------------------------------------------------------------------------
// the kernel: grid = one CTA per SM (cooperative launch), 512 threads
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kStreamThreads, 1) k_decode_stream(const __grid_constant__ StreamBatch bp) {
  extern __shared__ __align__(128) uint8_t stream_smem[];
  __shared__ StreamShared sh;
  unsigned* bar = g_stream_bar[bp.bar_slot];
  const int nC = (int)gridDim.x, cta = (int)blockIdx.x;
  const int warp = threadIdx.x >> 5;
  const long long T = bp.total_chunks;
  const int span_lo = (int)(T * cta / nC), span_hi = (int)(T * (cta + 1) / nC);

  if (bp.prefetch) {
    // the sign bits of this CTA's span do not depend on phase 1: let them travel to L2 while it runs
    for (int l = 0; l < bp.n; ++l) {
      const StreamLinear& L = bp.lin[l];
      const int lo = max(span_lo, L.chunk0) - L.chunk0, hi = min(span_hi, L.chunk0 + L.G * L.C) - L.chunk0;
      if (lo >= hi) continue;
      const char* base = reinterpret_cast<const char*>(L.bits_il + (long long)lo * 128);
      const long long lines = (long long)(hi - lo) * 16;   // 128-byte lines
      for (long long i = threadIdx.x; i < lines; i += kStreamThreads) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + i * 128));
    }
  }

  // phase 0: this CTA's share of every linear's accumulators and counters starts at zero
  for (int l = 0; l < bp.n; ++l) {
    const StreamLinear& L = bp.lin[l];
    const long long z_lo = (long long)L.zero_words * cta / nC, z_hi = (long long)L.zero_words * (cta + 1) / nC;
    for (long long i = z_lo + threadIdx.x; i < z_hi; i += kStreamThreads) L.acc[i] = 0;
  }

  // phase 1: token work of the linears this CTA's span touches
  for (int l = 0; l < bp.n; ++l) {
    const StreamLinear& L = bp.lin[l];
    if (cta < L.cta_first || cta >= L.cta_first + L.cta_count) continue;
    const int s = cta - L.cta_first;
    const int rp = max(L.r, 1);
    const long long U = (long long)L.M * rp;
    const int u_lo = (int)(U * s / L.cta_count), u_hi = (int)(U * (s + 1) / L.cta_count);
    if (u_lo >= u_hi) continue;
    for (int t = u_lo / rp; t <= (u_hi - 1) / rp; ++t) {
      const int j_lo = max(u_lo, t * rp) - t * rp, j_hi = min(u_hi, (t + 1) * rp) - t * rp;
      stream_token(L, t, j_lo, j_hi, j_lo == 0, reinterpret_cast<uint4*>(stream_smem), sh);
    }
  }
  stream_bar_arrive(bar);
  const bool ok = stream_bar_wait(bar, &sh.ok);

  // phase 2
  if (ok) {
    uint32_t* qs = reinterpret_cast<uint32_t*>(stream_smem);
    float* hs = reinterpret_cast<float*>(stream_smem + bp.off_h);
    DecodeTokInfo* toks = reinterpret_cast<DecodeTokInfo*>(stream_smem + bp.off_info);
    for (int l = 0; l < bp.n; ++l) {
      const StreamLinear& L = bp.lin[l];
      const int seg_lo = max(span_lo, L.chunk0) - L.chunk0, seg_hi = min(span_hi, L.chunk0 + L.G * L.C) - L.chunk0;
      if (seg_lo >= seg_hi) continue;
      const int qwords = L.C * 32;
      const int len = seg_hi - seg_lo;
      const int p_lo = seg_lo + (int)((long long)len * warp / kStreamWarps), p_hi = seg_lo + (int)((long long)len * (warp + 1) / kStreamWarps);
      for (int tg = 0; tg * kStreamTokenGroup < L.M; ++tg) {
        const int mg = min(kStreamTokenGroup, L.M - tg * kStreamTokenGroup);
        __syncthreads();   // the previous codes are no longer read
        {
          // written by other CTAs in phase 1: read through L2
          const uint4* from = reinterpret_cast<const uint4*>(L.qg + (long long)tg * kStreamTokenGroup * qwords);
          uint4* to = reinterpret_cast<uint4*>(qs);
          for (int i = threadIdx.x; i < mg * (qwords >> 2); i += kStreamThreads) to[i] = __ldcg(from + i);
          const float* hfrom = L.h + (long long)tg * kStreamTokenGroup * L.r;
          for (int i = threadIdx.x; i < mg * L.r; i += kStreamThreads) hs[i] = __ldcg(hfrom + i);
          const int4* ifrom = reinterpret_cast<const int4*>(L.info + tg * kStreamTokenGroup);
          if (threadIdx.x < mg) reinterpret_cast<int4*>(toks)[threadIdx.x] = __ldcg(ifrom + threadIdx.x);
        }
        __syncthreads();
        if (mg == 1) stream_bits<1>(L, tg, mg, p_lo, p_hi, qs, qwords, hs, toks);
        else if (mg == 2) stream_bits<2>(L, tg, mg, p_lo, p_hi, qs, qwords, hs, toks);
        else if (mg <= 4) stream_bits<4>(L, tg, mg, p_lo, p_hi, qs, qwords, hs, toks);
        else stream_bits<8>(L, tg, mg, p_lo, p_hi, qs, qwords, hs, toks);
      }
    }
  }
  stream_bar_depart(bar);
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static inline size_t s_up256(size_t x) { return (x + 255) / 256 * 256; }

// bytes this path needs in an item's workspace beyond what decode_workspace_bytes() counts
size_t decode_stream_extra_bytes(int M, int K, int N, int r) {
  const size_t G = (N + 127) / 128, C = (K + 127) / 128;
  const size_t groups = (M + kStreamTokenGroup - 1) / kStreamTokenGroup;
  return s_up256((size_t)M * C * 128) + s_up256((size_t)M * std::max(r, 1) * 4) + s_up256(((size_t)M * G * 128 + groups * G) * 4);
}

static int g_decode_stream_on = 1;
static int g_decode_stream_prefetch = 1;
void decode_stream_enable(int on) { g_decode_stream_on = on ? 1 : 0; }
void decode_stream_prefetch(int on) { g_decode_stream_prefetch = on ? 1 : 0; }
bool decode_stream_enabled() { return g_decode_stream_on != 0; }

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
  long long total = 0;
  size_t region0 = 0, hbytes = 0;
  for (int i = 0; i < n; ++i) {
    const DecodeItemArgs& it = items[i];
    const int M = it.a.T, K = it.a.K, N = it.a.N, r = it.a.r;
    if (!it.bits_il || (r > 0 && !it.B_il) || (r & 7) || M > 16) return PQ_ERR_UNSUPPORTED;
    StreamLinear& L = bp.lin[i];
    L.X = it.X; L.Wr = it.a.Wr; L.A = it.a.A; L.B_il = reinterpret_cast<const uint4*>(it.B_il);
    L.bits_il = reinterpret_cast<const uint4*>(it.bits_il);
    L.w_scales = it.a.w_scales; L.alpha = it.a.alpha; L.beta = it.a.beta; L.Y = it.Y;
    L.norm_w = it.norm_weight; L.norm_eps = it.norm_eps;
    L.M = M; L.K = K; L.N = N; L.r = r; L.E = (r > 0 && it.a.E > 1) ? it.a.E : 1; L.sstride = it.a.scale_stride;
    L.G = (N + 127) / 128; L.C = (K + 127) / 128;
    uint8_t* w = static_cast<uint8_t*>(it.ws);
    L.info = reinterpret_cast<DecodeTokInfo*>(w);
    L.acc_dump = it.dump ? decode_view(M, K, N, r, it.ws, true).acc : nullptr;
    w += decode_workspace_bytes(M, K, N, r, it.dump);
    L.qg = reinterpret_cast<uint32_t*>(w); w += s_up256((size_t)M * L.C * 128);
    L.h = reinterpret_cast<float*>(w); w += s_up256((size_t)M * std::max(r, 1) * 4);
    L.acc = reinterpret_cast<int*>(w);
    const int groups = (M + kStreamTokenGroup - 1) / kStreamTokenGroup;
    L.cnt = reinterpret_cast<unsigned*>(L.acc + (size_t)M * L.G * 128);
    L.zero_words = M * L.G * 128 + groups * L.G;
    L.chunk0 = (int)total;
    total += (long long)L.G * L.C;
    if (total > (1ll << 30)) return PQ_ERR_UNSUPPORTED;
    // the bit product is instantiated for 1, 2, 4 or 8 tokens and reads that many rows of codes (the surplus rows are
    // never used, but they must lie inside the allocation)
    const int mt = M >= 5 ? 8 : M >= 3 ? 4 : M;
    region0 = std::max(region0, std::max((size_t)K * 2, (size_t)mt * L.C * 128));
    hbytes = std::max(hbytes, (size_t)kStreamTokenGroup * std::max(r, 1) * 4);
  }
  bp.total_chunks = (int)total;
  const int nC = sms;
  for (int i = 0; i < n; ++i) {
    StreamLinear& L = bp.lin[i];
    const long long lo = L.chunk0, hi = L.chunk0 + (long long)L.G * L.C;
    int first = -1, count = 0;
    for (int c = 0; c < nC; ++c) {
      const long long s_lo = total * c / nC, s_hi = total * (c + 1) / nC;
      if (std::max(s_lo, lo) < std::min(s_hi, hi)) { if (first < 0) first = c; ++count; }
    }
    if (first < 0) return PQ_ERR_UNSUPPORTED;
    L.cta_first = first; L.cta_count = count;
  }
  region0 = s_up256(region0);
  bp.off_h = (int)region0;
  bp.off_info = (int)(region0 + s_up256(hbytes));
  const size_t smem = bp.off_info + 256;
  if (smem > kStreamSmemLimit) return PQ_ERR_UNSUPPORTED;
  bp.bar_slot = stream_bar_slot(st);
  if (bp.bar_slot < 0) return PQ_ERR_UNSUPPORTED;
  bp.prefetch = g_decode_stream_prefetch;
  static const bool limit_set = cudaFuncSetAttribute(k_decode_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit) == cudaSuccess;
  if (!limit_set) return PQ_ERR_CUDA;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cudaLaunchConfig_t cfg{};
  cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
  cfg.gridDim = dim3(nC, 1, 1); cfg.blockDim = dim3(kStreamThreads, 1, 1); cfg.dynamicSmemBytes = smem;
  LaunchScope ls(KID_DECODE_STREAM, st);
  if (cudaLaunchKernelEx(&cfg, k_decode_stream, bp) != cudaSuccess) return PQ_ERR_CUDA;
  return PQ_OK;
}

}  // namespace pq
