// Decode path of the pQuant layer (App. A): M <= 16 tokens against weights stored as
// packed sign bits.  The work is bound by the bytes of the weights (N K / 8 bytes of bits,
// 2 r (K + N) bytes per expert in use), so the kernels are built around streaming them once:
//
//   k_decode_prep  one CTA per (linear, token, slice of the r hidden rows): absmax quantisation
//                  of the token (Eq. 7-9), router (Sec. 3.3), and its slice of h = A_e x.
//   k_decode_main  one CTA per SM, each owning a contiguous range of output features of every
//                  linear of the batch.  A producer warp first fetches the routing of all linears,
//                  then streams, linear after linear, the sign bits, the activations and the expert
//                  rows B_e of that range into rings of shared-memory buffers by bulk copies
//                  (mbarrier full/empty pairs), as far ahead as the rings allow.  Each consumer warp
//                  owns whole (linear, token group, 16-feature tile) items: 1-bit product on mma.sync
//                  (u8 bit masks x s8 activations, exact in int32) over all of K, expert product on
//                  bf16 mma.sync, epilogue Y = alpha g (B_e h) + beta (lam / gamma) (q . S)
//                  (Eq. 10-11) straight from its registers; warps never wait for one another.
// A batch is a set of INDEPENDENT linears (the gate and up projections of one block, the q/k/v
// projections, other sequences): their weights then stream back to back.
//
// The sum over k of q S is evaluated as 2 * (sum over the set bits of q) - (sum of q): the bit
// words feed the tensor cores as 0/1 masks without expansion to +-1.
#include <algorithm>

#include "pq_kernels.cuh"

namespace pq {

constexpr int kDecodeMaxConsumerWarps = 16;                 // 8 are launched unless a CTA owns more than 128 features
constexpr int kDecodeMainThreads = 32 * kDecodeMaxConsumerWarps + 32;   // + the producer warp
constexpr int kDecodeMaxTokens = 16;
constexpr int kDecodeMaxSlots = 4;      // linears whose sign bits are in flight or in use per CTA
constexpr int kDecodeMaxQ = 4;          // activation buffers
constexpr int kDecodeMaxRing = 8;       // expert-row buffers
constexpr int kDecodeMaxBatch = 16;     // linears per launch (their descriptors travel as kernel parameters)

struct DecodeTokInfo {  // one per token, written by k_decode_prep
  int expert;
  float gate;
  float gamma;
  int rowsum;           // sum over k of q[k]
};


__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void mma_u8s8(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---------------------------------------------------------------------------
// Layout of the quantised activations handed from prep to main ("q fragments").
// The contraction index k is walked in pairs of 32-bit weight words (64 values of k).  For pair
// ip, the thread of a warp with quad index c (lane & 3) takes from a weight word w the bits
// c + 8 j (mask 0x01010101 of w >> c) and c + 4 + 8 j (mask 0x10101010, i.e. the value 16), j = 0..3.
// Its four 4-byte operand registers for the tokens' side therefore hold, for token g = lane >> 2,
//   r0: q[64 ip      + c     + 8 j]   r1: q[64 ip + 32 + c     + 8 j]      (weight-1 masks)
//   r2: q[64 ip      + c + 4 + 8 j]   r3: q[64 ip + 32 + c + 4 + 8 j]      (weight-16 masks)
// stored as 16 bytes; only the tokens that exist are stored: with Mg = min(8, M - 8 group) tokens in the group,
// the piece of (pair ip, token g, quad index c) sits at uint4 index group * npairs * 32 + (ip * Mg + g) * 4 + c.
// ---------------------------------------------------------------------------

// One linear of a batch: device pointers and sizes (the workspace pointers are carved by the host).
struct DecodeLinear {
  const uint4* X;           // [M, K] bf16
  const uint4* Wr;          // [E, K] bf16 or null
  const uint16_t* A;        // [E, r, K]
  const uint16_t* B;        // [E, N, r]
  const uint32_t* bits;     // [N, K/32]
  const float* w_scales;
  const float* alpha;
  const float* beta;
  uint16_t* Y;              // [M, N]
  DecodeTokInfo* info;      // [16]
  uint4* qfrag;             // [2, npairs, 32] fragments
  uint4* hfrag;             // [2 groups][2 planes (hi, lo)][ceil(r/32)][32] fragments of h = A_e x
  int* acc_dump;            // [M, N] exact 1-bit accumulators (test hook) or null
  const uint4* norm_w;      // [K] bf16 RMSNorm gain or null
  float norm_eps;
  int M, K, N, r, E, sstride, slices, rows_per_slice;
  // partition of the N / 8 feature groups over the CTAs of k_decode_main: the first `grp_rem` CTAs own grp_base + 1 groups
  int grp_base, grp_rem;
};
struct DecodeBatch {
  DecodeLinear lin[kDecodeMaxBatch];
  int n;
  // shared-memory carve-up of k_decode_main (bytes from the 128-byte aligned base)
  int nwarps;               // consumer warps per CTA
  int prep_rows;            // rows of K values k_decode_prep keeps in shared memory beside the token (2..8, two buffers)
  int nslot, nq, nring;     // depths of the three buffer rings
  int off_slots, slot_bytes, off_slot_h, off_q, q_bytes, off_ring, ring_stage_bytes;
};
// position in a ring of buffers with mbarrier full/empty pairs: the producer waits for empty(idx) with
// parity phase ^ 1, a consumer for full(idx) with parity phase
struct DecodeCursor {
  int idx = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void next(int n) { if (++idx == n) { idx = 0; phase ^= 1u; } }
};

// Wait with a bound.  Once any wait of the CTA has run out, every later wait returns at once, so that
// all threads keep the same control flow and the kernel ends (with an error status and undefined output).
__device__ __forceinline__ void decode_wait(uint32_t bar, uint32_t parity, volatile int* fail) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*fail) return;
    if (clock64() - t0 > c_spin_cycles) {
      report_timeout(WHERE_OTHER);
      *fail = 1;
      return;
    }
  }
}

// grid (slices, M, linears), 256 threads.  Dynamic shared memory: the token's K bf16 values, then two buffers of
// `prep_rows` / 2 rows of K bf16 values each (router rows first, rows of A_e afterwards).  Whole rows arrive by bulk
// copies, a round of rows at a time, the next round in flight while one is used, and the dot products run out of
// shared memory: with plain loads every lane went to memory several times in a row for a long row, and that
// latency was most of the kernel.
__global__ void __launch_bounds__(256) k_decode_prep(const __grid_constant__ DecodeBatch bp) {
  extern __shared__ __align__(128) uint4 xs4[];
  __shared__ __align__(8) uint64_t pbar[3];   // token; the two row buffers
  __shared__ float red_f[8];
  __shared__ int red_i[8];
  __shared__ float logit_sh[kMaxExperts];
  __shared__ int fail_sh;
  volatile int* fail = &fail_sh;
  if (threadIdx.x == 0) {
    fail_sh = 0;
    for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&pbar[i]), 1);
    mbar_fence_init();
  }
  pdl_launch_dependents();
  pdl_wait();   // X may come from the previous kernel; the buffers written here may still be read by it
  __syncthreads();
  const DecodeLinear& L = bp.lin[blockIdx.z];
  const int m = blockIdx.y, slice = blockIdx.x;
  if (m >= L.M || slice >= L.slices) return;
  const int K = L.K, E = L.E, r = L.r;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = K >> 3;
  const uint32_t row_bytes = (uint32_t)K * 2u;
  const int R = bp.prep_rows >> 1;                             // rows of one buffer (<= 4, one per warp)
  const uint4* rows4 = xs4 + chunks;
  const uint32_t rows_s = smem_u32(xs4) + row_bytes;
  // rounds of up to R rows of a [*, K] bf16 matrix alternate between the two buffers; all threads count them
  int issued = 0, taken = 0;
  uint32_t phase0 = 0, phase1 = 0;
  auto issue = [&](const uint16_t* base, long long row0, int n) {
    const int b = issued & 1;
    if (threadIdx.x == 0) {
      mbar_expect_tx(smem_u32(&pbar[1 + b]), (uint32_t)n * row_bytes);
      for (int i = 0; i < n; ++i) bulk_load(rows_s + (uint32_t)(b * R + i) * row_bytes, base + (row0 + i) * K, row_bytes, smem_u32(&pbar[1 + b]));
    }
    ++issued;
  };
  auto take = [&]() {   // waits for the oldest round in flight and returns its buffer's first row
    const int b = taken & 1;
    decode_wait(smem_u32(&pbar[1 + b]), b ? phase1 : phase0, fail);
    if (b) phase1 ^= 1u; else phase0 ^= 1u;
    ++taken;
    return rows4 + (size_t)(b * R) * chunks;
  };

  // the token, and with it the first two rounds of router rows
  if (threadIdx.x == 0) {
    mbar_expect_tx(smem_u32(&pbar[0]), row_bytes);
    bulk_load(smem_u32(xs4), reinterpret_cast<const uint16_t*>(L.X) + (long long)m * K, row_bytes, smem_u32(&pbar[0]));
  }
  const uint16_t* Wr = reinterpret_cast<const uint16_t*>(L.Wr);
  const int router_rounds = E > 1 ? (E + R - 1) / R : 0;
  for (int k = 0; k < min(2, router_rounds); ++k) issue(Wr, k * R, min(R, E - k * R));
  decode_wait(smem_u32(&pbar[0]), 0, fail);
  if (L.norm_w) {
    // RMSNorm fused in front of the quantiser (App. A): mean of squares and its reciprocal root in fp64 (thread sums
    // in ascending chunk order, then a fixed tree), the factor rounded once to fp32; the token in shared memory is
    // replaced by bf16(fp32(fp32(x s) w)), which every later step reads.
    __shared__ double red_d[8];
    double ss = 0.0;
    for (int c = threadIdx.x; c < chunks; c += 256) {
      const uint4 v = xs4[c];
      const double d0 = bf16lo(v.x), d1 = bf16hi(v.x), d2 = bf16lo(v.y), d3 = bf16hi(v.y);
      const double d4 = bf16lo(v.z), d5 = bf16hi(v.z), d6 = bf16lo(v.w), d7 = bf16hi(v.w);
      ss += ((d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3)) + ((d4 * d4 + d5 * d5) + (d6 * d6 + d7 * d7));
    }
    for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
    if (lane == 0) red_d[warp] = ss;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red_d[w];
    const float s = (float)(1.0 / sqrt(tot / (double)K + (double)L.norm_eps));
    for (int c = threadIdx.x; c < chunks; c += 256) {
      const uint4 v = xs4[c], g = __ldg(L.norm_w + c);
      uint4 o;
      o.x = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.x), s), bf16lo(g.x)), __fmul_rn(__fmul_rn(bf16hi(v.x), s), bf16hi(g.x)));
      o.y = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.y), s), bf16lo(g.y)), __fmul_rn(__fmul_rn(bf16hi(v.y), s), bf16hi(g.y)));
      o.z = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.z), s), bf16lo(g.z)), __fmul_rn(__fmul_rn(bf16hi(v.z), s), bf16hi(g.z)));
      o.w = pack_bf16x2(__fmul_rn(__fmul_rn(bf16lo(v.w), s), bf16lo(g.w)), __fmul_rn(__fmul_rn(bf16hi(v.w), s), bf16hi(g.w)));
      xs4[c] = o;
    }
    // each thread reads back only the chunks it wrote itself in the pass below; the barrier after it publishes them
  }
  float amax = 0.f;
  for (int c = threadIdx.x; c < chunks; c += 256) {
    const uint4 v = xs4[c];
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.x)), fabsf(bf16hi(v.x))), fmaxf(fabsf(bf16lo(v.y)), fabsf(bf16hi(v.y)))));
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16lo(v.z)), fabsf(bf16hi(v.z))), fmaxf(fabsf(bf16lo(v.w)), fabsf(bf16hi(v.w)))));
  }
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  if (lane == 0) red_f[warp] = amax;
  __syncthreads();
  amax = red_f[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) amax = fmaxf(amax, red_f[w]);
  const float gamma = __fdiv_rn(kActQmax, fmaxf(amax, kActAmaxFloor));

  // router: the same pinned fp32 order as the training path (lane j owns the chunks c = j mod 32, ascending,
  // fused multiply-add; butterfly 16, 8, 4, 2, 1), one warp per expert of the round
  int best = 0;
  float gate = 1.0f;
  if (E > 1) {
    for (int k = 0; k < router_rounds; ++k) {
      const int n = min(R, E - k * R);
      const uint4* buf = take();
      if (warp < n) {
        float acc = 0.f;
        const uint4* wrow = buf + (size_t)warp * chunks;
        for (int c = lane; c < chunks; c += 32) {
          const uint4 xv = xs4[c], wv = wrow[c];
          acc = fmaf(bf16lo(xv.x), bf16lo(wv.x), acc); acc = fmaf(bf16hi(xv.x), bf16hi(wv.x), acc);
          acc = fmaf(bf16lo(xv.y), bf16lo(wv.y), acc); acc = fmaf(bf16hi(xv.y), bf16hi(wv.y), acc);
          acc = fmaf(bf16lo(xv.z), bf16lo(wv.z), acc); acc = fmaf(bf16hi(xv.z), bf16hi(wv.z), acc);
          acc = fmaf(bf16lo(xv.w), bf16lo(wv.w), acc); acc = fmaf(bf16hi(xv.w), bf16hi(wv.w), acc);
        }
        for (int d = 16; d > 0; d >>= 1) acc = acc + __shfl_xor_sync(0xffffffffu, acc, d);
        if (lane == 0) logit_sh[k * R + warp] = acc;
      }
      __syncthreads();                                         // this buffer is free, its logits are visible
      if (k + 2 < router_rounds) issue(Wr, (k + 2) * R, min(R, E - (k + 2) * R));
    }
    float lmax = logit_sh[0];
    for (int e = 1; e < E; ++e)
      if (logit_sh[e] > lmax) { lmax = logit_sh[e]; best = e; }
    float den = 0.f, pbest = 0.f;
    for (int e = 0; e < E; ++e) {
      const float pe = expf(logit_sh[e] - lmax);
      den += pe;
      if (e == best) pbest = pe;
    }
    gate = pbest * (1.0f / den);
  }
  // the first two rounds of this slice's rows of A_e are on their way while slice 0 quantises the token
  const int j0 = slice * L.rows_per_slice, j1 = min(r, j0 + L.rows_per_slice);
  const int h_rounds = (r > 0 && j0 < j1) ? (j1 - j0 + R - 1) / R : 0;
  const long long arow0 = (long long)best * r + j0;
  for (int k = 0; k < min(2, h_rounds); ++k) issue(L.A, arow0 + k * R, min(R, j1 - j0 - k * R));

  if (slice == 0) {
    // Eq. 7-9 for this token; every thread turns pairs of weight words (64 values of k) into fragment order
    const int npairs = (K + 63) >> 6;
    const int group = m >> 3, g = m & 7, mg = min(8, L.M - 8 * group);
    int rowsum = 0;
    for (int ip = threadIdx.x; ip < npairs; ip += 256) {
      int qv[64];
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        const bool in = 8 * ip + ch < chunks;
        const uint4 v = in ? xs4[8 * ip + ch] : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int q0 = in ? max(-128, min(127, __float2int_rn(__fmul_rn(bf16lo(w[u]), gamma)))) : 0;
          const int q1 = in ? max(-128, min(127, __float2int_rn(__fmul_rn(bf16hi(w[u]), gamma)))) : 0;
          qv[8 * ch + 2 * u] = q0;
          qv[8 * ch + 2 * u + 1] = q1;
          rowsum += q0 + q1;
        }
      }
      uint4 out[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t w[4];
#pragma unroll
        for (int reg = 0; reg < 4; ++reg) {
          const int base = (reg & 1) * 32 + c + (reg >> 1) * 4;
          w[reg] = (qv[base] & 0xFF) | ((qv[base + 8] & 0xFF) << 8) | ((qv[base + 16] & 0xFF) << 16) | ((qv[base + 24] & 0xFF) << 24);
        }
        out[c] = make_uint4(w[0], w[1], w[2], w[3]);
      }
      uint4* dst = L.qfrag + ((long long)group * npairs * 32 + (long long)(ip * mg + g) * 4);
#pragma unroll
      for (int c = 0; c < 4; ++c) dst[c] = out[c];
    }
    for (int d = 16; d > 0; d >>= 1) rowsum += __shfl_xor_sync(0xffffffffu, rowsum, d);
    if (lane == 0) red_i[warp] = rowsum;
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int w = 0; w < 8; ++w) tot += red_i[w];
      L.info[m] = DecodeTokInfo{best, gate, gamma, tot};
    }
  }

  // this slice of h = A_e x (fp32 accumulation over the bf16 operands), one warp per row of the round
  for (int k = 0; k < h_rounds; ++k) {
    const int n = min(R, j1 - j0 - k * R);
    const uint4* buf = take();
    if (warp < n) {
      const int j = j0 + k * R + warp;
      const uint4* arow = buf + (size_t)warp * chunks;
      float a0 = 0.f, a1 = 0.f;
      for (int c = lane; c < chunks; c += 32) {
        const uint4 xv = xs4[c], wv = arow[c];
        a0 = fmaf(bf16lo(xv.x), bf16lo(wv.x), a0); a1 = fmaf(bf16hi(xv.x), bf16hi(wv.x), a1);
        a0 = fmaf(bf16lo(xv.y), bf16lo(wv.y), a0); a1 = fmaf(bf16hi(xv.y), bf16hi(wv.y), a1);
        a0 = fmaf(bf16lo(xv.z), bf16lo(wv.z), a0); a1 = fmaf(bf16hi(xv.z), bf16hi(wv.z), a1);
        a0 = fmaf(bf16lo(xv.w), bf16lo(wv.w), a0); a1 = fmaf(bf16hi(xv.w), bf16hi(wv.w), a1);
      }
      float a = a0 + a1;
      for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
      if (lane == 0) {
        // element (token m, hidden index j) of the expert product's token-side operand: step j / 32, lane
        // 4 (m % 8) + (j % 32) / 8, 16-bit slot j % 8; hi = bf16(a), lo = bf16(a - hi)
        const int rsteps = (r + 31) >> 5;
        const __nv_bfloat16 hi = __float2bfloat16_rn(a), lo = __float2bfloat16_rn(a - __bfloat162float(hi));
        uint16_t* base = reinterpret_cast<uint16_t*>(L.hfrag);
        const long long pos = ((long long)((m >> 3) * 2 * rsteps + (j >> 5)) * 32 + (m & 7) * 4 + ((j & 31) >> 3)) * 8 + (j & 7);
        base[pos] = __bfloat16_as_ushort(hi);
        base[pos + (long long)rsteps * 32 * 8] = __bfloat16_as_ushort(lo);
      }
    }
    if (k + 2 < h_rounds) {
      __syncthreads();                                         // this buffer is free
      issue(L.A, arow0 + (k + 2) * R, min(R, j1 - j0 - (k + 2) * R));
    }
  }
}

// Range of output features of CTA b: whole groups of 8, spread evenly (no division on the device).
__device__ __forceinline__ void decode_range(int b, const DecodeLinear& L, int& n_lo, int& n_hi) {
  n_lo = (b * L.grp_base + min(b, L.grp_rem)) << 3;
  n_hi = n_lo + ((L.grp_base + (b < L.grp_rem ? 1 : 0)) << 3);
}
constexpr int kDecodeMetaBytes = 256;   // token info at the start of a slot

// Experts used by the tokens [8 G, 8 G + 8) as a bit mask; producer and consumers walk it in ascending order.
__device__ __forceinline__ unsigned decode_expert_mask(const DecodeTokInfo* tok, int M, int G) {
  unsigned mask = 0u;
  for (int t = 8 * G; t < min(M, 8 * G + 8); ++t) mask |= 1u << (tok[t].expert & 15);
  return mask;
}

__global__ void __launch_bounds__(kDecodeMainThreads) k_decode_main(const __grid_constant__ DecodeBatch bp) {
  extern __shared__ __align__(128) uint8_t smem[];
  // barriers: token info; slot, q and expert-row rings, a full/empty pair per buffer
  __shared__ __align__(8) uint64_t bars[1 + 2 * kDecodeMaxSlots + 2 * kDecodeMaxQ + 2 * kDecodeMaxRing];
  __shared__ int fail_sh;
  volatile int* fail = &fail_sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(&bars[0]);
  const uint32_t info_full = bar0;
  auto slot_full = [&](int s) { return bar0 + 8u * (1 + s); };
  auto slot_empty = [&](int s) { return bar0 + 8u * (1 + kDecodeMaxSlots + s); };
  auto q_full = [&](int i) { return bar0 + 8u * (1 + 2 * kDecodeMaxSlots + i); };
  auto q_empty = [&](int i) { return bar0 + 8u * (1 + 2 * kDecodeMaxSlots + kDecodeMaxQ + i); };
  auto ring_full = [&](int i) { return bar0 + 8u * (1 + 2 * kDecodeMaxSlots + 2 * kDecodeMaxQ + i); };
  auto ring_empty = [&](int i) { return bar0 + 8u * (1 + 2 * kDecodeMaxSlots + 2 * kDecodeMaxQ + kDecodeMaxRing + i); };
  if (threadIdx.x == 0) {
    fail_sh = 0;
    mbar_init(info_full, 1);
    for (int s = 0; s < bp.nslot; ++s) { mbar_init(slot_full(s), 1); mbar_init(slot_empty(s), bp.nwarps); }
    for (int s = 0; s < bp.nq; ++s) { mbar_init(q_full(s), 1); mbar_init(q_empty(s), bp.nwarps); }
    for (int s = 0; s < bp.nring; ++s) { mbar_init(ring_full(s), 1); mbar_init(ring_empty(s), bp.nwarps); }
    mbar_fence_init();
  }
  pdl_launch_dependents();
  __syncthreads();
  if (warp != bp.nwarps) pdl_wait();   // the producer waits later: weights do not depend on the previous kernel

  // token info of every linear of the batch sits at the start; a slot holds, for one linear, the sign bits
  // of this CTA's features | the h fragments (both groups)
  auto info_ptr = [&](int l) { return reinterpret_cast<const DecodeTokInfo*>(smem + l * kDecodeMetaBytes); };
  auto slot_ptr = [&](int s) { return smem + bp.off_slots + (size_t)s * bp.slot_bytes; };
  uint4* q_s = reinterpret_cast<uint4*>(smem + bp.off_q);
  uint8_t* ring = smem + bp.off_ring;

  if (warp == bp.nwarps) {
    // ------------------------------------------------------------------ producer (one thread issues everything)
    if (lane != 0) return;
    // The sign bits of the first linears (as many as there are slots) go out before the previous kernel, which
    // prepares this one's tokens, is known to have finished: weights are not its output.
    int early = 0;
    {
      DecodeCursor c0;
      for (int l = 0; l < bp.n && early < bp.nslot; ++l) {
        const DecodeLinear& L = bp.lin[l];
        int n_lo, n_hi;
        decode_range(blockIdx.x, L, n_lo, n_hi);
        const int ncols = n_hi - n_lo;
        if (ncols == 0) continue;
        const uint32_t bits_bytes = (uint32_t)ncols * (uint32_t)(L.K >> 3);
        const uint32_t h_bytes = L.r > 0 ? (uint32_t)(((L.M + 7) >> 3) * 2 * ((L.r + 31) >> 5)) * 512u : 0u;
        mbar_expect_tx(slot_full(c0.idx), bits_bytes + h_bytes);
        bulk_load(smem_u32(slot_ptr(c0.idx)), L.bits + (long long)n_lo * (L.K >> 5), bits_bytes, slot_full(c0.idx));
        c0.next(bp.nslot);
        ++early;
      }
    }
    pdl_wait();
    // The routing of every linear's tokens first: it decides which expert rows are fetched, and with it in
    // hand nothing below waits for data, only for free buffers, so the loads run as far ahead as the rings allow.
    mbar_expect_tx(info_full, (uint32_t)bp.n * kDecodeMetaBytes);
    for (int l = 0; l < bp.n; ++l) bulk_load(smem_u32(smem + l * kDecodeMetaBytes), bp.lin[l].info, kDecodeMetaBytes, info_full);
    decode_wait(info_full, 0, fail);
    if (*fail) return;                                       // nothing below may be issued from data that never arrived
    DecodeCursor cs, cq, cr;
    for (int l = 0; l < bp.n; ++l) {
      const DecodeLinear& L = bp.lin[l];
      int n_lo, n_hi;
      decode_range(blockIdx.x, L, n_lo, n_hi);
      const int ncols = n_hi - n_lo;
      if (ncols == 0) continue;
      {
        const uint32_t bits_bytes = (uint32_t)ncols * (uint32_t)(L.K >> 3);
        const uint32_t h_bytes = L.r > 0 ? (uint32_t)(((L.M + 7) >> 3) * 2 * ((L.r + 31) >> 5)) * 512u : 0u;
        if (early > 0) {
          --early;                                          // bits already on their way
        } else {
          decode_wait(slot_empty(cs.idx), cs.phase ^ 1u, fail);
          if (*fail) return;
          mbar_expect_tx(slot_full(cs.idx), bits_bytes + h_bytes);
          bulk_load(smem_u32(slot_ptr(cs.idx)), L.bits + (long long)n_lo * (L.K >> 5), bits_bytes, slot_full(cs.idx));
        }
        if (h_bytes) bulk_load(smem_u32(slot_ptr(cs.idx) + bp.off_slot_h), L.hfrag, h_bytes, slot_full(cs.idx));
        cs.next(bp.nslot);
      }
      const int npairs = ((L.K >> 5) + 1) >> 1;
      const uint32_t row_bytes = (uint32_t)L.r * 2u;
      const int ngroups = (L.M + 7) >> 3;
      for (int G = 0; G < ngroups; ++G) {
        const uint32_t q_bytes = (uint32_t)(npairs * min(8, L.M - 8 * G)) * 64u;
        decode_wait(q_empty(cq.idx), cq.phase ^ 1u, fail);
        if (*fail) return;
        mbar_expect_tx(q_full(cq.idx), q_bytes);
        bulk_load(smem_u32(q_s) + cq.idx * bp.q_bytes, L.qfrag + (long long)G * npairs * 32, q_bytes, q_full(cq.idx));
        cq.next(bp.nq);
        unsigned emask = L.r > 0 ? decode_expert_mask(info_ptr(l), L.M, G) : 0u;
        for (; emask; emask &= emask - 1) {
          const int e = __ffs(emask) - 1;
          decode_wait(ring_empty(cr.idx), cr.phase ^ 1u, fail);
          if (*fail || e >= L.E) return;
          mbar_expect_tx(ring_full(cr.idx), (uint32_t)ncols * row_bytes);
          bulk_load(smem_u32(ring + cr.idx * bp.ring_stage_bytes), L.B + ((long long)e * L.N + n_lo) * L.r,
                    (uint32_t)ncols * row_bytes, ring_full(cr.idx));
          cr.next(bp.nring);
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  // The work of a CTA is a list of items (linear, token group, tile of 16 features), in that order; item i
  // belongs to warp i mod nwarps, which contracts over all of K, adds the expert product and writes the 16 x 8
  // outputs: no warp waits for another.  Every warp walks every buffer of the three rings in the producer's
  // order, waits for it to be full and hands it back exactly once (the empty barriers count nwarps arrivals),
  // whether it used it or not: a warp that skipped ahead without waiting could arrive twice in one phase.
  const int g = lane >> 2, c = lane & 3;
  DecodeCursor cs, cq, cr;
  decode_wait(info_full, 0, fail);
  int base_mod = 0;                                          // (items before the current (linear, group)) mod nwarps
  for (int l = 0; l < bp.n; ++l) {
    const DecodeLinear& L = bp.lin[l];
    int n_lo, n_hi;
    decode_range(blockIdx.x, L, n_lo, n_hi);
    const int ncols = n_hi - n_lo;
    if (ncols == 0) continue;
    const int ntile = (ncols + 15) >> 4;                     // <= nwarps (checked by the host)
    const int nks = L.K >> 5, npairs = (nks + 1) >> 1;
    const int rsteps = (L.r + 31) >> 5;                      // 32 hidden values per step of the expert product
    const uint32_t row_bytes = (uint32_t)L.r * 2u;
    const int ngroups = (L.M + 7) >> 3;
    const DecodeTokInfo* tok = info_ptr(l);
    const int s = cs.idx;
    decode_wait(slot_full(s), cs.phase, fail);
    cs.next(bp.nslot);
    const uint32_t* bits_s = reinterpret_cast<const uint32_t*>(slot_ptr(s));
    const uint4* h_all = reinterpret_cast<const uint4*>(slot_ptr(s) + bp.off_slot_h);

    for (int G = 0; G < ngroups; ++G) {
      int my_tile = warp - base_mod;                         // tile j of this (linear, group) is item base + j
      if (my_tile < 0) my_tile += bp.nwarps;
      const bool mine = my_tile < ntile;
      base_mod += ntile;
      if (base_mod >= bp.nwarps) base_mod -= bp.nwarps;
      unsigned emask = L.r > 0 ? decode_expert_mask(tok, L.M, G) : 0u;
      const int qb = cq.idx;
      const uint32_t q_phase = cq.phase;
      cq.next(bp.nq);
      if (!mine) {
        // nothing of this group is this warp's: hand its buffers back as they arrive
        decode_wait(q_full(qb), q_phase, fail);
        if (lane == 0) mbar_arrive(q_empty(qb));
        for (; emask; emask &= emask - 1) {
          decode_wait(ring_full(cr.idx), cr.phase, fail);
          if (lane == 0) mbar_arrive(ring_empty(cr.idx));
          cr.next(bp.nring);
        }
        continue;
      }
      const int row0 = 16 * my_tile + g, row1 = row0 + 8;    // this thread's two features (local index)
      const bool has0 = row0 < ncols, has1 = row1 < ncols;
      // per-feature factors of the epilogue, fetched before anything is waited for
      float lam = L.w_scales[0];
      float be0 = 0.f, be1 = 0.f, al0 = 0.f, al1 = 0.f;
      if (has0) { be0 = L.beta[(n_lo + row0) * L.sstride]; if (L.r > 0) al0 = L.alpha[(n_lo + row0) * L.sstride]; }
      if (has1) { be1 = L.beta[(n_lo + row1) * L.sstride]; if (L.r > 0) al1 = L.alpha[(n_lo + row1) * L.sstride]; }
      const int mg = min(8, L.M - 8 * G);
      decode_wait(q_full(qb), q_phase, fail);
      // the epilogue's factors are in registers from here on: their loads were issued before the wait and must not
      // be moved down to their first use, where a warp would sit out a trip to global memory per tile
      asm volatile("" : "+f"(lam), "+f"(be0), "+f"(be1), "+f"(al0), "+f"(al1));

      // ---- 1-bit product: masked sums, weight 1 and weight 16; two independent chains of accumulators.
      // Threads of tokens that do not exist read the last token's fragments (their results are never stored),
      // threads of features beyond the range read feature 0.
      int acc1[4] = {0, 0, 0, 0}, acc16[4] = {0, 0, 0, 0}, bcc1[4] = {0, 0, 0, 0}, bcc16[4] = {0, 0, 0, 0};
      {
        const uint4* qp = reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(q_s) + qb * bp.q_bytes) + min(g, mg - 1) * 4 + c;
        const int qstep = mg * 4;
        const uint32_t* w0 = bits_s + (has0 ? row0 : 0) * nks;
        const uint32_t* w1 = bits_s + (has1 ? row1 : 0) * nks;
        auto mac = [&](uint32_t x00, uint32_t x01, uint32_t x10, uint32_t x11, const uint4& qv, int (&x1)[4], int (&x16)[4]) {
          const uint32_t t00 = x00 >> c, t01 = x01 >> c, t10 = x10 >> c, t11 = x11 >> c;
          const uint32_t a1[4] = {t00 & 0x01010101u, t10 & 0x01010101u, t01 & 0x01010101u, t11 & 0x01010101u};
          const uint32_t a16[4] = {t00 & 0x10101010u, t10 & 0x10101010u, t01 & 0x10101010u, t11 & 0x10101010u};
          mma_u8s8(x1, a1, qv.x, qv.y);
          mma_u8s8(x16, a16, qv.z, qv.w);
        };
        if ((nks & 1) == 0) {
          // Rows are 8-byte aligned: one load per pair of weight words.  Software pipeline without branches:
          // two register sets of four steps each; while one is multiplied the other is being loaded (the
          // loads past the end are clamped to the last step and never used).
          const uint2* v0 = reinterpret_cast<const uint2*>(w0);
          const uint2* v1 = reinterpret_cast<const uint2*>(w1);
          struct Set { uint2 a[4], b[4]; uint4 q[4]; };
          const int last = npairs - 1;
          auto fetch = [&](Set& f, int ip) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int i = min(ip + j, last);
              f.a[j] = v0[i]; f.b[j] = v1[i]; f.q[j] = qp[i * qstep];
            }
          };
          auto macs = [&](const Set& f) {
            mac(f.a[0].x, f.a[0].y, f.b[0].x, f.b[0].y, f.q[0], acc1, acc16);
            mac(f.a[1].x, f.a[1].y, f.b[1].x, f.b[1].y, f.q[1], bcc1, bcc16);
            mac(f.a[2].x, f.a[2].y, f.b[2].x, f.b[2].y, f.q[2], acc1, acc16);
            mac(f.a[3].x, f.a[3].y, f.b[3].x, f.b[3].y, f.q[3], bcc1, bcc16);
          };
          Set A, B;
          int ip = 0;
          fetch(A, 0);
          for (; ip + 8 <= npairs; ip += 8) {
            fetch(B, ip + 4);
            macs(A);
            fetch(A, ip + 8);
            macs(B);
          }
          // fewer than eight steps left; A holds steps ip .. ip + 3 (clamped)
          if (ip + 4 <= npairs) { macs(A); ip += 4; fetch(A, ip); }
          for (int j = 0; ip + j < npairs; ++j) {
            if (j == 0) mac(A.a[0].x, A.a[0].y, A.b[0].x, A.b[0].y, A.q[0], acc1, acc16);
            if (j == 1) mac(A.a[1].x, A.a[1].y, A.b[1].x, A.b[1].y, A.q[1], bcc1, bcc16);
            if (j == 2) mac(A.a[2].x, A.a[2].y, A.b[2].x, A.b[2].y, A.q[2], acc1, acc16);
          }
        } else {
          for (int ip = 0; ip < npairs; ++ip) {
            const int i0 = 2 * ip, i1 = min(2 * ip + 1, nks - 1);   // the odd last word pairs with zeros of q
            mac(w0[i0], w0[i1], w1[i0], w1[i1], qp[ip * qstep], acc1, acc16);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(q_empty(qb));              // this warp is done with the q fragments
      // ---- expert product z = B_e h, tokens of other experts masked out; four independent chains
      float z0[4] = {0.f, 0.f, 0.f, 0.f}, z1[4] = {0.f, 0.f, 0.f, 0.f}, z2[4] = {0.f, 0.f, 0.f, 0.f}, z3[4] = {0.f, 0.f, 0.f, 0.f};
      const int my_tok = 8 * G + g;                          // the token whose h this thread feeds
      const int my_tok_e = my_tok < L.M ? tok[my_tok].expert : -1;
      const uint4* h_hi = h_all + (size_t)(G * 2) * rsteps * 32;
      const uint4* h_lo = h_hi + (size_t)rsteps * 32;
      for (; emask; emask &= emask - 1) {
        const int e = __ffs(emask) - 1;
        const int stage = cr.idx;
        decode_wait(ring_full(stage), cr.phase, fail);
        cr.next(bp.nring);
        const uint8_t* rows = ring + stage * bp.ring_stage_bytes;
        const uint4* r0p = reinterpret_cast<const uint4*>(rows + (has0 ? row0 : 0) * row_bytes);
        const uint4* r1p = reinterpret_cast<const uint4*>(rows + (has1 ? row1 : 0) * row_bytes);
        const bool feeds = my_tok_e == e;
        for (int st = 0; st < rsteps; ++st) {
          const int chunk = 4 * st + c;
          const bool in = chunk * 8 < L.r;
          uint4 b0 = make_uint4(0, 0, 0, 0), b1 = b0, hh = b0, hl = b0;
          if (in) { b0 = r0p[chunk]; b1 = r1p[chunk]; }
          if (feeds && in) { hh = h_hi[st * 32 + lane]; hl = h_lo[st * 32 + lane]; }
          mma_bf16(z0, b0.x, b1.x, b0.y, b1.y, hh.x, hh.y);
          mma_bf16(z1, b0.z, b1.z, b0.w, b1.w, hh.z, hh.w);
          mma_bf16(z2, b0.x, b1.x, b0.y, b1.y, hl.x, hl.y);
          mma_bf16(z3, b0.z, b1.z, b0.w, b1.w, hl.z, hl.w);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(ring_empty(stage));      // this warp is done with the buffer
      }

      // ---- epilogue (Eq. 10-11)
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        // accumulator u: feature row0 (u < 2) or row1, token 8G + 2c + (u & 1)
        const int nl = (u < 2) ? row0 : row1, t = 8 * G + 2 * c + (u & 1);
        if (nl < ncols && t < L.M) {
          const int n = n_lo + nl;
          const int m = (acc1[u] + bcc1[u]) + ((acc16[u] + bcc16[u]) >> 4);   // the weight-16 sums are exact multiples of 16
          const int acc = 2 * m - tok[t].rowsum;
          float y = ((u < 2) ? be0 : be1) * __fdiv_rn(lam, tok[t].gamma) * (float)acc;
          if (L.r > 0) y = fmaf(((u < 2) ? al0 : al1) * tok[t].gate, (z0[u] + z1[u]) + (z2[u] + z3[u]), y);
          L.Y[(long long)t * L.N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
          if (L.acc_dump) L.acc_dump[(long long)t * L.N + n] = acc;
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(slot_empty(s));               // this warp is done with the slot of linear l
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

size_t decode_workspace_bytes(int M, int K, int N, int r, bool dump) {
  const size_t npairs = ((size_t)K / 32 + 1) / 2;
  size_t b = up256(sizeof(DecodeTokInfo) * kDecodeMaxTokens);
  b += up256(2 * npairs * 32 * sizeof(uint4));
  b += up256((size_t)2 * 2 * ((r + 31) / 32 > 0 ? (r + 31) / 32 : 1) * 512);
  if (dump) b += up256(sizeof(int) * (size_t)M * N);
  return b;
}

DecodeViewPtrs decode_view(int M, int K, int N, int r, void* ws, bool dump) {
  uint8_t* w = static_cast<uint8_t*>(ws);
  const size_t npairs = ((size_t)K / 32 + 1) / 2;
  DecodeViewPtrs v{w, nullptr};
  w += up256(sizeof(DecodeTokInfo) * kDecodeMaxTokens) + up256(2 * npairs * 32 * sizeof(uint4)) +
       up256((size_t)2 * 2 * ((r + 31) / 32 > 0 ? (r + 31) / 32 : 1) * 512);
  if (dump) v.acc = reinterpret_cast<int*>(w);
  (void)M; (void)N;
  return v;
}

// Launch option: programmatic stream serialisation of the two decode kernels (on by default).
static int g_decode_pdl = 1;
void decode_set_pdl(int on) { g_decode_pdl = on ? 1 : 0; }

static int decode_sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  return n;
}

constexpr size_t kDecodeMainSmemLimit = 226 * 1024;   // dynamic shared memory of k_decode_main (its barriers are static)
constexpr size_t kDecodePrepSmemLimit = 200 * 1024;   // K bf16 values of one token

// One launch pair for up to kDecodeMaxBatch independent linears.
static int decode_launch_with(const DecodeItemArgs* items, int n, int nwarps, cudaStream_t st) {
  static int sms = decode_sm_count();
  // One CTA per SM.  Eight consumer warps keep up with what the buffer rings can hold in flight (measured: more warps,
  // or two smaller CTAs per SM, are not faster); sixteen only when a CTA's feature range needs more than eight tiles.
  const int nctas = sms;
  const size_t smem_limit = kDecodeMainSmemLimit;
  DecodeBatch bp{};
  bp.n = n; bp.nwarps = nwarps;
  size_t slot_bits = 0, slot_h = 0, q_bytes = 0, ring_stage = 0, prep_smem = 0;
  int max_slices = 1, max_m = 1, max_k = 0;
  for (int i = 0; i < n; ++i) {
    const DecodeItemArgs& it = items[i];
    const int M = it.a.T, K = it.a.K, N = it.a.N, r = it.a.r;
    DecodeLinear& L = bp.lin[i];
    uint8_t* w = static_cast<uint8_t*>(it.ws);
    const size_t npairs = ((size_t)K / 32 + 1) / 2;
    L.info = reinterpret_cast<DecodeTokInfo*>(w); w += up256(sizeof(DecodeTokInfo) * kDecodeMaxTokens);
    L.qfrag = reinterpret_cast<uint4*>(w); w += up256(2 * npairs * 32 * sizeof(uint4));
    L.hfrag = reinterpret_cast<uint4*>(w); w += up256((size_t)2 * 2 * ((r + 31) / 32 > 0 ? (r + 31) / 32 : 1) * 512);
    L.acc_dump = it.dump ? reinterpret_cast<int*>(w) : nullptr;
    L.X = reinterpret_cast<const uint4*>(it.X); L.Wr = reinterpret_cast<const uint4*>(it.a.Wr); L.A = it.a.A; L.B = it.a.B;
    L.bits = it.bits; L.w_scales = it.a.w_scales; L.alpha = it.a.alpha; L.beta = it.a.beta; L.Y = it.Y;
    L.norm_w = reinterpret_cast<const uint4*>(it.norm_weight); L.norm_eps = it.norm_eps;
    L.M = M; L.K = K; L.N = N; L.r = r; L.E = (r > 0 && it.a.E > 1) ? it.a.E : 1; L.sstride = it.a.scale_stride;
    if (M > max_m) max_m = M;
    const int groups = N / 8;
    L.grp_base = groups / nctas; L.grp_rem = groups % nctas;
    const int max_cols = ((groups + nctas - 1) / nctas) * 8;
    if (max_cols > 16 * nwarps) return PQ_ERR_UNSUPPORTED;       // at most one tile of 16 features per warp and token group
    slot_bits = std::max(slot_bits, up256((size_t)max_cols * (K / 8)));
    slot_h = std::max(slot_h, r > 0 ? up256((size_t)((M + 7) / 8) * 2 * ((r + 31) / 32) * 512) : (size_t)0);   // token groups in use only
    q_bytes = std::max(q_bytes, up256(npairs * (size_t)std::min(M, 8) * 64));
    ring_stage = std::max(ring_stage, up256((size_t)max_cols * r * 2));
    max_k = std::max(max_k, K);
  }
  // Buffer rings: at least two slots, one activation buffer and (with experts) two expert-row buffers; then
  // deeper, in turn, while shared memory lasts, so that the loads of several linears are in flight at once.
  const size_t slot_bytes = slot_bits + slot_h;
  const size_t fixed = (size_t)n * kDecodeMetaBytes + 128;
  const bool experts = ring_stage > 0;
  bp.nslot = 2; bp.nq = 1; bp.nring = experts ? 2 : 1;
  auto total = [&](int ns, int nq, int nr) { return fixed + ns * slot_bytes + nq * q_bytes + nr * ring_stage; };
  for (bool grew = true; grew;) {
    grew = false;
    if (bp.nslot < kDecodeMaxSlots && total(bp.nslot + 1, bp.nq, bp.nring) <= smem_limit) { ++bp.nslot; grew = true; }
    if (experts && bp.nring < kDecodeMaxRing && total(bp.nslot, bp.nq, bp.nring + 1) <= smem_limit) { ++bp.nring; grew = true; }
    if (bp.nq < kDecodeMaxQ && bp.nq < bp.nslot * ((max_m + 7) / 8) && total(bp.nslot, bp.nq + 1, bp.nring) <= smem_limit) { ++bp.nq; grew = true; }
  }
  size_t off = (size_t)n * kDecodeMetaBytes;
  bp.off_slots = (int)off; bp.off_slot_h = (int)slot_bits; bp.slot_bytes = (int)slot_bytes;
  off += bp.nslot * slot_bytes;
  bp.q_bytes = (int)q_bytes;
  bp.off_q = (int)off; off += bp.nq * q_bytes;
  bp.ring_stage_bytes = (int)ring_stage;
  bp.off_ring = (int)off; off += bp.nring * ring_stage;
  const size_t smem_main = off + 128;
  if (smem_main > smem_limit) {
    return PQ_ERR_UNSUPPORTED;
  }
  // token preparation: the token and up to eight rows (router rows, then rows of A_e) of K bf16 values each
  bp.prep_rows = (int)std::min<size_t>(8, (kDecodePrepSmemLimit - (size_t)max_k * 2) / ((size_t)max_k * 2)) & ~1;   // two buffers
  if (bp.prep_rows < 2) return PQ_ERR_UNSUPPORTED;
  prep_smem = (size_t)max_k * 2 * (1 + bp.prep_rows);
  // Slices of the hidden rows: whole rounds of rows, as many slices as keep the grid within
  // one wave of resident CTAs (every slice repeats the token's absmax and router, and rounds run one after another).
  const int resident = sms * std::max<int>(1, (int)((227 * 1024) / (prep_smem + 1024)));
  int total_tokens = 0;
  for (int i = 0; i < n; ++i) total_tokens += items[i].a.T;
  for (int i = 0; i < n; ++i) {
    DecodeLinear& L = bp.lin[i];
    L.slices = 1; L.rows_per_slice = 1;
    if (L.r > 0) {
      int slices = std::max(1, resident / std::max(1, total_tokens));
      slices = std::min(slices, (L.r + 7) / 8);
      const int round_rows = bp.prep_rows / 2;
      L.rows_per_slice = ((L.r + slices - 1) / slices + round_rows - 1) / round_rows * round_rows;
      L.slices = (L.r + L.rows_per_slice - 1) / L.rows_per_slice;
    }
    max_slices = std::max(max_slices, L.slices);
  }
  // The opt-in limits are set once, to the largest request this file can make: a launch recorded in a CUDA graph
  // keeps its own shared-memory size, and a later call with a smaller one must not lower the limit under it.
  static const bool limits_set =
      cudaFuncSetAttribute(k_decode_main, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecodeMainSmemLimit) == cudaSuccess &&
      cudaFuncSetAttribute(k_decode_prep, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecodePrepSmemLimit) == cudaSuccess;
  if (!limits_set) return PQ_ERR_CUDA;

  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = g_decode_pdl ? 1 : 0;
  {
    cfg.gridDim = dim3(max_slices, max_m, n); cfg.blockDim = dim3(256, 1, 1); cfg.dynamicSmemBytes = prep_smem;
    LaunchScope ls(KID_DECODE_PREP, st);
    if (cudaLaunchKernelEx(&cfg, k_decode_prep, bp) != cudaSuccess) return PQ_ERR_CUDA;
  }
  {
    cfg.gridDim = dim3(nctas, 1, 1); cfg.blockDim = dim3(32 * nwarps + 32, 1, 1); cfg.dynamicSmemBytes = smem_main;
    LaunchScope ls(KID_DECODE_MAIN, st);
    if (cudaLaunchKernelEx(&cfg, k_decode_main, bp) != cudaSuccess) return PQ_ERR_CUDA;
  }
  return PQ_OK;
}

static int decode_launch(const DecodeItemArgs* items, int n, cudaStream_t st) {
  const int rc = decode_launch_with(items, n, 8, st);
  return rc == PQ_ERR_UNSUPPORTED ? decode_launch_with(items, n, kDecodeMaxConsumerWarps, st) : rc;
}

// the launch groups of the streaming kernel are larger than those of the two-kernel path (defined in pq_decode_stream.cu)
int decode_stream_max_batch();

int decode_batch(const DecodeItemArgs* items, int n, cudaStream_t st) {
  int i = 0;
  while (i < n) {
    // The streaming kernel takes a group whose items all carry its weight layout, where it pays.  (Measured on the 3B
    // shapes: its grid barrier and its longer chain of dependent steps cost about as much as eight linears' worth of
    // streaming, so small groups, and mid-sized groups of many tokens, stay on the two kernels above.)
    const int mode_opt = decode_stream_mode();
    int m = std::min(n - i, decode_stream_max_batch());
    bool all = true, hp8 = false;
    int max_m = 1, run = 0;
    for (int k = 0; k < m; ++k) {
      if (!items[i + k].bits_il) { all = false; break; }
      ++run;
      hp8 = hp8 || items[i + k].A8 != nullptr;
      max_m = std::max(max_m, items[i + k].a.T);
    }
    int rc = PQ_ERR_UNSUPPORTED;
    if (!all) m = run;                                       // the items in front that carry the layout, if any
    const int mode = hp8 ? 2 : mode_opt;
    if (m > 0 && mode > 0 && (mode > 1 || hp8 || m >= 12 || (m >= 6 && max_m <= 2))) {
      rc = decode_stream_launch(items + i, m, st);
      if (hp8 && rc == PQ_ERR_UNSUPPORTED) return rc;        // the INT8 branch exists on the streaming kernel only
    }
    if (rc == PQ_ERR_UNSUPPORTED) {
      // the two-kernel path: the same run of items that carry the layout, or the run in front that does not
      if (m == 0)
        while (i + m < n && m < kDecodeMaxBatch && !items[i + m].bits_il) ++m;
      m = std::min(m, kDecodeMaxBatch);
      for (int k = 0; k < m; ++k)
        if (items[i + k].A8) return PQ_ERR_UNSUPPORTED;
      rc = decode_launch(items + i, m, st);
    }
    if (rc) return rc;
    i += m;
  }
  return PQ_OK;
}

int decode_forward(const LayerArgs& a, const uint16_t* X, const uint32_t* bits, uint16_t* Y, void* ws, bool dump, cudaStream_t st) {
  DecodeItemArgs it{a, X, bits, Y, ws, dump};
  return decode_launch(&it, 1, st);
}

}  // namespace pq
