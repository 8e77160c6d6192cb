// C ABI of the pQuant layer: argument checks, carving of the caller's saved /
// workspace buffers, launch sequencing.  No device allocation, no device
// synchronisation (except pq_device_status, which says so).
#include <algorithm>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <utility>

#include "pq_kernels.cuh"

namespace pq {

static inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct Carver {
  uint8_t* base;
  size_t off = 0;
  explicit Carver(void* b) : base(static_cast<uint8_t*>(b)) {}
  template <class T>
  T* take(size_t count) {
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += align_up(count * sizeof(T));
    return p;
  }
};

static inline int mtiles_of(const pq_desc* d) { return (d->T + kTileRows - 1) / kTileRows; }
static inline int experts_of(const pq_desc* d) { return d->r > 0 ? (d->E < 1 ? 1 : d->E) : 1; }
static inline int max_items_of(const pq_desc* d) { return mtiles_of(d) + experts_of(d) - 1; }
static inline bool routed(const pq_desc* d) { return d->r > 0 && d->E > 1; }
static inline bool normed(const pq_desc* d) { return (d->flags & PQ_FUSED_RMSNORM) != 0; }

// top_k = E with unit gates (a test mode of the training-size forward): every expert is active with weight one, which is
// a dense branch of width E r whose A is the experts' rows stacked and whose B is their columns side by side
static inline bool all_experts(const pq_desc* d) { return d->r > 0 && d->E > 1 && d->top_k == d->E; }
static inline pq_desc dense_equivalent(const pq_desc* d) {
  pq_desc e = *d;
  e.r = d->r * d->E; e.E = 1; e.top_k = 1; e.flags = d->flags & ~(uint32_t)PQ_UNIT_GATES;
  return e;
}

static int check_desc(const pq_desc* d, bool training) {
  if (!d) return PQ_ERR_NULL;
  if (d->size != sizeof(pq_desc)) return PQ_ERR_SHAPE;
  if (d->T < 1 || d->K < 32 || d->N < 32 || d->K % 32 || d->N % 32) return PQ_ERR_SHAPE;
  if (d->r < 0 || d->r % 8 || d->r > 256) return PQ_ERR_SHAPE;
  if (d->r > 0 && (d->E < 1 || d->E > kMaxExperts)) return PQ_ERR_SHAPE;
  if (d->r > 0 && d->top_k != 1) {
    // only k = 1 (the paper's setting) and, forward only and on the training-size path, k = E with unit gates
    if (!all_experts(d) || !(d->flags & PQ_UNIT_GATES) || !training || d->r * d->E > 128) return PQ_ERR_UNSUPPORTED;
  }
  if (training && d->r > 128) return PQ_ERR_UNSUPPORTED;
  return PQ_OK;
}

// saved buffer layout; base == nullptr only measures
static size_t carve_saved(const pq_desc* d, void* base, SavedPtrs* out) {
  Carver c(base);
  SavedPtrs s{};
  const size_t T = d->T, K = d->K;
  const int E = experts_of(d);
  s.max_items = max_items_of(d);
  s.q = c.take<int8_t>(T * K);
  s.xt = c.take<uint16_t>(T * K);
  s.xs = (routed(d) || normed(d)) ? c.take<uint16_t>(T * K) : nullptr;   // with a fused norm: the normalised activation
  s.gamma = c.take<float>(T);
  s.gate = c.take<float>(T);
  s.probs = routed(d) ? c.take<float>(T * E) : nullptr;
  s.expert = c.take<int>(T);
  s.perm = c.take<int>(T);
  s.pos = c.take<int>(T);
  s.offsets = c.take<int>(E + 1);
  s.h = d->r > 0 ? c.take<uint16_t>((size_t)2 * s.max_items * kTileRows * d->r) : nullptr;  // hi and lo planes
  s.rt.n_items = c.take<int>(1);
  s.rt.items = c.take<int4>(s.max_items);
  s.rt.tile_item_begin = c.take<int>(mtiles_of(d) + 1);
  s.rt.expert_item_begin = c.take<int>(E + 1);
  if (out) *out = s;
  return c.off;
}

static size_t carve_fwd_scratch(const pq_desc* d, void* base, FwdScratch* out) {
  Carver c(base);
  FwdScratch s{};
  const int E = experts_of(d);
  const size_t nblocks = (d->T + kRouterTokensPerBlock - 1) / kRouterTokensPerBlock;
  s.gate_tok = c.take<float>(d->T);
  s.probs_tok = c.take<float>((size_t)d->T * E);
  s.block_counts = c.take<int>(nblocks * E);
  s.block_base = c.take<int>(nblocks * E);
  s.rms = c.take<float>(d->T);
  if (out) *out = s;
  return c.off;
}

struct BwdScratch {
  uint16_t* dys;
  uint16_t* sb;
  uint16_t* ba;
  uint16_t* dhc;
  uint16_t* gh;
  float* dl;
  uint16_t* dlc;
  float* dbeta_partial;
  float* dalpha_partial;
  double* blk_sums;      // scalar feature scales: per-block fp64 sums of k_finalize_scales, [2 * ceil(N/128)]
  unsigned* arrivals;    // ... and its arrival counter
};

static size_t carve_bwd_scratch(const pq_desc* d, void* base, BwdScratch* out) {
  Carver c(base);
  BwdScratch s{};
  const size_t T = d->T, K = d->K, N = d->N, r = d->r;
  const int E = experts_of(d);
  const bool vec = d->flags & PQ_SCALE_VECTOR;
  s.dys = routed(d) ? c.take<uint16_t>(T * N) : nullptr;
  s.sb = c.take<uint16_t>(N * K);
  s.ba = (r > 0 && vec) ? c.take<uint16_t>((size_t)E * N * r) : nullptr;
  s.dhc = r > 0 ? c.take<uint16_t>((size_t)2 * max_items_of(d) * kTileRows * r) : nullptr;
  s.gh = r > 0 ? c.take<uint16_t>((size_t)2 * max_items_of(d) * kTileRows * r) : nullptr;
  s.dl = routed(d) ? c.take<float>(T * E) : nullptr;
  s.dlc = routed(d) ? c.take<uint16_t>(T * 16) : nullptr;
  s.dbeta_partial = c.take<float>(2 * ((K + 255) / 256) * N);   // two slots per 256-column tile of K
  s.dalpha_partial = r > 0 ? c.take<float>((size_t)2 * E * N) : nullptr;
  s.blk_sums = c.take<double>(2 * ((N + 127) / 128));
  s.arrivals = c.take<unsigned>(4);
  if (out) *out = s;
  return c.off;
}

static inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

// ---------------------------------------------------------------------------
// Helper stream: kernels of one call that do not depend on one another run side
// by side (forward of a dense layer with an HP branch: the activation quantisation
// next to the HP up-projection; backward: the weight-gradient GEMM next to the chain
// scaled sign matrix -> HP gradient GEMM -> dX, each filling the other's last wave).
// Every caller stream gets one non-blocking helper stream and three events, created
// on first use and kept; work forked to the helper is always joined back before the
// call's last kernel, so the caller sees plain stream order.  Event record and wait
// are legal under stream capture and become edges of the captured graph.
// ---------------------------------------------------------------------------
static int g_side_streams = 1;

struct SideCtx {
  cudaStream_t side = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, mid = nullptr;
};

static SideCtx* side_for(cudaStream_t st) {
  if (!g_side_streams) return nullptr;
  static std::mutex mu;
  static std::map<std::pair<int, cudaStream_t>, SideCtx> ctxs;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  SideCtx& c = ctxs[std::make_pair(dev, st)];
  if (!c.side) {
    // nothing is created while the caller's stream is being captured: such a call keeps plain stream order
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) {
      cudaGetLastError();
      return nullptr;
    }
    SideCtx n;
    if (cudaStreamCreateWithFlags(&n.side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&n.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&n.join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&n.mid, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;   // the caller falls back to plain stream order
    }
    c = n;
  }
  return &c;
}

// helper stream ordered after everything already in st
static bool side_fork(SideCtx* c, cudaStream_t st) {
  return cudaEventRecord(c->fork, st) == cudaSuccess && cudaStreamWaitEvent(c->side, c->fork, 0) == cudaSuccess;
}

// ---------------------------------------------------------------------------
// Allocation-free weight pack: the fp64 partial sums live in a fixed device array
// owned by the library instead of a caller-provided workspace.
// ---------------------------------------------------------------------------
constexpr int kStaticSlabElems = 16384;    // elements summed into one pair of partials
constexpr int kStaticMaxSlabs = 4096;      // 4096 x 2 doubles = 64 KiB
static __device__ __align__(256) double g_pack_scratch[2 * kStaticMaxSlabs];

// One block per slab of kStaticSlabElems consecutive elements: {sum, sum of |.|} in fp64,
// a fixed order inside the block, so the result does not depend on scheduling.
__global__ void __launch_bounds__(256) k_weight_slab_sums(const float4* __restrict__ W4, long long n4, double* __restrict__ partial) {
  pdl_launch_dependents();   // launched with programmatic stream serialisation: see launch_pdl
  pdl_wait();
  const long long base = (long long)blockIdx.x * (kStaticSlabElems / 4);
  double s = 0.0, a = 0.0;
  for (int i = threadIdx.x; i < kStaticSlabElems / 4; i += 256) {
    if (base + i < n4) {
      const float4 v = __ldg(W4 + base + i);
      s += (double)v.x + (double)v.y + (double)v.z + (double)v.w;
      a += (double)fabsf(v.x) + (double)fabsf(v.y) + (double)fabsf(v.z) + (double)fabsf(v.w);
    }
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
    partial[2 * blockIdx.x] = ts;      // every slot that k_binarize_pack reads is written here first:
    partial[2 * blockIdx.x + 1] = ta;  // nothing left over from an earlier call is ever used
  }
}

// In host code the name g_pack_scratch is only a handle for the device array, not a device
// address (handing it to a kernel would make the kernel touch the wrong memory).  The real
// address is asked for once per device, with that device current, and cached.
static int static_scratch_ptr(double** out) {
  constexpr int kMaxDevices = 64;
  static double* cache[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PQ_ERR_CUDA;
  if (!cache[dev]) {
    double* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_pack_scratch) != cudaSuccess || !ptr) return PQ_ERR_CUDA;
    cache[dev] = ptr;
  }
  *out = cache[dev];
  return PQ_OK;
}

static int pack_static(const float* W, int N, int K, uint32_t* bits, int8_t* s8, float* scales, cudaStream_t st) {
  const long long elems = (long long)N * K;
  const long long slabs = (elems + kStaticSlabElems - 1) / kStaticSlabElems;
  if (slabs > kStaticMaxSlabs) return PQ_ERR_TOO_LARGE;
  double* scratch = nullptr;
  int rc = static_scratch_ptr(&scratch);
  if (rc) return rc;
  const long long n4 = elems / 4;
  {
    LaunchScope ls(KID_PACK_SUMS, st);
    launch_pdl(k_weight_slab_sums, (int)slabs, 256, 0, st, reinterpret_cast<const float4*>(W), n4, scratch);
  }
  long long g = (n4 + 1023) / 1024;
  const int grid = (int)(g < 1 ? 1 : (g > 148 * 8 ? 148 * 8 : g));
  LaunchScope ls(KID_BINARIZE_PACK, st);
  launch_pdl(k_binarize_pack, grid, 256, 0, st, reinterpret_cast<const float4*>(W), n4, scratch, (int)slabs, 1.0 / (double)elems, bits,
                                        reinterpret_cast<uint32_t*>(s8), scales);
  return cudaGetLastError() == cudaSuccess ? PQ_OK : PQ_ERR_CUDA;
}

}  // namespace pq

using namespace pq;

extern "C" {

const char* pq_status_string(int s) {
  switch (s) {
    case PQ_OK: return "ok";
    case PQ_ERR_NULL: return "a required pointer is NULL";
    case PQ_ERR_SHAPE: return "a size violates the documented constraints";
    case PQ_ERR_ALIGN: return "a pointer is not 16-byte aligned";
    case PQ_ERR_WORKSPACE: return "workspace or saved buffer too small";
    case PQ_ERR_UNSUPPORTED: return "request not supported";
    case PQ_ERR_CUDA: return "a CUDA call failed";
    case PQ_ERR_TIMEOUT: return "a device-side bounded wait ran out";
    case PQ_ERR_TOO_LARGE: return "the problem needs more scratch than the library's fixed-size buffer holds";
    default: return "unknown status";
  }
}

size_t pq_saved_bytes(const pq_desc* d) {
  if (d && d->size == sizeof(pq_desc) && all_experts(d)) {
    if (check_desc(d, true) != PQ_OK) return 0;
    const pq_desc e = dense_equivalent(d);
    return carve_saved(&e, nullptr, nullptr);
  }
  if (check_desc(d, false) != PQ_OK) return 0;
  return carve_saved(d, nullptr, nullptr);
}

size_t pq_workspace_bytes(const pq_desc* d, int phase) {
  if (!d || d->size != sizeof(pq_desc)) return 0;
  switch (phase) {
    case PQ_PHASE_PACK: return align_up(sizeof(double) * 2 * kPackPartials);
    case PQ_PHASE_FWD:
      if (check_desc(d, true) != PQ_OK) return 0;
      if (all_experts(d)) {   // the dense equivalent's needs, then the experts' B side by side
        const pq_desc e = dense_equivalent(d);
        return carve_fwd_scratch(&e, nullptr, nullptr) + carve_saved(&e, nullptr, nullptr) + align_up((size_t)d->N * e.r * 2);
      }
      return carve_fwd_scratch(d, nullptr, nullptr) + carve_saved(d, nullptr, nullptr);
    case PQ_PHASE_BWD:
      if (check_desc(d, true) != PQ_OK || all_experts(d)) return 0;
      return carve_bwd_scratch(d, nullptr, nullptr);
    case PQ_PHASE_DECODE:
      if (check_desc(d, false) != PQ_OK || d->T > 16) return 0;
      return decode_workspace_bytes(d->T, d->K, d->N, d->r, (d->flags & PQ_DECODE_DUMP_ACC) != 0) +
             decode_stream_extra_bytes(d->T, d->K, d->N, d->r, (d->flags & PQ_DECODE_DUMP_ACC) != 0);
    default: return 0;
  }
}

int pq_saved_view_init(const pq_desc* d, void* saved, pq_saved_view* out) {
  if (!d || !saved || !out) return PQ_ERR_NULL;
  int rc = check_desc(d, false);
  if (rc) return rc;
  SavedPtrs s;
  carve_saved(d, saved, &s);
  out->q = s.q; out->xt = s.xt; out->xs = s.xs; out->gamma = s.gamma; out->gate = s.gate; out->probs = s.probs;
  out->expert = s.expert; out->perm = s.perm; out->pos = s.pos; out->offsets = s.offsets; out->h = s.h;
  out->n_items = s.rt.n_items; out->items = reinterpret_cast<int32_t*>(s.rt.items);
  out->tile_item_begin = s.rt.tile_item_begin; out->expert_item_begin = s.rt.expert_item_begin;
  out->max_items = s.max_items;
  return PQ_OK;
}

int pq_bwd_view_init(const pq_desc* d, void* ws, pq_bwd_view* out) {
  if (!d || !ws || !out) return PQ_ERR_NULL;
  int rc = check_desc(d, true);
  if (rc) return rc;
  BwdScratch s;
  carve_bwd_scratch(d, ws, &s);
  out->dl = s.dl;
  return PQ_OK;
}

int pq_decode_view_init(const pq_desc* d, void* ws, pq_decode_view* out) {
  if (!d || !ws || !out) return PQ_ERR_NULL;
  int rc = check_desc(d, false);
  if (rc) return rc;
  if (d->T > 16) return PQ_ERR_SHAPE;
  const DecodeViewPtrs v = decode_view(d->T, d->K, d->N, d->r, ws, (d->flags & PQ_DECODE_DUMP_ACC) != 0);
  out->tokens = static_cast<pq_decode_token*>(v.tokens);
  out->acc = v.acc;
  decode_stream_view(d->T, d->K, d->N, d->r, ws, (d->flags & PQ_DECODE_DUMP_ACC) != 0, &out->hp_h_int, &out->hp_z_int);
  return PQ_OK;
}

int pq_pack_weights(const pq_desc* d, const float* W, uint32_t* w_bits, int8_t* w_s8, float* w_scales, void* ws, size_t ws_bytes,
                    void* stream) {
  if (!d || !W || !w_bits || !w_scales || !ws) return PQ_ERR_NULL;
  if (d->size != sizeof(pq_desc) || d->N < 1 || d->K < 32 || d->K % 32) return PQ_ERR_SHAPE;
  if (misaligned(W) || misaligned(w_bits) || misaligned(w_s8) || misaligned(ws)) return PQ_ERR_ALIGN;
  if (ws_bytes < pq_workspace_bytes(d, PQ_PHASE_PACK)) return PQ_ERR_WORKSPACE;
  cudaError_t e = launch_pack(W, d->N, d->K, w_bits, w_s8, w_scales, static_cast<double*>(ws), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? PQ_OK : PQ_ERR_CUDA;
}

int pq_pack_experts(const pq_desc* d, const uint16_t* A, const uint16_t* B, int8_t* A8, int8_t* B8, float* hp_scales, void* ws,
                    size_t ws_bytes, void* stream) {
  if (!d || !A || !B || !A8 || !B8 || !hp_scales || !ws) return PQ_ERR_NULL;
  int rc = check_desc(d, false);
  if (rc) return rc;
  if (d->r <= 0) return PQ_ERR_SHAPE;
  if (misaligned(A) || misaligned(B) || misaligned(A8) || misaligned(B8) || misaligned(ws)) return PQ_ERR_ALIGN;
  if (ws_bytes < pq_workspace_bytes(d, PQ_PHASE_PACK)) return PQ_ERR_WORKSPACE;
  cudaError_t e = launch_pack_experts(A, B, experts_of(d), d->r, d->K, d->N, A8, B8, hp_scales, static_cast<uint32_t*>(ws),
                                      static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? PQ_OK : PQ_ERR_CUDA;
}

int pq_pack_weights_static(const pq_desc* d, const float* W, uint32_t* w_bits, int8_t* w_s8, float* w_scales, void* stream) {
  if (!d || !W || !w_bits || !w_scales) return PQ_ERR_NULL;
  if (d->size != sizeof(pq_desc) || d->N < 1 || d->K < 32 || d->K % 32) return PQ_ERR_SHAPE;
  if (misaligned(W) || misaligned(w_bits) || misaligned(w_s8)) return PQ_ERR_ALIGN;
  return pack_static(W, d->N, d->K, w_bits, w_s8, w_scales, static_cast<cudaStream_t>(stream));
}

static int check_decode_item(const pq_desc* d, const uint16_t* X, const uint32_t* w_bits, const float* w_scales, const uint16_t* A,
                             const uint16_t* B, const uint16_t* Wr, const float* alpha, const float* beta, const uint16_t* Y, const void* ws,
                             size_t ws_bytes) {
  if (!d || !X || !w_scales || !beta || !Y || !w_bits || !ws) return PQ_ERR_NULL;
  int rc = check_desc(d, false);
  if (rc) return rc;
  if (d->T > 16) return PQ_ERR_SHAPE;
  if (d->r > 0 && (!A || !B || !alpha)) return PQ_ERR_NULL;
  if (routed(d) && !Wr) return PQ_ERR_NULL;
  if (misaligned(X) || misaligned(w_bits) || misaligned(A) || misaligned(B) || misaligned(Wr) || misaligned(ws)) return PQ_ERR_ALIGN;
  if (ws_bytes < decode_workspace_bytes(d->T, d->K, d->N, d->r, (d->flags & PQ_DECODE_DUMP_ACC) != 0)) return PQ_ERR_WORKSPACE;
  return PQ_OK;
}

// hp_scales != nullptr: INT8 HP branch, A and B are int8 codes (training path only)
static int forward_impl(const pq_desc* d, const uint16_t* X, const uint32_t* w_bits, const int8_t* w_s8, const float* w_scales,
                        const uint16_t* A, const uint16_t* B, const float* hp_scales, const uint16_t* Wr, const float* alpha, const float* beta,
                        uint16_t* Y, void* saved, size_t saved_bytes, void* ws, size_t ws_bytes, void* stream, bool hp_ext = false,
                        const uint16_t* norm_weight = nullptr, float norm_eps = 0.f) {
  if (!d || !X || !w_scales || !beta || !Y) return PQ_ERR_NULL;
  if (!w_s8) {
    if (hp_scales) return PQ_ERR_UNSUPPORTED;
    // decode: a few tokens straight from the packed sign bits
    int rc = check_decode_item(d, X, w_bits, w_scales, A, B, Wr, alpha, beta, Y, ws, ws_bytes);
    if (rc) return rc;
    const bool dump = (d->flags & PQ_DECODE_DUMP_ACC) != 0;
    LayerArgs a{d->T, d->K, d->N, d->r, experts_of(d), (d->flags & PQ_SCALE_VECTOR) ? 1 : 0, w_scales, alpha, beta, A, B, Wr};
    return decode_forward(a, X, w_bits, Y, ws, dump, static_cast<cudaStream_t>(stream));
  }
  int rc = check_desc(d, true);
  if (rc) return rc;
  (void)w_bits;
  if (all_experts(d)) {
    if (hp_scales || norm_weight || normed(d)) return PQ_ERR_UNSUPPORTED;
    if (!A || !B || !alpha || !ws) return PQ_ERR_NULL;
    if (misaligned(B) || misaligned(ws)) return PQ_ERR_ALIGN;
    const pq_desc e = dense_equivalent(d);
    const size_t side = align_up((size_t)d->N * e.r * 2);
    if (ws_bytes < side) return PQ_ERR_WORKSPACE;
    uint16_t* b_wide = reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(ws) + (ws_bytes - side) / 256 * 256);
    if (launch_concat_experts(B, d->E, d->N, d->r, b_wide, static_cast<cudaStream_t>(stream)) != cudaSuccess) return PQ_ERR_CUDA;
    return forward_impl(&e, X, w_bits, w_s8, w_scales, A, b_wide, nullptr, nullptr, alpha, beta, Y, saved, saved_bytes, ws,
                        (ws_bytes - side) / 256 * 256, stream);
  }
  if (normed(d) != (norm_weight != nullptr)) return PQ_ERR_NULL;           // the flag sizes the saved buffer
  if (norm_weight && (!(norm_eps > 0.f) || misaligned(norm_weight))) return norm_eps > 0.f ? PQ_ERR_ALIGN : PQ_ERR_SHAPE;
  if (d->r > 0 && (!A || !B || !alpha)) return PQ_ERR_NULL;
  if (routed(d) && !Wr) return PQ_ERR_NULL;
  if (!ws) return PQ_ERR_NULL;
  if (misaligned(X) || misaligned(w_s8) || misaligned(A) || misaligned(B) || misaligned(Wr) || misaligned(Y) || misaligned(saved) ||
      misaligned(ws))
    return PQ_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FwdScratch sc;
  size_t used = carve_fwd_scratch(d, ws, &sc);
  SavedPtrs sv;
  if (saved) {
    if (saved_bytes < carve_saved(d, nullptr, nullptr)) return PQ_ERR_WORKSPACE;
    carve_saved(d, saved, &sv);
  } else {
    used += carve_saved(d, static_cast<uint8_t*>(ws) + used, &sv);
  }
  if (ws_bytes < used) return PQ_ERR_WORKSPACE;
  const int E = experts_of(d);
  LayerArgs a{d->T, d->K, d->N, d->r, E, (d->flags & PQ_SCALE_VECTOR) ? 1 : 0, w_scales, alpha, beta, A, B, Wr};
  if (hp_scales) {
    if (d->r <= 0 || d->r % 16) return PQ_ERR_SHAPE;       // int8 rows of r bytes must be 16-byte multiples for TMA
    a.hp_scales = hp_scales;
    a.hp_ext = hp_ext;
  }
  // dense layer with a bf16 HP branch: the quantisation runs on the helper stream next to scan -> up-projection
  // (the INT8 branch multiplies the codes themselves, so its up-projection follows the quantisation)
  // (with a fused norm the up-projection reads the normalised copy the quantiser writes, so it follows it)
  SideCtx* side = (d->r > 0 && !routed(d) && !hp_scales && !norm_weight) ? side_for(st) : nullptr;
  if (side && !side_fork(side, st)) return PQ_ERR_CUDA;
  if (launch_route_and_quant(X, Wr, d->T, d->K, routed(d) ? E : 1, sv, sc, st, side ? side->side : st, norm_weight, norm_eps) != cudaSuccess)
    return PQ_ERR_CUDA;
  if (side && cudaEventRecord(side->join, side->side) != cudaSuccess) return PQ_ERR_CUDA;
  const uint16_t* xs = (routed(d) || norm_weight) ? sv.xs : X;
  return gemm_forward(a, w_s8, sv, xs, Y, st, side ? side->join : nullptr);
}

int pq_linear_forward(const pq_desc* d, const uint16_t* X, const uint32_t* w_bits, const int8_t* w_s8, const float* w_scales,
                      const uint16_t* A, const uint16_t* B, const uint16_t* Wr, const float* alpha, const float* beta, uint16_t* Y,
                      void* saved, size_t saved_bytes, void* ws, size_t ws_bytes, void* stream) {
  return forward_impl(d, X, w_bits, w_s8, w_scales, A, B, nullptr, Wr, alpha, beta, Y, saved, saved_bytes, ws, ws_bytes, stream);
}

int pq_linear_forward_rms(const pq_desc* d, const uint16_t* X, const uint16_t* norm_weight, float norm_eps, const int8_t* w_s8,
                          const float* w_scales, const uint16_t* A, const uint16_t* B, const uint16_t* Wr, const float* alpha, const float* beta,
                          uint16_t* Y, void* saved, size_t saved_bytes, void* ws, size_t ws_bytes, void* stream) {
  if (!w_s8 || !norm_weight) return PQ_ERR_NULL;
  return forward_impl(d, X, nullptr, w_s8, w_scales, A, B, nullptr, Wr, alpha, beta, Y, saved, saved_bytes, ws, ws_bytes, stream, false,
                      norm_weight, norm_eps);
}

int pq_linear_forward_hp8(const pq_desc* d, const uint16_t* X, const int8_t* w_s8, const float* w_scales, const int8_t* A8, const int8_t* B8,
                          const float* hp_scales, const uint16_t* Wr, const float* alpha, const float* beta, uint16_t* Y, void* saved,
                          size_t saved_bytes, void* ws, size_t ws_bytes, void* stream) {
  if (!w_s8 || !A8 || !B8 || !hp_scales) return PQ_ERR_NULL;
  return forward_impl(d, X, nullptr, w_s8, w_scales, reinterpret_cast<const uint16_t*>(A8), reinterpret_cast<const uint16_t*>(B8), hp_scales, Wr,
                      alpha, beta, Y, saved, saved_bytes, ws, ws_bytes, stream);
}

// ---------------------------------------------------------------------------
// FFN-level decoupling (Eq. 11): Y = alpha FFN_INT8[:r](x) + beta FFN_INT1[r:](x), composed of the entry points above.
// ---------------------------------------------------------------------------
static __device__ float g_unit_scale = 1.0f;   // beta of the 1-bit FFN's inner linears

struct FfnCarve {
  void* saved_x; size_t saved_x_bytes;
  void* saved_d; size_t saved_d_bytes;
  void* ws_fwd; size_t ws_fwd_bytes;
  uint16_t *G1, *U1, *M1;
  int *g_int, *u_int;
  size_t total;
};

static pq_desc ffn_linear_desc(const pq_ffn_desc* d, int K, int N, int r) {
  pq_desc x{};
  x.size = sizeof(pq_desc); x.flags = 0; x.T = d->T; x.K = K; x.N = N; x.r = r; x.E = r > 0 ? 1 : 0; x.top_k = 1;
  return x;
}

static int check_ffn_desc(const pq_ffn_desc* d) {
  if (!d) return PQ_ERR_NULL;
  if (d->size != sizeof(pq_ffn_desc)) return PQ_ERR_SHAPE;
  if (d->T < 1 || d->D < 32 || d->D % 32 || d->F1 < 32 || d->F1 % 32) return PQ_ERR_SHAPE;
  if (d->r < 16 || d->r % 16 || d->r > 128) return PQ_ERR_SHAPE;
  return PQ_OK;
}

static void carve_ffn(const pq_ffn_desc* d, void* base, FfnCarve* o) {
  Carver c(base);
  const pq_desc dx = ffn_linear_desc(d, d->D, d->F1, 0), dd = ffn_linear_desc(d, d->F1, d->D, d->r);
  o->saved_x_bytes = carve_saved(&dx, nullptr, nullptr);
  o->saved_d_bytes = carve_saved(&dd, nullptr, nullptr);
  o->ws_fwd_bytes = std::max(carve_fwd_scratch(&dx, nullptr, nullptr), carve_fwd_scratch(&dd, nullptr, nullptr));
  o->saved_x = c.take<uint8_t>(o->saved_x_bytes);
  o->saved_d = c.take<uint8_t>(o->saved_d_bytes);
  o->ws_fwd = c.take<uint8_t>(o->ws_fwd_bytes);
  const size_t tf = (size_t)d->T * d->F1, rows = (size_t)mtiles_of(&dx) * kTileRows;
  o->G1 = c.take<uint16_t>(tf); o->U1 = c.take<uint16_t>(tf); o->M1 = c.take<uint16_t>(tf);
  o->g_int = c.take<int>(rows * d->r); o->u_int = c.take<int>(rows * d->r);
  o->total = c.off;
}

static int unit_scale_ptr(const float** out) {
  constexpr int kMaxDevices = 64;
  static const float* cache[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PQ_ERR_CUDA;
  if (!cache[dev]) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_unit_scale) != cudaSuccess || !ptr) return PQ_ERR_CUDA;
    cache[dev] = ptr;
  }
  *out = cache[dev];
  return PQ_OK;
}

size_t pq_ffn_workspace_bytes(const pq_ffn_desc* d) {
  if (check_ffn_desc(d) != PQ_OK) return 0;
  FfnCarve c;
  carve_ffn(d, nullptr, &c);
  return c.total;
}

int pq_ffn_view_init(const pq_ffn_desc* d, void* ws, pq_ffn_view* out) {
  if (!d || !ws || !out) return PQ_ERR_NULL;
  int rc = check_ffn_desc(d);
  if (rc) return rc;
  FfnCarve c;
  carve_ffn(d, ws, &c);
  const pq_desc dx = ffn_linear_desc(d, d->D, d->F1, 0), dd = ffn_linear_desc(d, d->F1, d->D, d->r);
  SavedPtrs sx, sd;
  carve_saved(&dx, c.saved_x, &sx);
  carve_saved(&dd, c.saved_d, &sd);
  out->G1 = c.G1; out->U1 = c.U1; out->M1 = c.M1; out->g_int = c.g_int; out->u_int = c.u_int;
  out->qm = reinterpret_cast<int8_t*>(sd.h);
  out->gamma_m = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(sd.h) + align_up((size_t)sd.max_items * kTileRows * d->r));
  out->q_m1 = sd.q; out->gamma_m1 = sd.gamma;
  return PQ_OK;
}

int pq_ffn_forward(const pq_ffn_desc* d, const uint16_t* X, const int8_t* g_s8, const float* g_scales, const int8_t* u_s8,
                   const float* u_scales, const int8_t* d_s8, const float* d_scales, const int8_t* G8, const int8_t* U8, const int8_t* D8,
                   const float* hp_scales, const float* alpha, const float* beta, uint16_t* Y, void* ws, size_t ws_bytes, void* stream) {
  if (!X || !g_s8 || !g_scales || !u_s8 || !u_scales || !d_s8 || !d_scales || !G8 || !U8 || !D8 || !hp_scales || !alpha || !beta || !Y || !ws)
    return PQ_ERR_NULL;
  int rc = check_ffn_desc(d);
  if (rc) return rc;
  if (misaligned(X) || misaligned(g_s8) || misaligned(u_s8) || misaligned(d_s8) || misaligned(G8) || misaligned(U8) || misaligned(D8) ||
      misaligned(Y) || misaligned(ws))
    return PQ_ERR_ALIGN;
  FfnCarve c;
  carve_ffn(d, ws, &c);
  if (ws_bytes < c.total) return PQ_ERR_WORKSPACE;
  const float* one = nullptr;
  rc = unit_scale_ptr(&one);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const pq_desc dx = ffn_linear_desc(d, d->D, d->F1, 0), dd = ffn_linear_desc(d, d->F1, d->D, d->r);
  // 1-bit FFN, gate projection: also leaves the int8 codes of x and the tile table in saved_x
  rc = forward_impl(&dx, X, nullptr, g_s8, g_scales, nullptr, nullptr, nullptr, nullptr, nullptr, one, c.G1, c.saved_x, c.saved_x_bytes,
                    c.ws_fwd, c.ws_fwd_bytes, stream);
  if (rc) return rc;
  // INT8 FFN: exact sums of its gate and up projections on those codes, then its hidden activation as codes, written
  // where the fused down projection expects the codes of h
  SavedPtrs sx, sd;
  carve_saved(&dx, c.saved_x, &sx);
  carve_saved(&dd, c.saved_d, &sd);
  LayerArgs a8{d->T, d->D, d->D, d->r, 1, 0, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  rc = gemm_hp_up8(a8, sx, G8, c.g_int, st);
  if (rc) return rc;
  rc = gemm_hp_up8(a8, sx, U8, c.u_int, st);
  if (rc) return rc;
  int8_t* qm = reinterpret_cast<int8_t*>(sd.h);
  float* gamma_m = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(sd.h) + align_up((size_t)sd.max_items * kTileRows * d->r));
  if (launch_ffn8_act(c.g_int, c.u_int, sx.gamma, hp_scales, d->T, d->r, qm, gamma_m, st) != cudaSuccess) return PQ_ERR_CUDA;
  // 1-bit FFN, up projection and gate
  rc = forward_impl(&dx, X, nullptr, u_s8, u_scales, nullptr, nullptr, nullptr, nullptr, nullptr, one, c.U1, c.saved_x, c.saved_x_bytes,
                    c.ws_fwd, c.ws_fwd_bytes, stream);
  if (rc) return rc;
  if (launch_swiglu(c.G1, c.U1, c.M1, (long long)d->T * d->F1, st) != cudaSuccess) return PQ_ERR_CUDA;
  // down projections of both FFNs in one fused tile: beta (lam / gamma) (q(M1) . S_d) + alpha (D8 qm) / (gamma_D gamma_m)
  return forward_impl(&dd, c.M1, nullptr, d_s8, d_scales, reinterpret_cast<const uint16_t*>(D8), reinterpret_cast<const uint16_t*>(D8),
                      hp_scales + 1, nullptr, alpha, beta, Y, c.saved_d, c.saved_d_bytes, c.ws_fwd, c.ws_fwd_bytes, stream, true);
}

int pq_decode_pack_bytes(const pq_desc* d, size_t* bits_il_bytes, size_t* b_il_bytes) {
  if (!d || !bits_il_bytes || !b_il_bytes) return PQ_ERR_NULL;
  int rc = check_desc(d, false);
  if (rc) return rc;
  if (d->r % 8) return PQ_ERR_SHAPE;
  decode_pack_sizes(d->K, d->N, d->r, experts_of(d), bits_il_bytes, b_il_bytes);
  return PQ_OK;
}

int pq_pack_decode(const pq_desc* d, const uint32_t* w_bits, const uint16_t* B, uint32_t* w_bits_il, uint16_t* B_il, void* stream) {
  if (!d || !w_bits || !w_bits_il) return PQ_ERR_NULL;
  int rc = check_desc(d, false);
  if (rc) return rc;
  if (d->r % 8) return PQ_ERR_SHAPE;
  if (d->r > 0 && (!B || !B_il)) return PQ_ERR_NULL;
  if (misaligned(w_bits) || misaligned(B) || misaligned(w_bits_il) || misaligned(B_il)) return PQ_ERR_ALIGN;
  return decode_pack(d->K, d->N, d->r, experts_of(d), w_bits, B, w_bits_il, B_il, static_cast<cudaStream_t>(stream));
}

int pq_pack_decode_hp8(const pq_desc* d, const int8_t* B8, int8_t* B8_il, size_t b8_il_bytes, void* stream) {
  if (!d || !B8 || !B8_il) return PQ_ERR_NULL;
  int rc = check_desc(d, false);
  if (rc) return rc;
  if (d->r <= 0 || d->r % 16) return PQ_ERR_SHAPE;
  if (misaligned(B8) || misaligned(B8_il)) return PQ_ERR_ALIGN;
  if (b8_il_bytes < decode_pack_b8_bytes(d->N, d->r, experts_of(d))) return PQ_ERR_WORKSPACE;
  return decode_pack_b8(d->N, d->r, experts_of(d), B8, B8_il, static_cast<cudaStream_t>(stream));
}

size_t pq_decode_pack_hp8_bytes(const pq_desc* d) {
  if (check_desc(d, false) != PQ_OK || d->r <= 0 || d->r % 16) return 0;
  return decode_pack_b8_bytes(d->N, d->r, experts_of(d));
}

int pq_decode_batch(const pq_decode_item* items, int n, void* stream) {
  if (!items) return PQ_ERR_NULL;
  if (n < 1 || n > 4096) return PQ_ERR_SHAPE;
  DecodeItemArgs* args = new (std::nothrow) DecodeItemArgs[n];
  if (!args) return PQ_ERR_CUDA;
  int rc = PQ_OK;
  for (int i = 0; i < n && rc == PQ_OK; ++i) {
    const pq_decode_item& it = items[i];
    const bool hp8 = it.A8 != nullptr;
    // the INT8 branch brings its own expert matrices: the bf16 ones are not read
    rc = check_decode_item(&it.desc, it.X, it.w_bits, it.w_scales, hp8 ? reinterpret_cast<const uint16_t*>(it.A8) : it.A,
                           hp8 ? reinterpret_cast<const uint16_t*>(it.B8_il) : it.B, it.Wr, it.alpha, it.beta, it.Y, it.ws, it.ws_bytes);
    if (rc) break;
    if (hp8 && (!it.w_bits_il || !it.B8_il || !it.hp_scales)) { rc = PQ_ERR_NULL; break; }
    if (hp8 && (it.desc.r <= 0 || it.desc.r % 16)) { rc = PQ_ERR_SHAPE; break; }
    if (hp8 && (misaligned(it.A8) || misaligned(it.B8_il))) { rc = PQ_ERR_ALIGN; break; }
    const pq_desc* d = &it.desc;
    args[i].a = LayerArgs{d->T, d->K, d->N, d->r, experts_of(d), (d->flags & PQ_SCALE_VECTOR) ? 1 : 0, it.w_scales, it.alpha, it.beta, it.A, it.B, it.Wr};
    args[i].X = it.X; args[i].bits = it.w_bits; args[i].Y = it.Y; args[i].ws = it.ws;
    args[i].dump = (d->flags & PQ_DECODE_DUMP_ACC) != 0;
    if (misaligned(it.norm_weight)) { rc = PQ_ERR_ALIGN; break; }
    if (it.norm_weight && !(it.norm_eps > 0.f)) { rc = PQ_ERR_SHAPE; break; }   // an all-zero token needs it
    args[i].norm_weight = it.norm_weight; args[i].norm_eps = it.norm_eps;
    if (it.w_bits_il) {
      if (misaligned(it.w_bits_il) || misaligned(it.B_il)) { rc = PQ_ERR_ALIGN; break; }
      if (d->r > 0 && !it.B_il && !hp8) { rc = PQ_ERR_NULL; break; }
      if (it.ws_bytes < pq_workspace_bytes(d, PQ_PHASE_DECODE)) { rc = PQ_ERR_WORKSPACE; break; }
      args[i].bits_il = it.w_bits_il;
      args[i].B_il = hp8 ? reinterpret_cast<const uint16_t*>(it.B8_il) : it.B_il;
      args[i].A8 = it.A8; args[i].hp_scales = it.hp_scales;
    }
  }
  if (rc == PQ_OK) rc = decode_batch(args, n, static_cast<cudaStream_t>(stream));
  delete[] args;
  return rc;
}

int pq_linear_backward(const pq_desc* d, const uint16_t* dY, const uint16_t* X, const int8_t* w_s8, const float* w_scales,
                       const uint16_t* A, const uint16_t* B, const uint16_t* Wr, const float* alpha, const float* beta,
                       const void* saved, size_t saved_bytes, uint16_t* dX, float* dW, float* dA, float* dB, float* dWr, float* dalpha,
                       float* dbeta, void* ws, size_t ws_bytes, void* stream) {
  if (!d || !dY || !X || !w_s8 || !w_scales || !beta || !saved || !dX || !dW || !dbeta || !ws) return PQ_ERR_NULL;
  if (d->size == sizeof(pq_desc) && all_experts(d)) return PQ_ERR_UNSUPPORTED;   // the all-experts mode is forward only
  int rc = check_desc(d, true);
  if (rc) return rc;
  const bool hp = d->r > 0;
  if (hp && (!A || !B || !alpha || !dA || !dB || !dalpha)) return PQ_ERR_NULL;
  if (routed(d) && (!Wr || !dWr)) return PQ_ERR_NULL;
  if (misaligned(dY) || misaligned(X) || misaligned(w_s8) || misaligned(A) || misaligned(B) || misaligned(Wr) || misaligned(saved) ||
      misaligned(dX) || misaligned(dW) || misaligned(dA) || misaligned(dB) || misaligned(dWr) || misaligned(ws))
    return PQ_ERR_ALIGN;
  if (saved_bytes < carve_saved(d, nullptr, nullptr)) return PQ_ERR_WORKSPACE;
  if (ws_bytes < carve_bwd_scratch(d, nullptr, nullptr)) return PQ_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SavedPtrs sv;
  carve_saved(d, const_cast<void*>(saved), &sv);
  BwdScratch sc;
  carve_bwd_scratch(d, ws, &sc);
  const int E = experts_of(d);
  const int vec = (d->flags & PQ_SCALE_VECTOR) ? 1 : 0;
  LayerArgs a{d->T, d->K, d->N, d->r, E, vec, w_scales, alpha, beta, A, B, Wr};

  BwdBuffers b{};
  if (routed(d)) {
    if (launch_scatter_rows(dY, sc.dys, sv.pos, d->T, d->N, st) != cudaSuccess) return PQ_ERR_CUDA;
    b.dys = sc.dys;
    b.xs = sv.xs;
  } else {
    b.dys = dY;
    b.xs = normed(d) ? sv.xs : X;      // the layer's input is the normalised activation the forward left in `saved`
  }
  // With the helper stream: what leads to dX (scaled sign matrix, scaled B, HP gradient GEMM, dX) runs there, the
  // weight gradient on the caller's stream beside it; see BwdStreams.
  SideCtx* side = side_for(st);
  if (side && !side_fork(side, st)) return PQ_ERR_CUDA;
  cudaStream_t sx = side ? side->side : st;
  if (launch_scaled_sign(w_s8, sc.sb, beta, vec, d->N, d->K, sc.arrivals, sx) != cudaSuccess) return PQ_ERR_CUDA;
  b.sb = sc.sb;
  if (hp && vec) {
    if (launch_scaled_b(B, sc.ba, alpha, E, d->N, d->r, sx) != cudaSuccess) return PQ_ERR_CUDA;
    b.ba = sc.ba;
  } else {
    b.ba = B;
  }
  b.dhc = sc.dhc; b.gh = sc.gh; b.dl = sc.dl; b.dlc = sc.dlc;
  b.dbeta_partial = sc.dbeta_partial; b.dalpha_partial = sc.dalpha_partial;
  BwdStreams bs;
  if (side) { bs.side = side->side; bs.dh_done = side->mid; bs.side_done = side->join; }
  rc = gemm_backward(a, w_s8, sv, b, dX, dW, dA, dB, dWr, st, bs);
  if (rc) return rc;

  // dbeta_n = lam * sum over the column tiles of the partial sign-weighted row sums, dalpha_n = sum over experts
  // of the dB-weighted row sums; the scalar form sums over n as well
  if (dalpha && !hp && cudaMemsetAsync(dalpha, 0, sizeof(float) * (vec ? d->N : 1), st) != cudaSuccess) return PQ_ERR_CUDA;
  if (launch_finalize_scales(sc.dbeta_partial, 2 * ((d->K + 255) / 256), hp ? sc.dalpha_partial : nullptr, 2 * E, d->N, w_scales, vec, dbeta,
                             hp ? dalpha : nullptr, sc.blk_sums, sc.arrivals, st) != cudaSuccess)
    return PQ_ERR_CUDA;
  return PQ_OK;
}

int pq_debug_gemm(int mode, int M, int N, int K, const void* A, const void* B, void* D, void* stream) {
  if (!A || !B || !D) return PQ_ERR_NULL;
  if (M < 1 || N < 1 || K < 1 || M % 8 || N % 8 || K % (mode == 0 ? 16 : 8)) return PQ_ERR_SHAPE;
  if (misaligned(A) || misaligned(B) || misaligned(D)) return PQ_ERR_ALIGN;
  return gemm_debug(mode, M, N, K, A, B, D, 256, static_cast<cudaStream_t>(stream));
}

int pq_debug_gemm_tile(int mode, int M, int N, int K, const void* A, const void* B, void* D, int tile_n, void* stream) {
  if (!A || !B || !D) return PQ_ERR_NULL;
  if (M < 1 || N < 1 || K < 1 || M % 8 || N % 8 || K % (mode == 0 ? 16 : 8)) return PQ_ERR_SHAPE;
  if (misaligned(A) || misaligned(B) || misaligned(D)) return PQ_ERR_ALIGN;
  return gemm_debug(mode, M, N, K, A, B, D, tile_n, static_cast<cudaStream_t>(stream));
}

int pq_set_option(int option, int value) {
  switch (option) {
    case PQ_OPT_DECODE_PDL: decode_set_pdl(value); return PQ_OK;
    case PQ_OPT_SIDE_STREAM: g_side_streams = value ? 1 : 0; return PQ_OK;
    case PQ_OPT_DECODE_STREAM: decode_stream_enable(value); return PQ_OK;
    case PQ_OPT_DECODE_PREFETCH: decode_stream_prefetch(value); return PQ_OK;
    case PQ_OPT_DECODE_MMA_FROM: decode_stream_mma_from(value); return PQ_OK;
    case PQ_OPT_DECODE_INTERLEAVE: decode_stream_interleave(value); return PQ_OK;
    case PQ_OPT_SPIN_CYCLES: {
      // the limit lives in constant memory of the current device; the copy is ordered after everything
      // already enqueued there (a blocking copy), so no running kernel sees it change
      const long long cycles = value > 0 ? (long long)value : kDefaultSpinCycles;
      return cudaMemcpyToSymbol(c_spin_cycles, &cycles, sizeof(cycles)) == cudaSuccess ? PQ_OK : PQ_ERR_CUDA;
    }
    default: return PQ_ERR_UNSUPPORTED;
  }
}

long long pq_kernel_launches(void) { return g_launches; }

int pq_profile_events(int kernel_id, void* start_event, void* stop_event) {
  if (kernel_id < 0 || kernel_id >= KID_COUNT) return PQ_ERR_SHAPE;
  g_profile[kernel_id].start = static_cast<cudaEvent_t>(start_event);
  g_profile[kernel_id].stop = static_cast<cudaEvent_t>(stop_event);
  return PQ_OK;
}

int pq_device_status(void* stream, int* code, int* where) {
  if (!code || !where) return PQ_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return PQ_ERR_CUDA;
  int host[2] = {0, 0};
  if (cudaMemcpyFromSymbol(host, g_status, sizeof(host)) != cudaSuccess) return PQ_ERR_CUDA;
  *code = host[0];
  *where = host[1];
  if (host[0] != 0) {
    const int zero[2] = {0, 0};
    if (cudaMemcpyToSymbol(g_status, zero, sizeof(zero)) != cudaSuccess) return PQ_ERR_CUDA;
    // a kernel that gave up may have left the decode kernel's grid barrier half counted
    if (cudaDeviceSynchronize() != cudaSuccess) return PQ_ERR_CUDA;
    decode_stream_reset();
  }
  return PQ_OK;
}

}  // extern "C"
