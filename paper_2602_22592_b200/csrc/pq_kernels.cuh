// Internal declarations shared by the kernel translation units and the C ABI.
#pragma once
#include <cuda.h>

#include "pq_common.cuh"

namespace pq {

constexpr int kMaxExperts = 16;
constexpr int kRouterTokensPerBlock = 32;  // must equal the warp width (rank-in-block ballot)
constexpr int kTileRows = 128;             // rows of one tensor-core tile
constexpr int kPackPartials = 1024;        // fp64 partial sums of the weight reduction
constexpr float kActQmax = 128.0f;         // 2^7 of Eq. 9
constexpr float kActAmaxFloor = 1e-5f;     // all-zero row guard

// Kernel ids for launch counting and optional event timing (pq_profile_events).
enum KernelId : int {
  KID_PACK_SUMS = 0, KID_BINARIZE_PACK, KID_ROUTER, KID_ROUTE_SCAN, KID_ACT_QUANT, KID_HP_UP, KID_FWD, KID_SCATTER_ROWS,
  KID_SCALED_SIGN, KID_SCALED_B, KID_HP_DH, KID_BWD_DX, KID_BWD_DW, KID_HP_DB, KID_HP_DA, KID_ROUTER_WGRAD, KID_SUM_PARTIALS,
  KID_SUM_SCALAR, KID_DEBUG, KID_DECODE_PREP, KID_DECODE_MAIN, KID_REDUCE_DB, KID_REDUCE_DA, KID_DECODE_PACK, KID_DECODE_STREAM, KID_COUNT
};
struct ProfileSlot { cudaEvent_t start, stop; };
extern ProfileSlot g_profile[KID_COUNT];
extern long long g_launches;
// Brackets one kernel launch: counts it and, if events were registered for its id, records them.
struct LaunchScope {
  int id; cudaStream_t st;
  LaunchScope(int id_, cudaStream_t st_) : id(id_), st(st_) {
    ++g_launches;
    if (g_profile[id].start) cudaEventRecord(g_profile[id].start, st);
  }
  ~LaunchScope() { if (g_profile[id].stop) cudaEventRecord(g_profile[id].stop, st); }
};

// Item table of the expert-sorted token order (built by k_route_scan).
struct RoutingTables {
  int* n_items;            // [1]
  int4* items;             // [max_items] {tile, expert, first row, end row}
  int* tile_item_begin;    // [mtiles + 1]
  int* expert_item_begin;  // [E + 1]
};

// Device pointers into the caller's `saved` buffer.
struct SavedPtrs {
  int8_t* q;
  uint16_t* xt;
  uint16_t* xs;
  float* gamma;
  float* gate;
  float* probs;
  int* expert;
  int* perm;
  int* pos;
  int* offsets;
  uint16_t* h;
  RoutingTables rt;
  int max_items;
};

struct FwdScratch {
  float* gate_tok;
  float* probs_tok;
  int* block_counts;
  int* block_base;
  float* rms;          // [T] per-token factor of a fused RMSNorm
};

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor in the stream is
// still draining, which hides its launch latency and set-up.  Every kernel launched this way starts with
// griddepcontrol.launch_dependents and griddepcontrol.wait, i.e. touches no global memory before the predecessor
// has completed; the result of the launch is picked up by the caller's cudaGetLastError().
template <class... KArgs, class... Args>
inline void launch_pdl(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid, 1, 1); cfg.blockDim = dim3((unsigned)block, 1, 1); cfg.dynamicSmemBytes = smem;
  cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// elementwise launchers (pq_elementwise.cu)
cudaError_t launch_pack(const float* W, int N, int K, uint32_t* bits, int8_t* s8, float* scales, double* partial, cudaStream_t st);
// st_quant: the stream of the quantisation kernel; it may differ from st only when E == 1 (no routing to wait for)
// norm_weight != nullptr: X is un-normalised and RMSNorm (gain [K] bf16, epsilon) is applied on the fly; the sorted copy
// xs of the tokens is then written even without routing (it is the only place the normalised activation exists)
cudaError_t launch_route_and_quant(const uint16_t* X, const uint16_t* Wr, int T, int K, int E, const SavedPtrs& sv, const FwdScratch& sc,
                                   cudaStream_t st, cudaStream_t st_quant, const uint16_t* norm_weight = nullptr, float norm_eps = 0.f);
cudaError_t launch_scatter_rows(const uint16_t* src, uint16_t* dst, const int* pos, int T, int row_elems, cudaStream_t st);
// arrivals: counter of the call's k_finalize_scales launch, cleared here (null: nothing to clear)
cudaError_t launch_scaled_sign(const int8_t* s8, uint16_t* out, const float* beta, int beta_stride, int N, int K, unsigned* arrivals,
                               cudaStream_t st);
cudaError_t launch_scaled_b(const uint16_t* B, uint16_t* out, const float* alpha, int E, int N, int r, cudaStream_t st);
cudaError_t launch_finalize_scales(const float* dbeta_partial, int nslots, const float* dalpha_partial, int E, int N, const float* w_scales,
                                   int vec, float* dbeta, float* dalpha, double* blk_sums, unsigned* arrivals, cudaStream_t st);
cudaError_t launch_fill_zero(void* p, size_t bytes, cudaStream_t st);
cudaError_t launch_swiglu(const uint16_t* G, const uint16_t* U, uint16_t* M, long long n, cudaStream_t st);
cudaError_t launch_ffn8_act(const int* g_int, const int* u_int, const float* gamma, const float* hp_scales, int T, int r, int8_t* qm,
                            float* gamma_m, cudaStream_t st);
cudaError_t launch_concat_experts(const uint16_t* B, int E, int N, int r, uint16_t* out, cudaStream_t st);
cudaError_t launch_pack_experts(const uint16_t* A, const uint16_t* B, int E, int r, int K, int N, int8_t* A8, int8_t* B8, float* hp_scales,
                                uint32_t* amax_bits, cudaStream_t st);

// tensor-core launchers (pq_gemm_kernels.cu).  All return a PQ_* status.
struct LayerArgs {
  int T, K, N, r, E;
  int scale_stride;  // 0: scalar alpha/beta, 1: per-feature vectors
  const float* w_scales;  // {lam, mu}
  const float* alpha;
  const float* beta;
  const uint16_t* A;   // [E,r,K]
  const uint16_t* B;   // [E,N,r]
  const uint16_t* Wr;  // [E,K]
  const float* hp_scales = nullptr;   // INT8 HP branch: [E][2] = {gamma_A, gamma_B}, and A, B then point to int8 codes
  bool hp_ext = false;                // INT8 HP branch whose hidden codes and gamma_h are already in the saved h region
};

int gemm_debug(int mode, int M, int N, int K, const void* A, const void* B, void* D, int tile_n, cudaStream_t st);
// before_main: an event the fused forward GEMM waits for (work on another stream that feeds it), or nullptr
int gemm_hp_up8(const LayerArgs& a, const SavedPtrs& sv, const void* A8, int* raw, cudaStream_t st);
int gemm_forward(const LayerArgs& a, const int8_t* w_s8, const SavedPtrs& sv, const uint16_t* xs, uint16_t* Y, cudaStream_t st,
                 cudaEvent_t before_main);

// decode path (pq_decode.cu)
size_t decode_workspace_bytes(int M, int K, int N, int r, bool dump);
int decode_forward(const LayerArgs& a, const uint16_t* X, const uint32_t* bits, uint16_t* Y, void* ws, bool dump, cudaStream_t st);
struct DecodeViewPtrs { void* tokens; int* acc; };
struct DecodeItemArgs {
  LayerArgs a; const uint16_t* X; const uint32_t* bits; uint16_t* Y; void* ws; bool dump;
  const uint16_t* norm_weight = nullptr;   // RMSNorm gain [K] bf16, or null: X arrives normalised
  float norm_eps = 0.f;
  const uint32_t* bits_il = nullptr;       // weights laid out by decode_pack (streaming kernel), or null
  const uint16_t* B_il = nullptr;          // bf16 rows of B_e, or the int8 codes B8_e when A8 is set
  const int8_t* A8 = nullptr;              // INT8 high-precision branch: codes of A_e [E, r, K], or null
  const float* hp_scales = nullptr;        // [E][2] {gamma_A, gamma_B}
};
// streaming decode kernel (pq_decode_stream.cu)
void decode_pack_sizes(int K, int N, int r, int E, size_t* bits_bytes, size_t* b_bytes);
int decode_pack(int K, int N, int r, int E, const uint32_t* bits, const uint16_t* B, uint32_t* bits_il, uint16_t* B_il, cudaStream_t st);
size_t decode_stream_extra_bytes(int M, int K, int N, int r, bool dump);
void decode_stream_view(int M, int K, int N, int r, void* ws, bool dump, int** h_int, int** z_int);
size_t decode_pack_b8_bytes(int N, int r, int E);
int decode_pack_b8(int N, int r, int E, const int8_t* B8, int8_t* B8_il, cudaStream_t st);
int decode_stream_launch(const DecodeItemArgs* items, int n, cudaStream_t st);   // PQ_ERR_UNSUPPORTED: use the other kernels
void decode_stream_enable(int mode);   // 0 never, 1 where it pays (default), 2 wherever the items allow
void decode_stream_prefetch(int on);
void decode_stream_mma_from(int m);
void decode_stream_interleave(int mode);
int decode_stream_mode();
void decode_stream_reset();
int decode_batch(const DecodeItemArgs* items, int n, cudaStream_t st);   // independent linears, launched together
void decode_set_pdl(int on);
DecodeViewPtrs decode_view(int M, int K, int N, int r, void* ws, bool dump);

struct BwdBuffers {
  const uint16_t* dys;   // [T,N] bf16 upstream gradient in sorted order
  const uint16_t* xs;    // [T,K] bf16 activations in sorted order
  const uint16_t* sb;    // [N,K] bf16 sign * (beta_n or 1)
  const uint16_t* ba;    // [E,N,r] bf16 B * (alpha_n or 1)
  uint16_t* dhc;         // [2][items*128, r] bf16 hi/lo planes of dH / c
  uint16_t* gh;          // [2][items*128, r] bf16 hi/lo planes of g * H
  float* dl;             // [T,E] fp32 router logit gradient (sorted order), kept for inspection
  uint16_t* dlc;         // [T,16] bf16 dl / c
  float* dbeta_partial;  // [2 * ceil(K/256), N]
  float* dalpha_partial; // [2 * E, N]
};
// Where the backward GEMMs run.  side == nullptr: all on st, in the order HP gradient, dX, dW (one launch with the
// HP tiles).  Otherwise the weight-gradient tiles that need nothing from the HP gradient GEMM are launched on st at
// once, the HP gradient GEMM and dX follow one another on `side` (already ordered after the scaled sign matrix), and
// the HP tiles of the weight gradient (dB, dA, router) go to st after `dh_done`; st then waits for `side_done`.
// Kernels of the two streams fill one another's last waves.
struct BwdStreams {
  cudaStream_t side = nullptr;
  cudaEvent_t dh_done = nullptr;     // recorded on side after the HP gradient GEMM
  cudaEvent_t side_done = nullptr;   // recorded on side after dX
};
int gemm_backward(const LayerArgs& a, const int8_t* w_s8, const SavedPtrs& sv, const BwdBuffers& b, uint16_t* dX, float* dW, float* dA,
                  float* dB, float* dWr, cudaStream_t st, const BwdStreams& bs);

}  // namespace pq
