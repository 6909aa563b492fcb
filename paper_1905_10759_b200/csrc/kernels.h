// Internal launcher interface between the C-ABI layer (api.cu) and the kernel files.
// Host-only declarations; every launcher enqueues on `stream` and returns the launch status.
#pragma once
#include <atomic>
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace hbmm {

// A kernel's opt-in shared-memory size is a per-device attribute, so "already configured" is kept per device
// (one process may drive several GPUs); setting it twice is harmless, hence no lock.
struct DeviceOnce {
  std::atomic<uint64_t> mask{0};
  bool pending(int dev) const { return dev < 0 || dev >= 64 || !((mask.load(std::memory_order_acquire) >> dev) & 1u); }
  void mark(int dev) { if (dev >= 0 && dev < 64) mask.fetch_or(uint64_t{1} << dev, std::memory_order_release); }
};
// Current device and its multiprocessor count.
inline cudaError_t current_device(int* dev, int* sms) {
  cudaError_t e = cudaGetDevice(dev);
  if (e != cudaSuccess) return e;
  return cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, *dev);
}

// Device-side view of one packed Hadamard-binary operand (validated by the caller).
struct PackedView {
  const uint32_t* bits;   // [rows, ld_words]
  const void* scales;     // [rows, ld_scales], fp32 or bf16
  int64_t rows, K;
  int64_t ld_words, ld_scales;
  int32_t beta;           // group length along K; >= K means one group per row
  int32_t scale_bf16;     // 0: fp32 scales, 1: bf16 scales
};

// Dense full-precision operand (beta = 1).
struct DenseView {
  const void* data;       // [rows, ld]
  int64_t rows, K, ld;
  int32_t bf16;           // 0: fp32, 1: bf16
};

struct ConvGeom {
  int32_t B, C, H, W, kh, kw, sh, sw, ph, pw, Ho, Wo;
};

// ceil(K / beta) with beta clamped to K (one group per row when beta >= K).
inline int64_t num_groups(int64_t K, int64_t beta) { return beta >= K ? 1 : (K + beta - 1) / beta; }

cudaError_t launch_quantize(const void* x, int x_bf16, int64_t rows, int64_t K, int64_t ldx,
                            uint32_t* bits, int64_t ld_words, void* scales, int64_t ld_scales,
                            int scale_bf16, int32_t beta, cudaStream_t stream);

// Gradient through the Hadamard binarization (Eq. 6 with the straight-through estimator of Eq. 5).
cudaError_t launch_binarize_backward(const float* x, int64_t ldx, const float* gy, int64_t ldg, int64_t rows, int64_t K, int32_t beta,
                                     float* gx, int64_t ldo, cudaStream_t stream);

// The binarized tensor written out dense, fp32 or bf16 (Eq. 2; Eq. 3-4 on an activation map's rows).
cudaError_t launch_binarize_dense(const float* x, int64_t ldx, int64_t rows, int64_t K, int32_t beta, void* out, bool out_bf16,
                                  int64_t ldo, cudaStream_t stream);

// Packed x packed contraction on the integer pipe (XOR + POPC).
cudaError_t launch_gemm_popc(const PackedView& A, const PackedView& W, float* C, int64_t ldc,
                             cudaStream_t stream);
cudaError_t launch_partials_popc(const PackedView& A, const PackedView& W, int32_t* D,
                                 cudaStream_t stream);

// The same for at most eight activation rows (batch 1 .. 8 of a fully connected layer): one warp per weight
// row, bound by reading the packed weights once.  Segments of 32, 64 or 128 elements.
bool gemv_popc_supported(const PackedView& A, const PackedView& W);
cudaError_t launch_gemv_popc(const PackedView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream);

// The same for sub-word segments (the finer grouping is 2, 4, 8 or 16 elements): masked popcounts inside a word.
bool gemm_subword(const PackedView& A, const PackedView& W);
cudaError_t launch_gemm_popc_sub(const PackedView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream);
cudaError_t launch_partials_popc_sub(const PackedView& A, const PackedView& W, int32_t* D, cudaStream_t stream);

// Packed x packed contraction on the legacy b1 tensor instruction (segment multiple of 128 bits).
bool gemm_b1_supported(const PackedView& A, const PackedView& W);
cudaError_t launch_gemm_b1(const PackedView& A, const PackedView& W, float* C, int64_t ldc,
                           cudaStream_t stream);
cudaError_t launch_partials_b1(const PackedView& A, const PackedView& W, int32_t* D,
                               cudaStream_t stream);

// What a tensor-core contraction does with a finished product tile besides storing it as fp32 (the chain of the
// paper's layer order, Section 5: convolution -> activation -> batch normalisation -> binarization of the next block):
//   y = act(C), z = bn_scale[n] * y + bn_shift[n], then z stored dense (fp32 or bf16, [M, ld_out]) or each row of z
//   Hadamard-binarized along n (Eq. 3-4) and only its packed form stored.
enum EpiMode : int32_t { kEpiPlain = 0, kEpiDense = 1, kEpiPacked = 2 };
struct EpiArgs {
  int32_t mode;             // EpiMode
  int32_t act;              // 0 none, 1 max(0, .)
  const float* bn_scale; const float* bn_shift;      // device, per column; null = 1 / 0
  void* out; int32_t out_bf16; int64_t ld_out;       // dense
  uint32_t* nx_bits; void* nx_scales;                // packed: the next layer's operand (rows = M, K = N)
  int64_t nx_ld_words, nx_ld_scales;
  int32_t nx_bf16, nx_beta;
};
inline EpiArgs plain_epilogue() { EpiArgs e{}; e.mode = kEpiPlain; e.nx_beta = 32; return e; }

// Argument block of the tcgen05 HBMM kernel and of its weight-expansion routine.
struct UmmaArgs {
  const uint32_t* a_bits; const void* a_scales;
  const uint32_t* w_bits; const void* w_scales;
  float* C;
  int64_t M, N, lda_w, ldw_w, lda_s, ldw_s, ldc;
  int32_t a_bf16, w_bf16;
  int32_t ra, rw;          // A group = segment / ra, W group = segment / rw
  int64_t Ga, Gw;
  int64_t n_words;         // K / 32 (K is a multiple of 32 on this path)
  int64_t seg_words;       // K-words per segment
  const unsigned char* w_prep;   // W expanded into [n tile][stage][stage bytes]
};
// Argument block of the folded-scale tcgen05 HBMM kernel (group scales carried by fp16 operand pieces).
struct FoldArgs {
  const uint32_t* a_bits; const void* a_scales;
  const uint32_t* w_bits; const void* w_scales;
  float* C;
  int64_t M, N, lda_w, ldw_w, lda_s, ldw_s, ldc;
  int32_t a_bf16, w_bf16;
  int64_t n_words;         // K / 32 (K is a multiple of 32 on this path)
  int64_t a_gw, w_gw;      // K-words per scale group of A / W (n_words: one group per row)
  int32_t a_sub, w_sub;    // scale groups per K-word: 1, or 32 / beta for the sub-word groups beta = 2 .. 16
  const unsigned char* w_prep;   // W expanded into [n tile][stage][stage bytes]
  const float* w_down;           // per weight row: the power of two that undoes its normalisation
  EpiArgs ep;                    // what the epilogue does with a finished tile (ep.mode == kEpiPlain: store C as fp32)
  // Balanced schedule (sk_units > 0): the (tile, stage) pairs of the whole product, tile-major, are cut into
  // equal runs of sk_units, one per CTA, so a tile's K range may be shared by several CTAs.  A CTA that holds only
  // part of a tile stores its raw partial accumulator in its own slot of sk_partials and counts itself in
  // sk_counters[tile][epilogue warp]; the last one to arrive adds the tile's partials in CTA order and finishes it.
  int64_t sk_units;
  int32_t* sk_counters;          // [tiles][4]: zeroed by the weight expansion, left at zero by every launch
  int64_t sk_counter_count;
  float* sk_partials;            // [2 * CTAs][128][TN]
  float* a_rowmax;               // sub-word groups: largest scale of every activation row (nullptr: the scouts scan the rows)
  int32_t a_staged;              // sub-word groups: the activation scales of a stage reach the producers through shared memory
};
// The weight expansion as a job another kernel can run: n_stages x tiles_n tasks of tn threads each
// (n_stages counts tasks per column tile: single stages of the e4m3 layout, runs of stages of the folded one).
// folded == 0: the e4m3 kernel's layout (g); folded == 1: the folded-scale kernel's layout (f, out_down).
struct UmmaPrepJob {
  UmmaArgs g;
  FoldArgs f;
  unsigned char* out;
  float* out_down;
  int32_t folded;
  int32_t tn, n_stages, tiles_n;
};

// Packed x packed contraction with +-1 e4m3 operands on the tensor cores (tcgen05 / TMEM).
// *_health: the device-side error word of a kernel family (0 = no bounded wait has expired since it was
// last cleared) and the poll limit of its waits.  Read copies the word to *value, Clear zeroes it,
// SetSpinLimit stores *value polls (0 = the default).  All three synchronise with the device.
enum HealthOp { kHealthRead = 0, kHealthClear = 1, kHealthSetSpinLimit = 2 };
cudaError_t gemm_umma_health(int op, int* value);
cudaError_t hbwn_umma_health(int op, int* value);
bool gemm_tensor_supported(const PackedView& A, const PackedView& W);
size_t gemm_tensor_workspace_bytes(const PackedView& A, const PackedView& W);
// w_prepared: the workspace already holds the expanded weight operand of exactly these operands (a
// front-end kernel ran gemm_tensor_prep_job's tasks earlier on the same stream).
cudaError_t launch_gemm_tensor(const PackedView& A, const PackedView& W, float* C, int64_t ldc, void* workspace,
                               cudaStream_t stream, bool w_prepared = false);
void gemm_tensor_prep_job(const PackedView& A, const PackedView& W, void* workspace, UmmaPrepJob* job);

// Packed x packed contraction with the group scales folded into two fp16 pieces per operand (tcgen05 /
// TMEM, one accumulation over all of K, no per-group step).  Same operand support as the e4m3 kernel.
cudaError_t gemm_fold_health(int op, int* value);
// Test only: one thread waits on a barrier nobody arrives at, with the family's bounded wait (code 9).
cudaError_t launch_wait_expiry_selftest(cudaStream_t stream);
bool gemm_fold_supported(const PackedView& A, const PackedView& W);
size_t gemm_fold_workspace_bytes(const PackedView& A, const PackedView& W);
cudaError_t launch_gemm_fold(const PackedView& A, const PackedView& W, float* C, int64_t ldc, void* workspace,
                             cudaStream_t stream, bool w_prepared = false, const EpiArgs* ep = nullptr);
// Group sizes the fused epilogue can emit for an output of N columns.
bool gemm_fold_next_supported(int64_t N, int32_t beta_next);
void gemm_fold_prep_job(const PackedView& A, const PackedView& W, void* workspace, UmmaPrepJob* job);

// Dense x packed contraction (HBWN), three kernels:
//   select : sign bit XOR-ed into fp32 activations on the fp32 pipe (any dense dtype);
//   mma    : legacy warp-level bf16 mma.sync with per-group partial sums (bf16 activations);
//   umma   : tcgen05, weights as three stacked bf16 pieces prepared in a workspace (bf16 activations,
//            16-byte aligned rows).
cudaError_t launch_hbwn_select(const DenseView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream);
bool hbwn_mma_supported(const DenseView& A, const PackedView& W);
cudaError_t launch_hbwn_mma(const DenseView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream);
bool hbwn_umma_supported(const DenseView& A, const PackedView& W);
size_t hbwn_umma_workspace_bytes(const DenseView& A, const PackedView& W);
// exact: three bf16 pieces per weight (group scale to 2^-26); otherwise two (2^-17), the faster layout.
cudaError_t launch_hbwn_umma(const DenseView& A, const PackedView& W, float* C, int64_t ldc, void* workspace,
                             cudaStream_t stream, bool w_prepared = false, bool exact = false, const EpiArgs* ep = nullptr);

// HBWN convolution without the im2col matrix: NCHW -> NHWC bf16 copy (Cp = channels rounded up to 8;
// launch_hbwn_umma_conv does it in the same launch as the weight-piece layout), then the tcgen05 kernel
// reads its activation tiles from x_nhwc with im2col-mode tensor copies.
cudaError_t launch_nchw_to_nhwc_bf16(const void* x, int x_bf16, const ConvGeom& g, void* out, int Cp, cudaStream_t stream);
bool hbwn_umma_conv_supported(const ConvGeom& g, const PackedView& W);
size_t hbwn_umma_conv_workspace_bytes(const ConvGeom& g, const PackedView& W);
// w_prepared: the workspace still holds the weight pieces an earlier call with the same W and geometry laid out.
// ep (optional): epilogue chain instead of the fp32 store.  input_is_nhwc: x already is an NHWC bf16 image with
// channel pitch Cp (16-byte aligned), so the layout copy is skipped and x_nhwc is not used.
cudaError_t launch_hbwn_umma_conv(const void* x, int x_bf16, void* x_nhwc, int Cp, const ConvGeom& g, const PackedView& W, float* C,
                                  int64_t ldc, void* workspace, cudaStream_t stream, bool w_prepared = false,
                                  const EpiArgs* ep = nullptr, bool input_is_nhwc = false);

// im2col gather fused with Hadamard binarization (packed output), and bf16 dense gather.
cudaError_t launch_im2col_quantize(const void* x, int x_bf16, const ConvGeom& g, int32_t beta,
                                   uint32_t* bits, int64_t ld_words, void* scales, int64_t ld_scales,
                                   int scale_bf16, cudaStream_t stream);
// The packed front end with its input tile staged by tensor copies (fp32 input, beta = 32).
bool im2col_quantize_tma_supported(const void* x, int x_bf16, const ConvGeom& g, int32_t beta);
// prep (optional): weight-expansion tasks of the contraction that follows, run by extra CTAs of the launch.
cudaError_t launch_im2col_quantize_tma(const void* x, const ConvGeom& g, int32_t beta, uint32_t* bits, int64_t ld_words, void* scales,
                                       int64_t ld_scales, int scale_bf16, cudaStream_t stream, const UmmaPrepJob* prep = nullptr);
cudaError_t im2col_tma_health(int op, int* value);
// Register-only arithmetic loop for measuring a unit's issue rate (kind 0: XOR + POPC, 1: fp32 add, 2: fp32
// fused multiply-add): blocks x 1024 threads, iters x 8 operations each; *ops = operations per launch.
// sink: device, at least blocks * 1024 words (never written in practice).
cudaError_t launch_alu_rate(int kind, int blocks, int iters, uint32_t* sink, int64_t* ops, cudaStream_t stream);

cudaError_t launch_im2col_bf16(const void* x, int x_bf16, const ConvGeom& g, void* out, int64_t ld,
                               cudaStream_t stream);

}  // namespace hbmm
