// C-ABI layer: argument validation on the host, then dispatch to the kernel launchers.
// Nothing here allocates device memory or synchronises; see include/hbmm.h for the contract.
#include <cstdint>
#include <cstddef>
#include "../../include/hbmm.h"
#include "kernels.h"

using namespace hbmm;

namespace {

constexpr int32_t kVersion = 100;  // 0.1.0

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool valid_dtype(int32_t d) { return d == HBMM_F32 || d == HBMM_BF16; }
inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

inline int64_t words_ld(int64_t K) { return round_up((K + 31) / 32, 4); }
inline int64_t scales_ld(int64_t K, int32_t beta, int32_t dtype) {
  return round_up(num_groups(K, beta), dtype == HBMM_BF16 ? 8 : 4);
}

// beta values the packed kernels implement: whole words per group, one group per row, or the sub-word
// powers of two (the settings of the paper's experiments).
inline bool beta_supported(int64_t K, int32_t beta) {
  return beta >= 2 && (beta % 32 == 0 || beta >= K || beta == 2 || beta == 4 || beta == 8 || beta == 16);
}

hbmm_status check_packed(const hbmm_operand* op, bool need_buffers = true) {
  if (!op) return HBMM_ERR_INVALID_ARG;
  if (op->rows <= 0 || op->K <= 0 || op->beta < 2) return HBMM_ERR_INVALID_ARG;
  if (!valid_dtype(op->scale_dtype)) return HBMM_ERR_INVALID_ARG;
  if (!beta_supported(op->K, op->beta)) return HBMM_ERR_UNSUPPORTED;
  if (need_buffers) {
    if (!op->bits || !op->scales) return HBMM_ERR_INVALID_ARG;
    if (op->ld_words < (op->K + 31) / 32 || op->ld_scales < num_groups(op->K, op->beta)) return HBMM_ERR_INVALID_ARG;
    if (!aligned16(op->bits) || !aligned16(op->scales)) return HBMM_ERR_ALIGNMENT;
    if (op->ld_words % 4 != 0) return HBMM_ERR_ALIGNMENT;
    if (op->ld_scales % (op->scale_dtype == HBMM_BF16 ? 8 : 4) != 0) return HBMM_ERR_ALIGNMENT;
  }
  return HBMM_OK;
}

PackedView view_of(const hbmm_operand* op) {
  PackedView v;
  v.bits = op->bits; v.scales = op->scales; v.rows = op->rows; v.K = op->K;
  v.ld_words = op->ld_words; v.ld_scales = op->ld_scales; v.beta = op->beta;
  v.scale_bf16 = op->scale_dtype == HBMM_BF16;
  return v;
}

// Both packed: the coarser grouping must be a whole number of the finer groups.
bool segments_compatible(const hbmm_operand* A, const hbmm_operand* W) {
  const bool a_one = A->beta >= A->K, w_one = W->beta >= W->K;
  if (a_one || w_one) return true;
  const int64_t lo = A->beta < W->beta ? A->beta : W->beta, hi = A->beta < W->beta ? W->beta : A->beta;
  return hi % lo == 0;
}

hbmm_status check_c(const float* C, int64_t ldc, int64_t N) {
  if (!C || ldc < N) return HBMM_ERR_INVALID_ARG;
  if (!aligned16(C) || ldc % 4 != 0) return HBMM_ERR_ALIGNMENT;
  return HBMM_OK;
}

// Workspace of the tensor-core contraction for these (validated, packed) operands, 0 when that path
// cannot run them.
size_t tensor_workspace(const PackedView& a, const PackedView& w) {
  return gemm_tensor_supported(a, w) ? static_cast<size_t>(round_up(static_cast<int64_t>(gemm_tensor_workspace_bytes(a, w)), 256)) : 0;
}
size_t fold_workspace(const PackedView& a, const PackedView& w) {
  return gemm_fold_supported(a, w) ? static_cast<size_t>(round_up(static_cast<int64_t>(gemm_fold_workspace_bytes(a, w)), 256)) : 0;
}
// Which tensor-core kernel the automatic choice takes.  The folded-scale kernel sums the K individual
// products in fp32, so its error follows sum_k |A~||W~| rather than sum_g |deltaA deltaW D_g|; the two drift
// apart as groups grow (for a group of n random signs |D| is about sqrt(n)).  Up to 128 elements per
// group it stays well inside 1e-5 of the latter and is the faster kernel; beyond that the e4m3 kernel,
// whose integer group dots are exact and whose per-group step has become rare, is both.
bool prefer_fold(const PackedView& a, const PackedView& w) {
  const int64_t ba = a.beta >= a.K ? a.K : a.beta, bw = w.beta >= w.K ? w.K : w.beta;
  return gemm_fold_supported(a, w) && (ba < bw ? ba : bw) <= 128;
}
// What hbmm_gemm_workspace_bytes reports for two packed operands: enough for either tensor-core kernel.
size_t packed_workspace(const PackedView& a, const PackedView& w) {
  const size_t t = tensor_workspace(a, w), f = fold_workspace(a, w);
  return t > f ? t : f;
}
size_t hbwn_workspace(const DenseView& a, const PackedView& w) {
  return hbwn_umma_supported(a, w) ? static_cast<size_t>(round_up(static_cast<int64_t>(hbwn_umma_workspace_bytes(a, w)), 256)) : 0;
}
DenseView dense_view_of(const hbmm_operand* A) {
  DenseView dv;
  dv.data = A->dense; dv.rows = A->rows; dv.K = A->K; dv.ld = A->ld_dense; dv.bf16 = A->dense_dtype == HBMM_BF16;
  return dv;
}
inline bool workspace_ok(const void* ws, size_t have, size_t need) {
  return need == 0 || (ws != nullptr && have >= need && (reinterpret_cast<uintptr_t>(ws) & 15u) == 0);
}

// The integer-pipe contraction that fits the operands: matrix-vector shaped, sub-word segments, or tiled.
cudaError_t popc_any(const PackedView& a, const PackedView& w, float* C, int64_t ldc, cudaStream_t stream) {
  if (gemv_popc_supported(a, w)) return launch_gemv_popc(a, w, C, ldc, stream);
  return gemm_subword(a, w) ? launch_gemm_popc_sub(a, w, C, ldc, stream) : launch_gemm_popc(a, w, C, ldc, stream);
}

hbmm_status gemm_checked(const hbmm_operand* A, const hbmm_operand* W, float* C, int64_t ldc,
                         int32_t path, void* workspace, size_t workspace_bytes, cudaStream_t stream) {
  if (!A || !W) return HBMM_ERR_INVALID_ARG;
  if (W->beta == 1) return HBMM_ERR_UNSUPPORTED;  // the weight operand is always Hadamard-binary
  hbmm_status st = check_packed(W);
  if (st != HBMM_OK) return st;
  if (path < HBMM_PATH_AUTO || path > HBMM_PATH_FOLDED_PREPARED) return HBMM_ERR_INVALID_ARG;
  const bool w_prepared = path == HBMM_PATH_TENSOR_PREPARED || path == HBMM_PATH_FOLDED_PREPARED;
  if (path == HBMM_PATH_TENSOR_PREPARED) path = HBMM_PATH_TENSOR;
  if (path == HBMM_PATH_FOLDED_PREPARED) path = HBMM_PATH_FOLDED;
  if (A->beta == 1) {
    if (A->rows <= 0 || A->K <= 0 || !A->dense || A->ld_dense < A->K || !valid_dtype(A->dense_dtype))
      return HBMM_ERR_INVALID_ARG;
    if (A->K != W->K) return HBMM_ERR_INVALID_ARG;
    if ((st = check_c(C, ldc, W->rows)) != HBMM_OK) return st;
    const DenseView dv = dense_view_of(A);
    const PackedView w = view_of(W);
    const bool umma = hbwn_umma_supported(dv, w) && workspace_ok(workspace, workspace_bytes, hbwn_workspace(dv, w));
    cudaError_t e;
    switch (path) {
      case HBMM_PATH_POPC: e = launch_hbwn_select(dv, w, C, ldc, stream); break;
      case HBMM_PATH_B1MMA:
        if (!hbwn_mma_supported(dv, w)) return HBMM_ERR_UNSUPPORTED;
        e = launch_hbwn_mma(dv, w, C, ldc, stream);
        break;
      case HBMM_PATH_FOLDED:      // two bf16 pieces per weight (group scale to 2^-17)
      case HBMM_PATH_TENSOR:      // three (2^-26)
        if (!hbwn_umma_supported(dv, w)) return HBMM_ERR_UNSUPPORTED;
        if (!umma) return HBMM_ERR_WORKSPACE;
        e = launch_hbwn_umma(dv, w, C, ldc, workspace, stream, w_prepared, path == HBMM_PATH_TENSOR);
        break;
      default:
        if (umma) e = launch_hbwn_umma(dv, w, C, ldc, workspace, stream);
        else if (hbwn_mma_supported(dv, w)) e = launch_hbwn_mma(dv, w, C, ldc, stream);
        else e = launch_hbwn_select(dv, w, C, ldc, stream);
        break;
    }
    return e == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
  }
  if ((st = check_packed(A)) != HBMM_OK) return st;
  if (A->K != W->K) return HBMM_ERR_INVALID_ARG;
  if (!segments_compatible(A, W)) return HBMM_ERR_UNSUPPORTED;
  if ((st = check_c(C, ldc, W->rows)) != HBMM_OK) return st;
  const PackedView a = view_of(A), w = view_of(W);
  cudaError_t e;
  switch (path) {
    case HBMM_PATH_POPC: e = popc_any(a, w, C, ldc, stream); break;
    case HBMM_PATH_B1MMA:
      if (!gemm_b1_supported(a, w)) return HBMM_ERR_UNSUPPORTED;
      e = launch_gemm_b1(a, w, C, ldc, stream);
      break;
    case HBMM_PATH_TENSOR:
      if (!gemm_tensor_supported(a, w)) return HBMM_ERR_UNSUPPORTED;
      if (!workspace_ok(workspace, workspace_bytes, tensor_workspace(a, w))) return HBMM_ERR_WORKSPACE;
      e = launch_gemm_tensor(a, w, C, ldc, workspace, stream, w_prepared);
      break;
    case HBMM_PATH_FOLDED:
      if (!gemm_fold_supported(a, w)) return HBMM_ERR_UNSUPPORTED;
      if (!workspace_ok(workspace, workspace_bytes, fold_workspace(a, w))) return HBMM_ERR_WORKSPACE;
      e = launch_gemm_fold(a, w, C, ldc, workspace, stream, w_prepared);
      break;
    default:
      // a handful of activation rows: reading the packed weights once beats any tile kernel (and the expanded
      // weight operand of the tensor-core paths is 32 times larger than the packed one)
      if (gemv_popc_supported(a, w)) e = launch_gemv_popc(a, w, C, ldc, stream);
      // the tensor-core paths need their workspace; without one the integer-pipe path runs
      else if (prefer_fold(a, w) && workspace_ok(workspace, workspace_bytes, fold_workspace(a, w)))
        e = launch_gemm_fold(a, w, C, ldc, workspace, stream);
      else if (gemm_tensor_supported(a, w) && workspace_ok(workspace, workspace_bytes, tensor_workspace(a, w)))
        e = launch_gemm_tensor(a, w, C, ldc, workspace, stream);
      else
        e = popc_any(a, w, C, ldc, stream);
      break;
  }
  return e == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
}

hbmm_status check_geom(const hbmm_conv_geom* g, ConvGeom* out) {
  if (!g) return HBMM_ERR_INVALID_ARG;
  if (g->B <= 0 || g->C <= 0 || g->H <= 0 || g->W <= 0 || g->kh <= 0 || g->kw <= 0 || g->stride_h <= 0 ||
      g->stride_w <= 0 || g->pad_h < 0 || g->pad_w < 0)
    return HBMM_ERR_INVALID_ARG;
  const int64_t ho = (static_cast<int64_t>(g->H) + 2 * g->pad_h - g->kh) / g->stride_h + 1;
  const int64_t wo = (static_cast<int64_t>(g->W) + 2 * g->pad_w - g->kw) / g->stride_w + 1;
  if (g->H + 2 * g->pad_h < g->kh || g->W + 2 * g->pad_w < g->kw || ho <= 0 || wo <= 0) return HBMM_ERR_INVALID_ARG;
  if (static_cast<int64_t>(g->C) * g->kh * g->kw > INT32_MAX) return HBMM_ERR_INVALID_ARG;
  out->B = g->B; out->C = g->C; out->H = g->H; out->W = g->W; out->kh = g->kh; out->kw = g->kw;
  out->sh = g->stride_h; out->sw = g->stride_w; out->ph = g->pad_h; out->pw = g->pad_w;
  out->Ho = static_cast<int32_t>(ho); out->Wo = static_cast<int32_t>(wo);
  return HBMM_OK;
}

struct ConvLayout {
  int64_t M, K, ld_words, ld_scales, ld_dense;
  bool implicit;     // beta_a == 1 only: NHWC copy + im2col-mode tensor copies instead of the im2col matrix
  int32_t Cp;        // channel pitch of that copy
  size_t bits_bytes, scales_bytes, operand_bytes, gemm_bytes, total;
};

ConvLayout conv_layout(const ConvGeom& g, int32_t beta_a, int32_t scale_dtype, const hbmm_operand* W) {
  ConvLayout L{};
  L.M = static_cast<int64_t>(g.B) * g.Ho * g.Wo;
  L.K = static_cast<int64_t>(g.C) * g.kh * g.kw;
  if (beta_a == 1 && W && W->K == L.K && hbwn_umma_conv_supported(g, view_of(W))) {
    L.implicit = true;
    L.Cp = static_cast<int32_t>(round_up(g.C, 8));
    L.operand_bytes = static_cast<size_t>(round_up(static_cast<int64_t>(g.B) * g.H * g.W * L.Cp * 2, 256));
    L.gemm_bytes = static_cast<size_t>(round_up(static_cast<int64_t>(hbwn_umma_conv_workspace_bytes(g, view_of(W))), 256));
    L.total = L.operand_bytes + L.gemm_bytes;
  } else if (beta_a == 1) {
    L.ld_dense = round_up(L.K, 8);
    L.operand_bytes = static_cast<size_t>(round_up(L.M * L.ld_dense * 2, 256));
    // the tensor-core contraction's prepared weight pieces follow the bf16 rows
    DenseView a;
    a.data = nullptr; a.rows = L.M; a.K = L.K; a.ld = L.ld_dense; a.bf16 = 1;
    L.gemm_bytes = (W && W->K == L.K) ? hbwn_workspace(a, view_of(W)) : 0;
    L.total = L.operand_bytes + L.gemm_bytes;
  } else {
    L.ld_words = words_ld(L.K);
    L.ld_scales = scales_ld(L.K, beta_a, scale_dtype);
    L.bits_bytes = static_cast<size_t>(round_up(L.M * L.ld_words * 4, 256));
    L.scales_bytes = static_cast<size_t>(round_up(L.M * L.ld_scales * (scale_dtype == HBMM_BF16 ? 2 : 4), 256));
    L.operand_bytes = L.bits_bytes + L.scales_bytes;
    // the contraction's own workspace follows the packed activation operand
    PackedView a;
    a.bits = nullptr; a.scales = nullptr; a.rows = L.M; a.K = L.K; a.ld_words = L.ld_words; a.ld_scales = L.ld_scales;
    a.beta = beta_a; a.scale_bf16 = scale_dtype == HBMM_BF16;
    hbmm_operand Aop{};
    Aop.rows = L.M; Aop.K = L.K; Aop.beta = beta_a;
    L.gemm_bytes = (W && W->K == L.K && segments_compatible(&Aop, W)) ? packed_workspace(a, view_of(W)) : 0;
    L.total = L.operand_bytes + L.gemm_bytes;
  }
  return L;
}

// Validates a caller's epilogue description for an M x N product and translates it for the kernels.
hbmm_status make_epilogue(const hbmm_epilogue* ep, int64_t M, int64_t N, EpiArgs* out) {
  EpiArgs e = plain_epilogue();
  if (ep->activation != HBMM_ACT_NONE && ep->activation != HBMM_ACT_RELU) return HBMM_ERR_INVALID_ARG;
  if ((ep->bn_scale && reinterpret_cast<uintptr_t>(ep->bn_scale) % 4 != 0) || (ep->bn_shift && reinterpret_cast<uintptr_t>(ep->bn_shift) % 4 != 0))
    return HBMM_ERR_ALIGNMENT;
  e.act = ep->activation == HBMM_ACT_RELU ? 1 : 0;
  e.bn_scale = ep->bn_scale; e.bn_shift = ep->bn_shift;
  if (ep->out_kind == HBMM_OUT_DENSE) {
    if (!ep->out || !valid_dtype(ep->out_dtype) || ep->ld_out < N) return HBMM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(ep->out) % (ep->out_dtype == HBMM_BF16 ? 2 : 4) != 0) return HBMM_ERR_ALIGNMENT;
    e.mode = kEpiDense; e.out = ep->out; e.out_bf16 = ep->out_dtype == HBMM_BF16; e.ld_out = ep->ld_out;
  } else if (ep->out_kind == HBMM_OUT_PACKED) {
    const hbmm_operand* nx = ep->next;
    if (!nx || nx->rows != M || nx->K != N) return HBMM_ERR_INVALID_ARG;
    const hbmm_status st = check_packed(nx);
    if (st != HBMM_OK) return st;
    if (nx->beta >= nx->K) return HBMM_ERR_UNSUPPORTED;
    e.mode = kEpiPacked; e.nx_bits = nx->bits; e.nx_scales = nx->scales; e.nx_ld_words = nx->ld_words; e.nx_ld_scales = nx->ld_scales;
    e.nx_bf16 = nx->scale_dtype == HBMM_BF16; e.nx_beta = nx->beta;
  } else {
    return HBMM_ERR_INVALID_ARG;
  }
  *out = e;
  return HBMM_OK;
}

hbmm_status conv_checked(const void* x, int32_t x_dtype, const hbmm_conv_geom* g, int32_t beta_a, int32_t a_scale_dtype,
                         const hbmm_operand* W, float* C_out, int64_t ldc, const hbmm_epilogue* ep, void* workspace,
                         size_t workspace_bytes, uint32_t flags, void* stream);

}  // namespace

extern "C" {

hbmm_status hbmm_operand_bytes(int64_t rows, int64_t K, int32_t beta, int32_t scale_dtype,
                               size_t* bits_bytes, size_t* scales_bytes, int64_t* ld_words, int64_t* ld_scales) {
  if (rows <= 0 || K <= 0 || beta < 2 || !valid_dtype(scale_dtype)) return HBMM_ERR_INVALID_ARG;
  const int64_t lw = words_ld(K), ls = scales_ld(K, beta, scale_dtype);
  if (bits_bytes) *bits_bytes = static_cast<size_t>(rows) * lw * 4;
  if (scales_bytes) *scales_bytes = static_cast<size_t>(rows) * ls * (scale_dtype == HBMM_BF16 ? 2 : 4);
  if (ld_words) *ld_words = lw;
  if (ld_scales) *ld_scales = ls;
  return HBMM_OK;
}

hbmm_status hbmm_quantize(const void* x, int32_t x_dtype, int64_t rows, int64_t K, int64_t ldx,
                          const hbmm_operand* out, void* stream) {
  if (!x || !out || rows <= 0 || K <= 0 || ldx < K || !valid_dtype(x_dtype)) return HBMM_ERR_INVALID_ARG;
  if (out->rows != rows || out->K != K) return HBMM_ERR_INVALID_ARG;
  hbmm_status st = check_packed(out);
  if (st != HBMM_OK) return st;
  if ((reinterpret_cast<uintptr_t>(x) % (x_dtype == HBMM_BF16 ? 2 : 4)) != 0) return HBMM_ERR_ALIGNMENT;
  const cudaError_t e = launch_quantize(x, x_dtype == HBMM_BF16, rows, K, ldx, out->bits, out->ld_words, out->scales,
                                        out->ld_scales, out->scale_dtype == HBMM_BF16, out->beta,
                                        static_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return HBMM_ERR_UNSUPPORTED;
  return e == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
}

hbmm_status hbmm_binarize_backward(const float* x, int64_t ldx, const float* gy, int64_t ldg, int64_t rows, int64_t K,
                                   int32_t beta, float* gx, int64_t ldo, void* stream) {
  if (!x || !gy || !gx || rows <= 0 || K <= 0 || beta < 1 || ldx < K || ldg < K || ldo < K) return HBMM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(x) % 4 != 0 || reinterpret_cast<uintptr_t>(gy) % 4 != 0 || reinterpret_cast<uintptr_t>(gx) % 4 != 0)
    return HBMM_ERR_ALIGNMENT;
  return launch_binarize_backward(x, ldx, gy, ldg, rows, K, beta, gx, ldo, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? HBMM_OK : HBMM_ERR_CUDA;
}

hbmm_status hbmm_binarize_dense(const float* x, int64_t ldx, int64_t rows, int64_t K, int32_t beta, void* out, int32_t out_dtype,
                                int64_t ldo, void* stream) {
  if (!x || !out || rows <= 0 || K <= 0 || beta < 1 || ldx < K || ldo < K || !valid_dtype(out_dtype)) return HBMM_ERR_INVALID_ARG;
  const uintptr_t out_align = out_dtype == HBMM_BF16 ? 2 : 4;
  if (reinterpret_cast<uintptr_t>(x) % 4 != 0 || reinterpret_cast<uintptr_t>(out) % out_align != 0) return HBMM_ERR_ALIGNMENT;
  return launch_binarize_dense(x, ldx, rows, K, beta, out, out_dtype == HBMM_BF16, ldo, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? HBMM_OK : HBMM_ERR_CUDA;
}

hbmm_status hbmm_gemm_workspace_bytes(const hbmm_operand* A, const hbmm_operand* W, size_t* bytes) {
  if (!A || !W || !bytes) return HBMM_ERR_INVALID_ARG;
  *bytes = 0;
  if (A->beta >= 2 && W->beta >= 2 && check_packed(A, false) == HBMM_OK && check_packed(W, false) == HBMM_OK &&
      A->K == W->K && segments_compatible(A, W))
    *bytes = packed_workspace(view_of(A), view_of(W));
  else if (A->beta == 1 && W->beta >= 2 && A->dense && A->rows > 0 && A->K == W->K && A->ld_dense >= A->K &&
           valid_dtype(A->dense_dtype) && check_packed(W, false) == HBMM_OK)
    *bytes = hbwn_workspace(dense_view_of(A), view_of(W));
  return HBMM_OK;
}

hbmm_status hbmm_gemm(const hbmm_operand* A, const hbmm_operand* W, float* C, int64_t ldc, void* workspace,
                      size_t workspace_bytes, void* stream) {
  return gemm_checked(A, W, C, ldc, HBMM_PATH_AUTO, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

hbmm_status hbmm_gemm_ex(const hbmm_operand* A, const hbmm_operand* W, float* C, int64_t ldc, void* workspace,
                         size_t workspace_bytes, int32_t path, void* stream) {
  return gemm_checked(A, W, C, ldc, path, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

hbmm_status hbmm_gemm_fused(const hbmm_operand* A, const hbmm_operand* W, const hbmm_epilogue* ep, void* workspace,
                            size_t workspace_bytes, void* stream) {
  hbmm_status st;
  if (!A || !W || !ep) return HBMM_ERR_INVALID_ARG;
  if (W->beta == 1) return HBMM_ERR_UNSUPPORTED;                       // the weight operand is always Hadamard-binary
  if ((st = check_packed(W)) != HBMM_OK) return st;
  if (A->K != W->K) return HBMM_ERR_INVALID_ARG;
  EpiArgs e;
  if ((st = make_epilogue(ep, A->rows, W->rows, &e)) != HBMM_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const PackedView w = view_of(W);
  if (A->beta == 1) {
    if (A->rows <= 0 || A->K <= 0 || !A->dense || A->ld_dense < A->K || !valid_dtype(A->dense_dtype)) return HBMM_ERR_INVALID_ARG;
    const DenseView dv = dense_view_of(A);
    if (!hbwn_umma_supported(dv, w)) return HBMM_ERR_UNSUPPORTED;     // bf16 rows on 16-byte boundaries
    if (e.mode == kEpiPacked && !gemm_fold_next_supported(W->rows, e.nx_beta)) return HBMM_ERR_UNSUPPORTED;
    if (!workspace_ok(workspace, workspace_bytes, hbwn_workspace(dv, w))) return HBMM_ERR_WORKSPACE;
    return launch_hbwn_umma(dv, w, nullptr, 0, workspace, s, false, false, &e) == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
  }
  if ((st = check_packed(A)) != HBMM_OK) return st;
  const PackedView a = view_of(A);
  const bool a_subword = A->beta < 32 && A->beta < A->K;
  if (!segments_compatible(A, W) || !gemm_fold_supported(a, w) || a_subword) return HBMM_ERR_UNSUPPORTED;
  if (e.mode == kEpiPacked && !gemm_fold_next_supported(W->rows, e.nx_beta)) return HBMM_ERR_UNSUPPORTED;
  if (!workspace_ok(workspace, workspace_bytes, fold_workspace(a, w))) return HBMM_ERR_WORKSPACE;
  return launch_gemm_fold(a, w, nullptr, 0, workspace, s, false, &e) == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
}

hbmm_status hbmm_gemm_binarize_next(const hbmm_operand* A, const hbmm_operand* W, const float* bn_scale, const float* bn_shift,
                                    const hbmm_operand* next, void* workspace, size_t workspace_bytes, void* stream) {
  if (!A || !W || !next) return HBMM_ERR_INVALID_ARG;
  if (A->beta == 1 || W->beta == 1) return HBMM_ERR_UNSUPPORTED;       // both operands packed
  hbmm_epilogue ep{};
  ep.activation = HBMM_ACT_NONE; ep.out_kind = HBMM_OUT_PACKED; ep.bn_scale = bn_scale; ep.bn_shift = bn_shift; ep.next = next;
  return hbmm_gemm_fused(A, W, &ep, workspace, workspace_bytes, stream);
}

hbmm_status hbmm_gemm_partials(const hbmm_operand* A, const hbmm_operand* W, int32_t* D, int32_t path, void* stream) {
  hbmm_status st;
  if ((st = check_packed(A)) != HBMM_OK) return st;
  if ((st = check_packed(W)) != HBMM_OK) return st;
  if (!D || A->K != W->K) return HBMM_ERR_INVALID_ARG;
  if (!segments_compatible(A, W)) return HBMM_ERR_UNSUPPORTED;
  const PackedView a = view_of(A), w = view_of(W);
  cudaError_t e;
  if (path == HBMM_PATH_AUTO || path == HBMM_PATH_POPC) {
    e = gemm_subword(a, w) ? launch_partials_popc_sub(a, w, D, static_cast<cudaStream_t>(stream))
                           : launch_partials_popc(a, w, D, static_cast<cudaStream_t>(stream));
  } else if (path == HBMM_PATH_B1MMA) {
    if (!gemm_b1_supported(a, w)) return HBMM_ERR_UNSUPPORTED;
    e = launch_partials_b1(a, w, D, static_cast<cudaStream_t>(stream));
  } else {
    return HBMM_ERR_UNSUPPORTED;
  }
  return e == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
}

hbmm_status hbmm_conv_workspace_bytes(const hbmm_conv_geom* g, int32_t beta_a, int32_t a_scale_dtype,
                                      const hbmm_operand* W, size_t* bytes) {
  ConvGeom cg;
  hbmm_status st = check_geom(g, &cg);
  if (st != HBMM_OK) return st;
  if (!bytes || !W || beta_a < 1 || !valid_dtype(a_scale_dtype)) return HBMM_ERR_INVALID_ARG;
  const int64_t K = static_cast<int64_t>(cg.C) * cg.kh * cg.kw;
  if (beta_a >= 2 && !beta_supported(K, beta_a)) return HBMM_ERR_UNSUPPORTED;
  if (check_packed(W, false) != HBMM_OK) return check_packed(W, false);
  *bytes = conv_layout(cg, beta_a, a_scale_dtype, W).total;
  return HBMM_OK;
}

hbmm_status hbmm_conv_im2col(const void* x, int32_t x_dtype, const hbmm_conv_geom* g, int32_t beta_a,
                             int32_t a_scale_dtype, const hbmm_operand* W, float* C_out, int64_t ldc,
                             void* workspace, size_t workspace_bytes, void* stream) {
  return hbmm_conv_im2col_ex(x, x_dtype, g, beta_a, a_scale_dtype, W, C_out, ldc, workspace, workspace_bytes, 0u, stream);
}

hbmm_status hbmm_conv_im2col_ex(const void* x, int32_t x_dtype, const hbmm_conv_geom* g, int32_t beta_a,
                                int32_t a_scale_dtype, const hbmm_operand* W, float* C_out, int64_t ldc,
                                void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
  return conv_checked(x, x_dtype, g, beta_a, a_scale_dtype, W, C_out, ldc, nullptr, workspace, workspace_bytes, flags, stream);
}

hbmm_status hbmm_conv_im2col_fused(const void* x, int32_t x_dtype, const hbmm_conv_geom* g, int32_t beta_a,
                                   int32_t a_scale_dtype, const hbmm_operand* W, const hbmm_epilogue* ep,
                                   void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
  if (!ep || (flags & HBMM_CONV_PACK_ONLY)) return HBMM_ERR_INVALID_ARG;
  return conv_checked(x, x_dtype, g, beta_a, a_scale_dtype, W, nullptr, 0, ep, workspace, workspace_bytes, flags, stream);
}

}  // extern "C"

namespace {

hbmm_status conv_checked(const void* x, int32_t x_dtype, const hbmm_conv_geom* g, int32_t beta_a, int32_t a_scale_dtype,
                         const hbmm_operand* W, float* C_out, int64_t ldc, const hbmm_epilogue* ep, void* workspace,
                         size_t workspace_bytes, uint32_t flags, void* stream) {
  if (flags & ~static_cast<uint32_t>(HBMM_CONV_WEIGHTS_PREPARED | HBMM_CONV_PACK_ONLY | HBMM_CONV_INPUT_NHWC)) return HBMM_ERR_INVALID_ARG;
  const bool pack_only = (flags & HBMM_CONV_PACK_ONLY) != 0;
  const bool input_nhwc = (flags & HBMM_CONV_INPUT_NHWC) != 0;
  if (pack_only && beta_a < 2) return HBMM_ERR_INVALID_ARG;     // only a packed activation operand can be left behind
  // honoured on the two tensor-copy paths below; every other path expands the weights again (still correct)
  const bool w_prepared = (flags & HBMM_CONV_WEIGHTS_PREPARED) != 0;
  ConvGeom cg;
  hbmm_status st = check_geom(g, &cg);
  if (st != HBMM_OK) return st;
  if (!x || !W || beta_a < 1 || !valid_dtype(x_dtype) || !valid_dtype(a_scale_dtype)) return HBMM_ERR_INVALID_ARG;
  if ((st = check_packed(W)) != HBMM_OK) return st;
  const ConvLayout L = conv_layout(cg, beta_a, a_scale_dtype, W);
  if (W->K != L.K) return HBMM_ERR_INVALID_ARG;
  if (beta_a >= 2 && !beta_supported(L.K, beta_a)) return HBMM_ERR_UNSUPPORTED;
  EpiArgs epi = plain_epilogue();
  if (ep) {
    if ((st = make_epilogue(ep, L.M, W->rows, &epi)) != HBMM_OK) return st;
    if (epi.mode == kEpiPacked && !gemm_fold_next_supported(W->rows, epi.nx_beta)) return HBMM_ERR_UNSUPPORTED;
  } else if (!pack_only && (st = check_c(C_out, ldc, W->rows)) != HBMM_OK) {
    return st;
  }
  if (input_nhwc) {
    // an NHWC bf16 image (what a dense-output epilogue of the layer before wrote): the dense-activation
    // tensor-core path reads it as it is
    if (beta_a != 1 || x_dtype != HBMM_BF16) return HBMM_ERR_INVALID_ARG;
    if (!L.implicit || L.Cp != cg.C) return HBMM_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(x) % 16 != 0) return HBMM_ERR_ALIGNMENT;
  }
  if (!workspace || workspace_bytes < L.total) return HBMM_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return HBMM_ERR_ALIGNMENT;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  hbmm_operand A{};
  A.rows = L.M; A.K = L.K; A.beta = beta_a; A.scale_dtype = a_scale_dtype;
  if (beta_a == 1 && L.implicit) {
    return launch_hbwn_umma_conv(x, x_dtype == HBMM_BF16, workspace, L.Cp, cg, view_of(W), C_out, ldc,
                                 static_cast<char*>(workspace) + L.operand_bytes, s, w_prepared, ep ? &epi : nullptr,
                                 input_nhwc) == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
  }
  if (beta_a == 1) {
    if (ep) return HBMM_ERR_UNSUPPORTED;       // the epilogue chain needs the implicit tensor-core path (whole 64-channel blocks)
    if (launch_im2col_bf16(x, x_dtype == HBMM_BF16, cg, workspace, L.ld_dense, s) != cudaSuccess) return HBMM_ERR_CUDA;
    A.dense = workspace; A.ld_dense = L.ld_dense; A.dense_dtype = HBMM_BF16;
  } else {
    A.bits = static_cast<uint32_t*>(workspace);
    A.scales = static_cast<char*>(workspace) + L.bits_bytes;
    A.ld_words = L.ld_words; A.ld_scales = L.ld_scales;
    hbmm_operand Aseg = A;
    if (!segments_compatible(&Aseg, W)) return HBMM_ERR_UNSUPPORTED;
    // When the tensor-core contraction will run and the tensor-copy front end takes this input, the
    // front end's launch also expands the weight operand (a few extra CTAs) and the contraction skips it.
    const PackedView av = view_of(&A), wv = view_of(W);
    void* gemm_ws = static_cast<char*>(workspace) + L.operand_bytes;
    if (ep) {
      // the epilogue chain lives in the folded-scale kernel: activation groups of whole words, K in whole words
      const bool a_subword = beta_a < 32 && beta_a < L.K;
      if (!gemm_fold_supported(av, wv) || a_subword || L.gemm_bytes < fold_workspace(av, wv)) return HBMM_ERR_UNSUPPORTED;
    }
    if ((ep || prefer_fold(av, wv)) && L.gemm_bytes > 0 && L.gemm_bytes >= fold_workspace(av, wv) &&
        im2col_quantize_tma_supported(x, x_dtype == HBMM_BF16, cg, beta_a)) {
      UmmaPrepJob job{};
      gemm_fold_prep_job(av, wv, gemm_ws, &job);
      if (job.n_stages * job.tiles_n <= 4096) {
        if (launch_im2col_quantize_tma(x, cg, beta_a, A.bits, A.ld_words, A.scales, A.ld_scales, a_scale_dtype == HBMM_BF16, s,
                                       w_prepared ? nullptr : &job) != cudaSuccess)
          return HBMM_ERR_CUDA;
        if (pack_only) return HBMM_OK;
        return launch_gemm_fold(av, wv, C_out, ldc, gemm_ws, s, true, ep ? &epi : nullptr) == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
      }
    }
    if (launch_im2col_quantize(x, x_dtype == HBMM_BF16, cg, beta_a, A.bits, A.ld_words, A.scales, A.ld_scales,
                               a_scale_dtype == HBMM_BF16, s) != cudaSuccess)
      return HBMM_ERR_CUDA;
    if (pack_only) return HBMM_OK;
    if (ep)
      return launch_gemm_fold(av, wv, nullptr, 0, gemm_ws, s, w_prepared, &epi) == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
  }
  return gemm_checked(&A, W, C_out, ldc, HBMM_PATH_AUTO, static_cast<char*>(workspace) + L.operand_bytes, L.gemm_bytes, s);
}

}  // namespace

extern "C" {

hbmm_status hbmm_last_device_error(int32_t* code) {
  int c = 0;
  int c2 = 0;
  if (gemm_umma_health(kHealthRead, &c) != cudaSuccess || hbwn_umma_health(kHealthRead, &c2) != cudaSuccess) return HBMM_ERR_CUDA;
  if (c == 0 && c2 != 0) c = 100 + c2;    // codes of the HBWN kernel are reported as 100 + code
  int c3 = 0;
  if (im2col_tma_health(kHealthRead, &c3) != cudaSuccess) return HBMM_ERR_CUDA;
  if (c == 0 && c3 != 0) c = 200 + c3;    // the packed front end: 201..204
  int c4 = 0;
  if (gemm_fold_health(kHealthRead, &c4) != cudaSuccess) return HBMM_ERR_CUDA;
  if (c == 0 && c4 != 0) c = 300 + c4;    // the folded-scale HBMM kernel: 301..309
  if (code) *code = c;
  return c == 0 ? HBMM_OK : HBMM_ERR_TIMEOUT;
}

hbmm_status hbmm_clear_device_error(void) {
  int unused = 0;
  if (gemm_umma_health(kHealthClear, &unused) != cudaSuccess || hbwn_umma_health(kHealthClear, &unused) != cudaSuccess ||
      im2col_tma_health(kHealthClear, &unused) != cudaSuccess || gemm_fold_health(kHealthClear, &unused) != cudaSuccess)
    return HBMM_ERR_CUDA;
  return HBMM_OK;
}

hbmm_status hbmm_debug_set_wait_limit(uint32_t polls) {
  int v = static_cast<int>(polls);
  if (polls > 0x7FFFFFFFu) return HBMM_ERR_INVALID_ARG;
  if (gemm_umma_health(kHealthSetSpinLimit, &v) != cudaSuccess || hbwn_umma_health(kHealthSetSpinLimit, &v) != cudaSuccess ||
      im2col_tma_health(kHealthSetSpinLimit, &v) != cudaSuccess || gemm_fold_health(kHealthSetSpinLimit, &v) != cudaSuccess)
    return HBMM_ERR_CUDA;
  return HBMM_OK;
}

hbmm_status hbmm_debug_expire_wait(void* stream) {
  return launch_wait_expiry_selftest(static_cast<cudaStream_t>(stream)) == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
}

hbmm_status hbmm_bench_alu_rate(int32_t kind, int32_t blocks, int32_t iters, uint32_t* sink, int64_t* ops, void* stream) {
  if (kind < 0 || kind > 2 || blocks <= 0 || iters <= 0 || !sink) return HBMM_ERR_INVALID_ARG;
  return launch_alu_rate(kind, blocks, iters, sink, ops, static_cast<cudaStream_t>(stream)) == cudaSuccess ? HBMM_OK : HBMM_ERR_CUDA;
}

const char* hbmm_status_string(int32_t status) {
  switch (status) {
    case HBMM_OK: return "ok";
    case HBMM_ERR_INVALID_ARG: return "invalid argument";
    case HBMM_ERR_UNSUPPORTED: return "unsupported beta / dtype / path combination";
    case HBMM_ERR_ALIGNMENT: return "pointer or leading dimension violates the required alignment";
    case HBMM_ERR_WORKSPACE: return "workspace missing or too small";
    case HBMM_ERR_CUDA: return "CUDA runtime error at launch";
    case HBMM_ERR_TIMEOUT: return "bounded device-side wait expired";
    default: return "unknown status";
  }
}

int32_t hbmm_version(void) { return kVersion; }

}  // extern "C"
