// C ABI of libmxp: argument validation and dispatch.  No kernel lives here.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <vector>

#include <atomic>

#include "common.cuh"

namespace mxp {
namespace {
std::atomic<int> g_override[MXP_KNOB_COUNT_];
}
int override_get(int knob) { return knob >= 0 && knob < MXP_KNOB_COUNT_ ? g_override[knob].load(std::memory_order_relaxed) : 0; }
}  // namespace mxp

namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// modes every entry point takes: the 4-bit ones
bool valid_mode(int m)
{
    return m == MXP_MODE_MXFP4 || m == MXP_MODE_MXFP4_PLUS || m == MXP_MODE_MXFP4_PP;
}
// 6- and 8-bit element modes: quantize and decode only
bool wide_mode(int m) { return m >= MXP_MODE_MXFP6 && m <= MXP_MODE_MXFP8_PLUS; }
bool plus_mode(int m)
{
    return m == MXP_MODE_MXFP4_PLUS || m == MXP_MODE_MXFP4_PP || m == MXP_MODE_MXFP6_PLUS ||
           m == MXP_MODE_MXFP8_PLUS;
}
bool valid_dtype(int d) { return d == MXP_F32 || d == MXP_BF16; }

// Checks an operand descriptor (host struct, device planes).  `six_ok`: the caller also takes
// MXFP6 / MXFP6+ operands (the packed x packed GEMM does).
bool valid_packed(const mxp_packed* p, bool six_ok = false)
{
    if (p == nullptr) return false;
    const bool six = p->mode == MXP_MODE_MXFP6 || p->mode == MXP_MODE_MXFP6_PLUS ||
                     p->mode == MXP_MODE_MXFP8 || p->mode == MXP_MODE_MXFP8_PLUS;  // (and the 8-bit modes)
    if (!valid_mode(p->mode) && !(six_ok && six)) return false;
    if (p->rows < 0 || p->cols < 0 || p->cols % 32 != 0) return false;
    if (p->rows == 0 || p->cols == 0) return true;
    if (p->nibbles == nullptr || p->scales == nullptr) return false;
    if (!aligned(p->nibbles, 16)) return false;
    if (plus_mode(p->mode) && p->bm_index == nullptr) return false;
    return true;
}

}  // namespace

extern "C" {

const char* mxp_status_string(mxp_status s)
{
    switch (s) {
        case MXP_OK: return "ok";
        case MXP_ERR_INVALID_ARG: return "invalid argument";
        case MXP_ERR_UNSUPPORTED: return "unsupported configuration";
        case MXP_ERR_WORKSPACE: return "workspace missing or too small";
        case MXP_ERR_CUDA: return "CUDA error";
        case MXP_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

const char* mxp_version(void) { return "mxp 0.2 sm_100a"; }

mxp_status mxp_debug_override(int knob, int value)
{
    if (knob < 0 || knob >= MXP_KNOB_COUNT_ || value < 0 || value > 2) return MXP_ERR_INVALID_ARG;
    mxp::g_override[knob].store(value, std::memory_order_relaxed);
    return MXP_OK;
}

mxp_status mxp_quantize(const void* src, mxp_dtype src_dt, int64_t rows, int64_t cols,
                        int64_t ld_src, mxp_mode mode, uint8_t* nibbles, uint8_t* scales,
                        uint8_t* bm_index, void* cuda_stream)
{
    if ((!valid_mode(mode) && !wide_mode(mode)) || !valid_dtype(src_dt)) return MXP_ERR_INVALID_ARG;
    if (rows < 0 || cols < 0 || cols % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return MXP_OK;
    if (src == nullptr || nibbles == nullptr || scales == nullptr) return MXP_ERR_INVALID_ARG;
    if (plus_mode(mode) && bm_index == nullptr) return MXP_ERR_INVALID_ARG;
    if (ld_src < cols || ld_src % 8 != 0) return MXP_ERR_INVALID_ARG;
    if (!aligned(src, 16) || !aligned(nibbles, 16)) return MXP_ERR_INVALID_ARG;
    if (rows * (cols / 32) / 256 + 1 > 0x7FFFFFFFll) return MXP_ERR_UNSUPPORTED;
    if (wide_mode(mode))
        return mxp::launch_quantize_wide(src, src_dt, rows, cols, ld_src, mode, nibbles, scales,
                                         bm_index, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
                   ? MXP_OK
                   : MXP_ERR_CUDA;
    cudaError_t e = mxp::launch_quantize(src, src_dt, rows, cols, ld_src, mode, nibbles, scales,
                                         bm_index, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

mxp_status mxp_quantize_reordered(const void* src, mxp_dtype src_dt, int64_t rows, int64_t cols,
                                  int64_t ld_src, const int32_t* order, mxp_mode mode,
                                  uint8_t* nibbles, uint8_t* scales, uint8_t* bm_index,
                                  void* cuda_stream)
{
    if ((!valid_mode(mode) && !wide_mode(mode)) || !valid_dtype(src_dt)) return MXP_ERR_INVALID_ARG;
    if (rows < 0 || cols < 0 || cols % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return MXP_OK;
    if (src == nullptr || nibbles == nullptr || scales == nullptr || order == nullptr)
        return MXP_ERR_INVALID_ARG;
    if (plus_mode(mode) && bm_index == nullptr) return MXP_ERR_INVALID_ARG;
    if (ld_src < cols) return MXP_ERR_INVALID_ARG;
    if (!aligned(src, src_dt == MXP_BF16 ? 2 : 4) || !aligned(nibbles, 16) || !aligned(order, 16))
        return MXP_ERR_INVALID_ARG;
    if (wide_mode(mode) || cols > 0x7FFFFFFFll) return MXP_ERR_UNSUPPORTED;
    if (rows * (cols / 32) / 256 + 1 > 0x7FFFFFFFll) return MXP_ERR_UNSUPPORTED;
    cudaError_t e = mxp::launch_quantize_reordered(src, src_dt, rows, cols, ld_src, order, mode,
                                                   nibbles, scales, bm_index,
                                                   static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

mxp_status mxp_nvfp4_quantize(const void* src, mxp_dtype src_dt, int64_t rows, int64_t cols,
                              int64_t ld_src, float tensor_scale, int plus, uint8_t* nibbles,
                              uint8_t* scales, uint8_t* bm_index, void* cuda_stream)
{
    if (!valid_dtype(src_dt) || rows < 0 || cols < 0 || cols % 32 != 0) return MXP_ERR_INVALID_ARG;
    // 2^-100 .. 2^100: keeps value(byte) * ts and its reciprocal normal binary32 numbers
    if (!(tensor_scale >= 7.8886090522101181e-31f) || !(tensor_scale <= 1.2676506002282294e30f))
        return MXP_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return MXP_OK;
    if (src == nullptr || nibbles == nullptr || scales == nullptr) return MXP_ERR_INVALID_ARG;
    if (plus && bm_index == nullptr) return MXP_ERR_INVALID_ARG;
    if (ld_src < cols || ld_src % 8 != 0) return MXP_ERR_INVALID_ARG;
    if (!aligned(src, 16) || !aligned(nibbles, 16) || !aligned(scales, 2)) return MXP_ERR_INVALID_ARG;
    if (rows * (cols / 32) / 256 + 1 > 0x7FFFFFFFll) return MXP_ERR_UNSUPPORTED;
    cudaError_t e = mxp::launch_nvfp4_quantize(src, src_dt, rows, cols, ld_src, tensor_scale,
                                               plus != 0, nibbles, scales, bm_index,
                                               static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

mxp_status mxp_nvfp4_dequantize(const uint8_t* nibbles, const uint8_t* scales,
                                const uint8_t* bm_index, int64_t rows, int64_t cols,
                                float tensor_scale, int plus, void* dst, mxp_dtype dst_dt,
                                int64_t ld_dst, void* cuda_stream)
{
    if (!valid_dtype(dst_dt) || rows < 0 || cols < 0 || cols % 32 != 0) return MXP_ERR_INVALID_ARG;
    // 2^-100 .. 2^100: keeps value(byte) * ts and its reciprocal normal binary32 numbers
    if (!(tensor_scale >= 7.8886090522101181e-31f) || !(tensor_scale <= 1.2676506002282294e30f))
        return MXP_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return MXP_OK;
    if (nibbles == nullptr || scales == nullptr || dst == nullptr) return MXP_ERR_INVALID_ARG;
    if (plus && bm_index == nullptr) return MXP_ERR_INVALID_ARG;
    if (!aligned(nibbles, 4) || !aligned(dst, 16) || ld_dst < cols || ld_dst % 8 != 0)
        return MXP_ERR_INVALID_ARG;
    if (rows * (cols / 8) / 256 + 1 > 0x7FFFFFFFll) return MXP_ERR_UNSUPPORTED;
    cudaError_t e = mxp::launch_nvfp4_dequantize(nibbles, scales, bm_index, rows, cols, tensor_scale,
                                                 plus != 0, dst, dst_dt, ld_dst,
                                                 static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

mxp_status mxp_channel_order(const int64_t* outlier_count, int64_t cols, int32_t* order)
{
    if (outlier_count == nullptr || order == nullptr) return MXP_ERR_INVALID_ARG;
    if (cols <= 0 || cols % 32 != 0 || cols > 0x7FFFFFFFll) return MXP_ERR_INVALID_ARG;
    // channels by outlier count, most first; equal counts keep channel order
    std::vector<int32_t> by_count((size_t)cols);
    for (int64_t c = 0; c < cols; ++c) by_count[(size_t)c] = (int32_t)c;
    std::stable_sort(by_count.begin(), by_count.end(), [&](int32_t a, int32_t b) {
        return outlier_count[a] > outlier_count[b];
    });
    const int64_t nblk = cols / 32;
    // the nblk channels with the most outliers: one per block, at the block's first position
    for (int64_t j = 0; j < nblk; ++j) order[32 * j] = by_count[(size_t)j];
    // the rest fills the other positions front to back: first the half with fewer outliers,
    // then the half with more, each from its most-outlier channel down
    const int64_t rest = cols - nblk, upper = rest / 2;
    int64_t pos = 0;
    auto place = [&](int64_t from, int64_t to) {
        for (int64_t i = from; i < to; ++i) {
            if (pos % 32 == 0) ++pos;
            order[pos++] = by_count[(size_t)(nblk + i)];
        }
    };
    place(upper, rest);
    place(0, upper);
    return MXP_OK;
}

mxp_status mxp_dequantize(const mxp_packed* p, void* dst, mxp_dtype dst_dt, int64_t ld_dst,
                          void* cuda_stream)
{
    if (p != nullptr && wide_mode(p->mode)) {
        if (p->rows < 0 || p->cols < 0 || p->cols % 32 != 0 || !valid_dtype(dst_dt)) return MXP_ERR_INVALID_ARG;
        if (p->rows == 0 || p->cols == 0) return MXP_OK;
        if (p->nibbles == nullptr || p->scales == nullptr || !aligned(p->nibbles, 16)) return MXP_ERR_INVALID_ARG;
        if (plus_mode(p->mode) && p->bm_index == nullptr) return MXP_ERR_INVALID_ARG;
        if (dst == nullptr || !aligned(dst, 16) || ld_dst < p->cols || ld_dst % 8 != 0) return MXP_ERR_INVALID_ARG;
        if (p->rows * (p->cols / 32) / 256 + 1 > 0x7FFFFFFFll) return MXP_ERR_UNSUPPORTED;
        return mxp::launch_dequantize_wide(*p, dst, dst_dt, ld_dst, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
                   ? MXP_OK
                   : MXP_ERR_CUDA;
    }
    if (!valid_packed(p) || !valid_dtype(dst_dt)) return MXP_ERR_INVALID_ARG;
    if (p->rows == 0 || p->cols == 0) return MXP_OK;
    if (dst == nullptr || !aligned(dst, 16)) return MXP_ERR_INVALID_ARG;
    if (ld_dst < p->cols || ld_dst % 8 != 0) return MXP_ERR_INVALID_ARG;
    if (p->rows * p->cols / 8 / 256 + 1 > 0x7FFFFFFFll) return MXP_ERR_UNSUPPORTED;
    cudaError_t e =
        mxp::launch_dequantize(*p, dst, dst_dt, ld_dst, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

size_t mxp_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int a_dense, mxp_mode a_mode,
                                mxp_mode b_mode)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    if (a_dense) {
        // more than 64 activation rows: the tensor-core kernel, which needs room for both
        // operands' prepared forms; decode shapes need none
        if ((M > 64 && N >= 128) || wide_mode(b_mode)) {
            const size_t fast = mxp::stream_dense_workspace_bytes(M, N, K, b_mode);
            if (fast != 0 || wide_mode(b_mode)) return fast;
        }
        return mxp::skinny_workspace_bytes(M, N, K);
    }
    return mxp::tc_workspace_bytes(M, N, K, a_mode, b_mode);
}

size_t mxp_gemm_min_workspace_bytes(int64_t M, int64_t N, int64_t K, int a_dense, mxp_mode,
                                    mxp_mode)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    if (a_dense) return mxp::skinny_workspace_bytes(M, N, K);
    return mxp::tc_compact_workspace_bytes();
}

mxp_status mxp_gemm(int64_t M, int64_t N, int64_t K, const void* A_dense_bf16, int64_t lda,
                    const mxp_packed* A_packed, const mxp_packed* B_packed, void* D,
                    mxp_dtype d_dt, int64_t ldd, void* workspace, size_t workspace_bytes,
                    void* cuda_stream)
{
    if (M < 0 || N < 0 || K < 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (!valid_dtype(d_dt)) return MXP_ERR_INVALID_ARG;
    if ((A_dense_bf16 == nullptr) == (A_packed == nullptr)) return MXP_ERR_INVALID_ARG;
    if (!valid_packed(B_packed, true)) return MXP_ERR_INVALID_ARG;
    if (B_packed->rows != N || B_packed->cols != K) return MXP_ERR_INVALID_ARG;
    if (A_packed != nullptr) {
        if (!valid_packed(A_packed, true)) return MXP_ERR_INVALID_ARG;
        if (A_packed->rows != M || A_packed->cols != K) return MXP_ERR_INVALID_ARG;
    } else {
        if (lda < K || lda % 8 != 0 || !aligned(A_dense_bf16, 16)) return MXP_ERR_INVALID_ARG;
    }
    if (M == 0 || N == 0) return MXP_OK;
    if (D == nullptr || ldd < N) return MXP_ERR_INVALID_ARG;
    if (!aligned(D, d_dt == MXP_BF16 ? 2 : 4)) return MXP_ERR_INVALID_ARG;
    if (K == 0) return MXP_ERR_UNSUPPORTED;  // an empty sum; callers zero D themselves
    const size_t need = mxp_gemm_min_workspace_bytes(M, N, K, A_dense_bf16 != nullptr,
                                                     A_packed ? A_packed->mode : MXP_MODE_MXFP4,
                                                     B_packed->mode);
    if (need > 0) {
        if (workspace == nullptr || workspace_bytes < need) return MXP_ERR_WORKSPACE;
        if (!aligned(workspace, 256)) return MXP_ERR_INVALID_ARG;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (A_dense_bf16 != nullptr) {
        // the wider weight formats have the tensor-core kernel only, at any M and N
        const bool wide_b = wide_mode(B_packed->mode);
        if (wide_b && K % 128 != 0) return MXP_ERR_UNSUPPORTED;
        if ((wide_b || (M > 64 && N >= 128)) && workspace != nullptr && aligned(workspace, 256) &&
            aligned(B_packed->scales, 4) && mxp::override_get(MXP_KNOB_WEIGHT_ONLY_KERNEL) == 0 &&
            (B_packed->mode != MXP_MODE_MXFP4_PP || aligned(B_packed->bm_index, 4))) {
            const size_t fast = mxp::stream_dense_workspace_bytes(M, N, K, B_packed->mode);
            if (fast != 0 && workspace_bytes >= fast) {
                mxp_packed none = {};
                none.mode = MXP_MODE_MXFP4;
                return mxp::launch_gemm_tc_stream(M, N, K, none, *B_packed, nullptr, D, d_dt, ldd,
                                                  workspace, workspace_bytes, stream, false,
                                                  A_dense_bf16, lda);
            }
        }
        if (wide_b) return MXP_ERR_WORKSPACE;  // needs mxp_gemm_workspace_bytes(..., a_dense = 1, ...)
        cudaError_t e = mxp::launch_gemm_weight_only(M, N, K, A_dense_bf16, lda, *B_packed, D,
                                                     d_dt, ldd, workspace, workspace_bytes, stream);
        if (e == cudaErrorNotSupported) return MXP_ERR_UNSUPPORTED;
        return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
    }
    return mxp::launch_gemm_tc(M, N, K, *A_packed, *B_packed, D, d_dt, ldd, workspace,
                               workspace_bytes, stream);
}

mxp_status mxp_gemm_decode_chained(int64_t M, int64_t N, int64_t K, const void* A_dense_bf16,
                                   int64_t lda, const mxp_packed* B_packed, void* D,
                                   mxp_dtype d_dt, int64_t ldd, void* status_block,
                                   void* cuda_stream)
{
    if (M < 0 || N < 0 || K < 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (!valid_dtype(d_dt) || A_dense_bf16 == nullptr) return MXP_ERR_INVALID_ARG;
    if (!valid_packed(B_packed, false)) return MXP_ERR_INVALID_ARG;
    if (B_packed->rows != N || B_packed->cols != K) return MXP_ERR_INVALID_ARG;
    if (lda < K || lda % 8 != 0 || !aligned(A_dense_bf16, 16)) return MXP_ERR_INVALID_ARG;
    if (status_block != nullptr && !aligned(status_block, 16)) return MXP_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return MXP_OK;
    if (D == nullptr || ldd < N) return MXP_ERR_INVALID_ARG;
    if (!aligned(D, d_dt == MXP_BF16 ? 2 : 4)) return MXP_ERR_INVALID_ARG;
    if (K == 0 || M > 64) return MXP_ERR_UNSUPPORTED;
    if (!mxp::wo_stream_supported(M, N, K, A_dense_bf16, lda, *B_packed)) return MXP_ERR_UNSUPPORTED;
    const cudaError_t e = mxp::launch_gemm_wo_stream(M, N, K, A_dense_bf16, lda, *B_packed, D, d_dt,
                                                     ldd, status_block,
                                                     static_cast<cudaStream_t>(cuda_stream), true);
    if (e == cudaErrorNotSupported) return MXP_ERR_UNSUPPORTED;
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

size_t mxp_gemm_decode_prepack_bytes(int64_t N, int64_t K, mxp_mode b_mode)
{
    return mxp::decode_prepack_bytes(N, K, b_mode);
}

size_t mxp_gemm_decode_workspace_bytes(int64_t M, int64_t K)
{
    return mxp::decode_workspace_bytes(M, K);
}

mxp_status mxp_gemm_decode_prepack(const mxp_packed* B_packed, void* out, size_t out_bytes,
                                   void* cuda_stream)
{
    if (!valid_packed(B_packed, false)) return MXP_ERR_INVALID_ARG;
    if (B_packed->rows == 0 || B_packed->cols == 0) return MXP_ERR_UNSUPPORTED;
    if (B_packed->mode != MXP_MODE_MXFP4 && B_packed->mode != MXP_MODE_MXFP4_PLUS)
        return MXP_ERR_UNSUPPORTED;
    return mxp::decode_prepack(*B_packed, out, out_bytes, static_cast<cudaStream_t>(cuda_stream));
}

mxp_status mxp_gemm_decode_prepacked(int64_t M, int64_t N, int64_t K, const void* A_dense_bf16,
                                     int64_t lda, mxp_mode b_mode, const void* B_prepacked,
                                     size_t B_prepacked_bytes, void* D, mxp_dtype d_dt, int64_t ldd,
                                     void* workspace, size_t workspace_bytes, int chained,
                                     void* cuda_stream)
{
    return mxp_gemm_decode_prepacked_next(M, N, K, A_dense_bf16, lda, b_mode, B_prepacked, B_prepacked_bytes,
                                          D, d_dt, ldd, workspace, workspace_bytes, chained, nullptr, 0,
                                          cuda_stream);
}

mxp_status mxp_gemm_decode_prepacked_next(int64_t M, int64_t N, int64_t K, const void* A_dense_bf16,
                                          int64_t lda, mxp_mode b_mode, const void* B_prepacked,
                                          size_t B_prepacked_bytes, void* D, mxp_dtype d_dt, int64_t ldd,
                                          void* workspace, size_t workspace_bytes, int chained,
                                          const void* next_B_prepacked, size_t next_B_prepacked_bytes,
                                          void* cuda_stream)
{
    if ((next_B_prepacked == nullptr) != (next_B_prepacked_bytes == 0)) return MXP_ERR_INVALID_ARG;
    if (next_B_prepacked != nullptr && !aligned(next_B_prepacked, 256)) return MXP_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || K < 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (!valid_dtype(d_dt) || !valid_mode(b_mode)) return MXP_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return MXP_OK;
    if (A_dense_bf16 == nullptr || B_prepacked == nullptr || D == nullptr) return MXP_ERR_INVALID_ARG;
    if (lda < K || lda % 8 != 0 || !aligned(A_dense_bf16, 16) || ldd < N) return MXP_ERR_INVALID_ARG;
    if (!aligned(D, d_dt == MXP_BF16 ? 2 : 4) || !aligned(B_prepacked, 256)) return MXP_ERR_INVALID_ARG;
    if (workspace != nullptr && !aligned(workspace, 256)) return MXP_ERR_INVALID_ARG;
    return mxp::launch_gemm_decode_tc(M, N, K, A_dense_bf16, lda, b_mode, B_prepacked,
                                      B_prepacked_bytes, D, d_dt, ldd, workspace, workspace_bytes,
                                      chained != 0, next_B_prepacked, next_B_prepacked_bytes,
                                      static_cast<cudaStream_t>(cuda_stream));
}

size_t mxp_gemm_prepack_bytes(int64_t rows, int64_t K, int form)
{
    return mxp::stream_prepack_bytes(rows, K, form);
}

int mxp_gemm_prepack_form(mxp_mode a_mode, mxp_mode b_mode) { return mxp::stream_b_form(a_mode, b_mode); }

mxp_status mxp_gemm_prepack(const mxp_packed* P, int form, void* out, size_t out_bytes,
                            void* cuda_stream)
{
    if (!valid_packed(P, true)) return MXP_ERR_INVALID_ARG;
    if (form < MXP_PREPACK_PLAIN || form > MXP_PREPACK_WIDE8_X3) return MXP_ERR_INVALID_ARG;
    if (P->rows == 0 || P->cols == 0) return MXP_OK;
    if (P->mode != MXP_MODE_MXFP4 && form == MXP_PREPACK_PLAIN) return MXP_ERR_INVALID_ARG;
    if (P->mode != MXP_MODE_MXFP4_PLUS && form == MXP_PREPACK_SPLIT) return MXP_ERR_INVALID_ARG;
    return mxp::stream_prepack(*P, form, out, out_bytes, static_cast<cudaStream_t>(cuda_stream));
}

mxp_status mxp_gemm_prepacked(int64_t M, int64_t N, int64_t K, const mxp_packed* A_packed,
                              const mxp_packed* B_packed, const void* B_prepacked,
                              size_t B_prepacked_bytes, void* D, mxp_dtype d_dt, int64_t ldd,
                              void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (M < 0 || N < 0 || K < 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (!valid_dtype(d_dt)) return MXP_ERR_INVALID_ARG;
    if (!valid_packed(A_packed, true) || !valid_packed(B_packed, true)) return MXP_ERR_INVALID_ARG;
    if (A_packed->rows != M || A_packed->cols != K || B_packed->rows != N || B_packed->cols != K)
        return MXP_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return MXP_OK;
    if (K == 0) return MXP_ERR_UNSUPPORTED;
    if (B_prepacked == nullptr || D == nullptr || ldd < N) return MXP_ERR_INVALID_ARG;
    if (!aligned(D, d_dt == MXP_BF16 ? 2 : 4)) return MXP_ERR_INVALID_ARG;
    if (!aligned(A_packed->scales, 4) || !aligned(B_packed->scales, 4)) return MXP_ERR_INVALID_ARG;
    if (mxp::stream_workspace_bytes(M, N, K, A_packed->mode, B_packed->mode) == 0)
        return MXP_ERR_UNSUPPORTED;
    // the copy must be the one this pairing of modes reads, made for this shape: its size says so
    const int form = mxp::stream_b_form(A_packed->mode, B_packed->mode);
    const size_t want = mxp::stream_prepack_bytes(N, K, form);
    if (want == 0) return MXP_ERR_UNSUPPORTED;
    if (B_prepacked_bytes != want || !aligned(B_prepacked, 256)) return MXP_ERR_INVALID_ARG;
    if ((form == MXP_PREPACK_PLAIN || form == MXP_PREPACK_SPLIT) &&
        mxp::stream_sparse_workspace_bytes(M, N, K, A_packed->mode, B_packed->mode, true) != 0)
        return mxp::launch_gemm_tc_sparse(M, N, K, *A_packed, *B_packed, B_prepacked, D, d_dt, ldd,
                                          workspace, workspace_bytes,
                                          static_cast<cudaStream_t>(cuda_stream));
    return mxp::launch_gemm_tc_stream(M, N, K, *A_packed, *B_packed, B_prepacked, D, d_dt, ldd,
                                      workspace, workspace_bytes,
                                      static_cast<cudaStream_t>(cuda_stream));
}

size_t mxp_gemm_dense_prepacked_workspace_bytes(int64_t M, int64_t K)
{
    return mxp::stream_dense_prepacked_workspace_bytes(M, K);
}

mxp_status mxp_gemm_dense_prepacked(int64_t M, int64_t N, int64_t K, const void* A_dense_bf16,
                                    int64_t lda, const mxp_packed* B_packed,
                                    const void* B_prepacked, size_t B_prepacked_bytes, void* D,
                                    mxp_dtype d_dt, int64_t ldd, void* workspace,
                                    size_t workspace_bytes, void* cuda_stream)
{
    if (M < 0 || N < 0 || K < 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (!valid_dtype(d_dt) || A_dense_bf16 == nullptr) return MXP_ERR_INVALID_ARG;
    if (!valid_packed(B_packed, false)) return MXP_ERR_INVALID_ARG;
    if (B_packed->rows != N || B_packed->cols != K) return MXP_ERR_INVALID_ARG;
    if (lda < K || lda % 8 != 0 || !aligned(A_dense_bf16, 16)) return MXP_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return MXP_OK;
    if (B_prepacked == nullptr || D == nullptr || ldd < N) return MXP_ERR_INVALID_ARG;
    if (!aligned(D, d_dt == MXP_BF16 ? 2 : 4)) return MXP_ERR_INVALID_ARG;
    const size_t need = mxp::stream_dense_prepacked_workspace_bytes(M, K);
    const int wform = mxp::stream_wide_form(B_packed->mode);
    if (need == 0 || mxp::stream_prepack_bytes(N, K, wform) == 0) return MXP_ERR_UNSUPPORTED;
    if (B_prepacked_bytes != mxp::stream_prepack_bytes(N, K, wform) || !aligned(B_prepacked, 256))
        return MXP_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < need) return MXP_ERR_WORKSPACE;
    mxp_packed none = {};
    none.mode = MXP_MODE_MXFP4;
    return mxp::launch_gemm_tc_stream(M, N, K, none, *B_packed, B_prepacked, D, d_dt, ldd, workspace,
                                      workspace_bytes, static_cast<cudaStream_t>(cuda_stream),
                                      false, A_dense_bf16, lda);
}

mxp_status mxp_quantize_gemm_ready(const void* src, mxp_dtype src_dt, int64_t M, int64_t K,
                                   int64_t ld_src, mxp_mode mode, mxp_mode b_mode, uint8_t* nibbles,
                                   uint8_t* scales, uint8_t* bm_index, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream)
{
    if (mode != MXP_MODE_MXFP4 && mode != MXP_MODE_MXFP4_PLUS) return MXP_ERR_UNSUPPORTED;
    if (!valid_dtype(src_dt) || M <= 0 || K <= 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (src == nullptr || nibbles == nullptr || scales == nullptr) return MXP_ERR_INVALID_ARG;
    if (mode != MXP_MODE_MXFP4 && bm_index == nullptr) return MXP_ERR_INVALID_ARG;
    if (!aligned(src, 16) || !aligned(nibbles, 16)) return MXP_ERR_INVALID_ARG;
    if (src_dt != MXP_BF16 || ld_src != K) return MXP_ERR_UNSUPPORTED;  // the fused kernel's case
    if (b_mode < MXP_MODE_MXFP4 || b_mode > MXP_MODE_MXFP8_PLUS) return MXP_ERR_INVALID_ARG;
    if (mode == MXP_MODE_MXFP4_PLUS && mxp::stream_b_form(mode, b_mode) == MXP_PREPACK_PLAIN) {
        // MXFP4+ against plain MXFP4: Eq. 4's split for the sparse residual instruction
        size_t at = 0, mn = 0, rs = 0, mt = 0, po = 0, pb = 0, tot = 0;
        if (!mxp::stream_a_split_layout(M, K, &at, &mn, &rs, &mt, &po, &pb, &tot)) return MXP_ERR_UNSUPPORTED;
        if (workspace == nullptr || workspace_bytes < tot) return MXP_ERR_WORKSPACE;
        if (!aligned(workspace, 256)) return MXP_ERR_INVALID_ARG;
        uint8_t* w8 = static_cast<uint8_t*>(workspace);
        const mxp::QuantizeSplitOut sp = {w8 + mn, w8 + rs, w8 + mt, po, pb};
        cudaError_t e = mxp::launch_quantize_ready(src, M, K, mode, nibbles, scales, bm_index, w8 + at, nullptr,
                                                   &sp, workspace, static_cast<cudaStream_t>(cuda_stream));
        if (e == cudaErrorNotSupported) return MXP_ERR_UNSUPPORTED;
        return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
    }
    size_t atoms = 0, slots = 0, total = 0;
    if (!mxp::stream_a_ready_layout(M, K, &atoms, &slots, &total)) return MXP_ERR_UNSUPPORTED;
    if (workspace == nullptr || workspace_bytes < total) return MXP_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return MXP_ERR_INVALID_ARG;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaError_t e = mxp::launch_quantize_ready(src, M, K, mode, nibbles, scales, bm_index, ws + atoms,
                                               ws + slots, nullptr, workspace,
                                               static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

mxp_status mxp_gemm_ready(int64_t M, int64_t N, int64_t K, const mxp_packed* A_packed,
                          const mxp_packed* B_packed, const void* B_prepacked,
                          size_t B_prepacked_bytes, void* D, mxp_dtype d_dt, int64_t ldd,
                          void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (M < 0 || N < 0 || K < 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (!valid_dtype(d_dt)) return MXP_ERR_INVALID_ARG;
    if (!valid_packed(A_packed) || !valid_packed(B_packed)) return MXP_ERR_INVALID_ARG;
    if (A_packed->rows != M || A_packed->cols != K || B_packed->rows != N || B_packed->cols != K)
        return MXP_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return MXP_OK;
    if (K == 0) return MXP_ERR_UNSUPPORTED;
    if (B_prepacked == nullptr || D == nullptr || ldd < N) return MXP_ERR_INVALID_ARG;
    if (!aligned(D, d_dt == MXP_BF16 ? 2 : 4)) return MXP_ERR_INVALID_ARG;
    if (!aligned(B_packed->scales, 4)) return MXP_ERR_INVALID_ARG;
    size_t atoms = 0, slots = 0, total = 0;
    if (!mxp::stream_a_ready_layout(M, K, &atoms, &slots, &total) || N <= 128)
        return MXP_ERR_UNSUPPORTED;
    if (mxp::stream_workspace_bytes(M, N, K, A_packed->mode, B_packed->mode) == 0)
        return MXP_ERR_UNSUPPORTED;
    if (A_packed->mode == MXP_MODE_MXFP4_PLUS &&
        mxp::stream_b_form(A_packed->mode, B_packed->mode) == MXP_PREPACK_PLAIN) {
        // A was split by the quantizer (Eq. 4), B comes with plain scale atoms: sparse residual path
        if (B_prepacked_bytes != mxp::stream_prepack_bytes(N, K, MXP_PREPACK_PLAIN) || !aligned(B_prepacked, 256))
            return MXP_ERR_INVALID_ARG;
        return mxp::launch_gemm_tc_sparse(M, N, K, *A_packed, *B_packed, B_prepacked, D, d_dt, ldd, workspace,
                                          workspace_bytes, static_cast<cudaStream_t>(cuda_stream), true);
    }
    if (B_prepacked_bytes != mxp::stream_prepack_bytes(N, K, mxp::stream_wide_form(B_packed->mode)) ||
        !aligned(B_prepacked, 256))
        return MXP_ERR_INVALID_ARG;
    return mxp::launch_gemm_tc_stream(M, N, K, *A_packed, *B_packed, B_prepacked, D, d_dt, ldd,
                                      workspace, workspace_bytes,
                                      static_cast<cudaStream_t>(cuda_stream), true);
}

mxp_status mxp_wait_selftest(void* workspace, size_t workspace_bytes, int64_t limit_cycles,
                             void* cuda_stream)
{
    if (workspace == nullptr || workspace_bytes < sizeof(mxp::StatusBlock) || !aligned(workspace, 16))
        return MXP_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > 2000000000ll) return MXP_ERR_INVALID_ARG;  // <= ~1 s
    return mxp::launch_wait_selftest(workspace, limit_cycles, static_cast<cudaStream_t>(cuda_stream));
}

mxp_status mxp_gemm_status(const void* workspace, void* cuda_stream)
{
    if (workspace == nullptr) return MXP_ERR_INVALID_ARG;
    mxp::StatusBlock sb;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(&sb, workspace, sizeof(sb), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return MXP_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return MXP_ERR_CUDA;
    return sb.code == 0 ? MXP_OK : static_cast<mxp_status>(sb.code);
}

mxp_status mxp_gemm_clock_stamp(const void* workspace, void* cuda_stream, uint64_t* sm_cycles,
                                uint64_t* nanoseconds)
{
    if (workspace == nullptr || sm_cycles == nullptr || nanoseconds == nullptr)
        return MXP_ERR_INVALID_ARG;
    mxp::ClockStamp cs;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(&cs, static_cast<const uint8_t*>(workspace) + mxp::kClockStampOffset,
                        sizeof(cs), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return MXP_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return MXP_ERR_CUDA;
    if (cs.ns_end <= cs.ns_begin || cs.clk_end <= cs.clk_begin) return MXP_ERR_UNSUPPORTED;
    *sm_cycles = cs.clk_end - cs.clk_begin;
    *nanoseconds = cs.ns_end - cs.ns_begin;
    return MXP_OK;
}

mxp_status mxp_tensor_peak_probe(int kind, int iters, double* ms, double* flops)
{
    if (ms == nullptr || flops == nullptr || iters <= 0 || kind < 0 || kind > 5)
        return MXP_ERR_INVALID_ARG;
    return mxp::tensor_peak_probe(kind, iters, ms, flops);
}

}  // extern "C"
