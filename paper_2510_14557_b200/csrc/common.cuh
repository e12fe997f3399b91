// Shared declarations of the libmxp translation units (device launchers + helpers).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mxp.h"

namespace mxp {

// ---- launchers (each validates nothing: the C ABI layer has done that) -----------------
cudaError_t launch_quantize(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                            int64_t ld_src, mxp_mode mode, uint8_t* nibbles, uint8_t* scales,
                            uint8_t* bm_index, cudaStream_t stream);

cudaError_t launch_quantize_reordered(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                                      int64_t ld_src, const int32_t* order, mxp_mode mode,
                                      uint8_t* nibbles, uint8_t* scales, uint8_t* bm_index,
                                      cudaStream_t stream);

cudaError_t launch_nvfp4_quantize(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                                  int64_t ld_src, float ts, bool plus, uint8_t* nibbles,
                                  uint8_t* scales, uint8_t* bm_index, cudaStream_t stream);
cudaError_t launch_nvfp4_dequantize(const uint8_t* nibbles, const uint8_t* scales,
                                    const uint8_t* bm_index, int64_t rows, int64_t cols, float ts,
                                    bool plus, void* dst, mxp_dtype dt, int64_t ld_dst,
                                    cudaStream_t stream);

cudaError_t launch_dequantize(const mxp_packed& p, void* dst, mxp_dtype dt, int64_t ld_dst,
                              cudaStream_t stream);

// Weight-only form: D = A(bf16, M x K) * dec(B)^T.
size_t skinny_workspace_bytes(int64_t M, int64_t N, int64_t K);
cudaError_t launch_gemm_weight_only(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                    const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                                    void* workspace, size_t workspace_bytes,
                                    cudaStream_t stream);

// Streamed variant for decode shapes (N % 16 == 0, K % 256 == 0, activations that fit shared
// memory).  `status` (may be nullptr) is a StatusBlock the kernel writes only when a wait
// runs out.
bool wo_stream_supported(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                         const mxp_packed& B);
cudaError_t launch_gemm_wo_stream(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                  const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                                  void* status, cudaStream_t stream, bool chained = false);

// MXFP6(+) / MXFP8(+): quantize and decode only (quantize_wide.cu).
cudaError_t launch_quantize_wide(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                                 int64_t ld_src, mxp_mode mode, uint8_t* codes, uint8_t* scales,
                                 uint8_t* bm_index, cudaStream_t stream);
cudaError_t launch_dequantize_wide(const mxp_packed& p, void* dst, mxp_dtype dt, int64_t ld_dst,
                                   cudaStream_t stream);

// Decode shapes (M <= 16) on the FP4 tensor path with weights re-tiled once (gemm_decode_tc.cu).
size_t decode_prepack_bytes(int64_t N, int64_t K, mxp_mode mode);  // 0: not supported
size_t decode_workspace_bytes(int64_t M, int64_t K);               // 0: not supported
mxp_status decode_prepack(const mxp_packed& B, void* out, size_t out_bytes, cudaStream_t stream);
mxp_status launch_gemm_decode_tc(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                 mxp_mode b_mode, const void* b_prepacked, size_t b_prepacked_bytes,
                                 void* D, mxp_dtype d_dt, int64_t ldd, void* workspace,
                                 size_t workspace_bytes, bool chained, const void* next_prepacked,
                                 size_t next_prepacked_bytes, cudaStream_t stream);

// Block-scaled tensor-core form: both operands packed.
size_t tc_workspace_bytes(int64_t M, int64_t N, int64_t K, mxp_mode a_mode, mxp_mode b_mode);
size_t tc_compact_workspace_bytes();  // enough for the kernels that work in place
mxp_status launch_gemm_tc(int64_t M, int64_t N, int64_t K, const mxp_packed& A,
                          const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                          void* workspace, size_t workspace_bytes, cudaStream_t stream);

// Streamed CTA-pair kernel on prepacked operands (scale atoms, MX+ data widened to E2M3 or E4M3
// codes): needs
// M, N > 128 and a workspace of stream_workspace_bytes() (0 = shape not supported).
size_t stream_workspace_bytes(int64_t M, int64_t N, int64_t K, mxp_mode a_mode, mxp_mode b_mode);
mxp_status launch_gemm_tc_stream(int64_t M, int64_t N, int64_t K, const mxp_packed& A,
                                 const mxp_packed& B, const void* b_prepacked, void* D,
                                 mxp_dtype d_dt, int64_t ldd, void* workspace,
                                 size_t workspace_bytes, cudaStream_t stream, bool a_ready = false,
                                 const void* a_dense = nullptr, int64_t lda = 0);
// Weight-only form on the same kernel (bf16 activations as two E4M3 planes): workspace it
// needs, 0 = not supported (K % 128, weights other than the 4-bit modes).
size_t stream_dense_workspace_bytes(int64_t M, int64_t N, int64_t K, mxp_mode b_mode);
size_t stream_dense_prepacked_workspace_bytes(int64_t M, int64_t K);  // with B prepacked
// Quantizer that also writes A in the form that kernel reads (with a prepacked B no prepack
// launch is left): offsets inside the GEMM's workspace, and the launch (bf16, contiguous rows,
// MXFP4 / MXFP4+).
bool stream_a_ready_layout(int64_t M, int64_t K, size_t* atoms, size_t* slots, size_t* total);
// The same for the sparse-residual form (A is MXFP4+, its partner plain MXFP4): where inside the
// workspace the quantizer writes Eq. 4's split of A, and which of the metadata's bytes belong to
// rows past A's end (they are filled with valid nibbles before the quantizer runs).
struct QuantizeSplitOut {
    uint8_t *main, *res, *meta;
    size_t meta_pad_offset, meta_pad_bytes;
};
bool stream_a_split_layout(int64_t M, int64_t K, size_t* atoms, size_t* main, size_t* res, size_t* meta,
                           size_t* meta_pad_offset, size_t* meta_pad_bytes, size_t* total);
cudaError_t launch_quantize_ready(const void* src, int64_t rows, int64_t cols, mxp_mode mode,
                                  uint8_t* nibbles, uint8_t* scales, uint8_t* bm_index,
                                  uint8_t* atoms, uint8_t* slots, const QuantizeSplitOut* split, void* status,
                                  cudaStream_t stream);
// One operand in the form that kernel reads, written once, e.g. for weights.  `form` is an
// mxp_prepack_form: scale atoms only, atoms + widened codes, or atoms + the Eq. 4 split of an
// MXFP4+ operand.  stream_prepack_bytes() == 0: shape or form not supported.
size_t stream_prepack_bytes(int64_t rows, int64_t K, int form);
mxp_status stream_prepack(const mxp_packed& P, int form, void* out, size_t out_bytes,
                          cudaStream_t stream);
// One MXFP4+ operand against one MXFP4 operand: FP4 main pass plus sparse residual MMA (Eq. 4,
// Algorithm 1).  Workspace it needs (0: not this case, or shape not supported); `b_prepacked`:
// B comes prepacked (form MXP_PREPACK_SPLIT if B is the MXFP4+ side, MXP_PREPACK_PLAIN if not).
size_t stream_sparse_workspace_bytes(int64_t M, int64_t N, int64_t K, mxp_mode a_mode, mxp_mode b_mode,
                                     bool b_prepacked);
mxp_status launch_gemm_tc_sparse(int64_t M, int64_t N, int64_t K, const mxp_packed& A, const mxp_packed& B,
                                 const void* b_prepacked, void* D, mxp_dtype d_dt, int64_t ldd,
                                 void* workspace, size_t workspace_bytes, cudaStream_t stream,
                                 bool a_ready = false);
// The form of B's prepacked copy that a packed x packed GEMM with these modes reads.
int stream_b_form(mxp_mode a_mode, mxp_mode b_mode);
// The widened form of an operand of this mode: MXP_PREPACK_WIDE (E2M3 codes) or MXP_PREPACK_WIDE8 (E4M3 bytes).
int stream_wide_form(mxp_mode b_mode);

// Kernel choices a test or a measurement may force (mxp_debug_override): process-wide, 0 = the
// library decides.
int override_get(int knob);

// cuTensorMapEncodeTiled through the runtime's driver entry point (no libcuda link).
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                              const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                              const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn tensormap_encode_fn();
int sm_count();  // of the current device, cached; -1 on error

// Raises a kernel's dynamic shared-memory limit once per device (the attribute belongs to
// the device's context, and the call is not free).  `done` is the caller's per-kernel record.
struct SmemAttrOnce {
    bool done[64] = {};
};
template <typename Kernel>
cudaError_t ensure_dynamic_smem(Kernel kern, int bytes, SmemAttrOnce& once)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && once.done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && dev >= 0 && dev < 64) once.done[dev] = true;
    return e;
}

// Launches the bounded-wait self-test (see selftest.cu); the result is read with the status
// block like a GEMM's.
mxp_status launch_wait_selftest(void* workspace, int64_t limit_cycles, cudaStream_t stream);

mxp_status tensor_peak_probe(int kind, int iters, double* ms, double* flops);

// First 16 bytes of every GEMM workspace.
struct StatusBlock {
    uint32_t code;    // 0 = ok, otherwise an mxp_status
    uint32_t where;   // which wait gave up (kernel-specific tag)
    uint32_t pad[2];
};
constexpr size_t kStatusBytes = 256;  // keeps what follows 256-byte aligned

// Bytes 64..95 of a workspace of the streamed tensor-core GEMM: SM cycle counter and global
// nanosecond timer, read by its first CTA when it starts and when it has stored its last tile.
// cycles / nanoseconds is the SM clock the kernel actually ran at (the power cap lowers it).
struct ClockStamp {
    unsigned long long clk_begin, ns_begin, clk_end, ns_end;
};
constexpr size_t kClockStampOffset = 64;

}  // namespace mxp
