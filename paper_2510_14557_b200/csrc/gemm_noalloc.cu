// mxp_gemm_noalloc: the packed-operand GEMM for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: code that runs inside another
// framework's memory pool and must not grow the process's footprint, a plugin loaded after
// the pool has claimed the whole device, or a caller that has no allocator of its own to ask
// for the few hundred bytes of workspace mxp_gemm wants.  For them the kernel's scratch (the
// status block the bounded waits report into) lives in a file-scope device array that the
// library carries itself; inputs and outputs still come from the caller.
#include <mutex>

#include "common.cuh"

namespace {

// Every device that loads the library holds these bytes until the process exits.
constexpr size_t kScratchBytes = 4096;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_mu;

// In host code `g_noalloc_scratch` names a host-side stand-in, not device memory: the address
// a kernel may use has to be asked for, once per device, with that device current.
cudaError_t scratch_for_current_device(void** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" mxp_status mxp_gemm_noalloc(int64_t M, int64_t N, int64_t K, const mxp_packed* A_packed,
                                       const mxp_packed* B_packed, void* D, mxp_dtype d_dt,
                                       int64_t ldd, mxp_status* kernel_status, void* cuda_stream)
{
    if (M < 0 || N < 0 || K < 0 || K % 32 != 0) return MXP_ERR_INVALID_ARG;
    if (d_dt != MXP_F32 && d_dt != MXP_BF16) return MXP_ERR_INVALID_ARG;
    if (A_packed == nullptr || B_packed == nullptr) return MXP_ERR_INVALID_ARG;
    for (const mxp_packed* p : {A_packed, B_packed}) {
        if (p->mode < MXP_MODE_MXFP4 || p->mode > MXP_MODE_MXFP8_PLUS) return MXP_ERR_INVALID_ARG;
        if (p->rows < 0 || p->cols != K) return MXP_ERR_INVALID_ARG;
        if (p->rows > 0 && p->cols > 0) {  // an empty operand needs no planes (as for mxp_gemm)
            if (p->nibbles == nullptr || p->scales == nullptr) return MXP_ERR_INVALID_ARG;
            if (reinterpret_cast<uintptr_t>(p->nibbles) % 16 != 0) return MXP_ERR_INVALID_ARG;
            if (p->mode != MXP_MODE_MXFP4 && p->mode != MXP_MODE_MXFP6 && p->mode != MXP_MODE_MXFP8 &&
                p->bm_index == nullptr)
                return MXP_ERR_INVALID_ARG;
        }
    }
    if (A_packed->rows != M || B_packed->rows != N) return MXP_ERR_INVALID_ARG;
    if (M > 0 && N > 0) {
        if (K == 0) return MXP_ERR_UNSUPPORTED;
        if (D == nullptr || ldd < N) return MXP_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(D) % (d_dt == MXP_BF16 ? 2 : 4) != 0) return MXP_ERR_INVALID_ARG;
        // MX++ and the 6- and 8-bit modes run only on operands prepared in a workspace
        if (A_packed->mode > MXP_MODE_MXFP4_PLUS || B_packed->mode > MXP_MODE_MXFP4_PLUS) return MXP_ERR_UNSUPPORTED;
    }
    // every argument is acceptable from here on: only now is the out-parameter touched
    if (kernel_status != nullptr) *kernel_status = MXP_OK;
    if (M == 0 || N == 0) return MXP_OK;

    // the scratch this problem needs must fit the array the library carries
    const size_t need = mxp::tc_compact_workspace_bytes();
    if (need > kScratchBytes) return MXP_ERR_WORKSPACE;

    void* scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) return MXP_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps what the last call left in it; launch_gemm_tc clears the status block
    // it reads (a memset on the stream), nothing else has to start at zero
    mxp_status st = mxp::launch_gemm_tc(M, N, K, *A_packed, *B_packed, D, d_dt, ldd, scratch,
                                        kScratchBytes, stream);
    if (st != MXP_OK) return st;
    if (kernel_status != nullptr) {
        mxp::StatusBlock sb;
        if (cudaMemcpyAsync(&sb, scratch, sizeof(sb), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
            return MXP_ERR_CUDA;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return MXP_ERR_CUDA;
        *kernel_status = sb.code == 0 ? MXP_OK : static_cast<mxp_status>(sb.code);
    }
    return MXP_OK;
}
