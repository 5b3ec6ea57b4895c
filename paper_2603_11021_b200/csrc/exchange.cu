// Exchange buffers and rank-to-rank signalling for the row-sharded GEMV (one process per GPU).
//
// Each rank allocates one exchange buffer with the CUDA allocator proper (so that the whole allocation can be
// exported), hands its IPC handle to the other ranks through whatever host channel they share, and maps theirs.
// A rank's band of y is written into every rank's buffer by the GEMV kernel itself; afterwards the rank raises an
// epoch number in a flag word of every peer (one word per writer), and each rank waits, with an iteration limit,
// until all its writers have raised the epoch before it reads the vector.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "ctx.h"
#include "llvq.h"

using llvq::DeviceGuard;
using llvq::aligned;

namespace {

constexpr int kMaxRanks = 8;
constexpr uint32_t kWaitSpins = 1u << 20;          // about a second of polling a remote-written word at most

struct PeerFlags {
    uint32_t* at[kMaxRanks];
};

// Runs after the GEMV in stream order (an ordinary launch: every store of the GEMV, remote ones included, has been
// performed when this kernel starts).  Thread p makes them visible system-wide and raises the epoch at peer p.
__global__ void signal_ranks_kernel(PeerFlags pf, int n, uint32_t epoch)
{
    const int p = threadIdx.x;
    if (p >= n) return;
    __threadfence_system();
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(pf.at[p]), "r"(epoch) : "memory");
}

// Thread p waits until writer p has raised its word to `epoch` (or beyond: the comparison is modular).
// Launched as a programmatic dependent: it may start while the kernel before it on the stream is still running
// (the polling then overlaps that kernel's tail), lets the kernel after it start its own prologue, and returns
// only after the kernel before it has completed, so that stream order means what it always means.
__global__ void wait_ranks_kernel(const uint32_t* flags, int world, int skip, uint32_t epoch, uint32_t spins, uint32_t* err_flags)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int p = threadIdx.x;
    if (p < world && p != skip) {
        bool seen = false;
        for (uint32_t it = 0; it < spins && !seen; ++it) {
            uint32_t v;
            asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(flags + p) : "memory");
            seen = (int32_t)(v - epoch) >= 0;
            if (!seen) __nanosleep(64);
        }
        if (!seen) atomicOr(err_flags, (uint32_t)LLVQ_FLAG_WAIT_TIMEOUT);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

int status()
{
    return cudaGetLastError() == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

}  // namespace

extern "C" {

int llvq_exchange_create(const llvq_ctx* ctx, size_t bytes, void** d_buf, unsigned char* handle64)
{
    if (!ctx || ctx->device < 0 || !d_buf || !handle64 || bytes == 0) return LLVQ_EINVAL;
    static_assert(sizeof(cudaIpcMemHandle_t) == LLVQ_EXCHANGE_HANDLE_BYTES, "handle size");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) return LLVQ_ECUDA;
    cudaIpcMemHandle_t h;
    if (cudaMemset(p, 0, bytes) != cudaSuccess || cudaIpcGetMemHandle(&h, p) != cudaSuccess) {
        cudaFree(p);
        cudaGetLastError();
        return LLVQ_ECUDA;
    }
    std::memcpy(handle64, &h, sizeof h);
    *d_buf = p;
    return LLVQ_OK;
}

int llvq_exchange_destroy(const llvq_ctx* ctx, void* d_buf)
{
    if (!ctx || ctx->device < 0) return LLVQ_EINVAL;
    if (!d_buf) return LLVQ_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    return cudaFree(d_buf) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

int llvq_exchange_open(const llvq_ctx* ctx, const unsigned char* handle64, void** d_peer_buf)
{
    if (!ctx || ctx->device < 0 || !handle64 || !d_peer_buf) return LLVQ_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaIpcMemHandle_t h;
    std::memcpy(&h, handle64, sizeof h);
    void* p = nullptr;
    if (cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) {
        cudaGetLastError();
        return LLVQ_ECUDA;
    }
    *d_peer_buf = p;
    return LLVQ_OK;
}

int llvq_exchange_close(const llvq_ctx* ctx, void* d_peer_buf)
{
    if (!ctx || ctx->device < 0) return LLVQ_EINVAL;
    if (!d_peer_buf) return LLVQ_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    return cudaIpcCloseMemHandle(d_peer_buf) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

int llvq_signal_ranks(const llvq_ctx* ctx, uint32_t* const* d_flag_words, int n, uint32_t epoch, void* stream)
{
    if (!ctx || ctx->device < 0 || n < 0 || n > kMaxRanks || (n > 0 && !d_flag_words)) return LLVQ_EINVAL;
    if (n == 0) return LLVQ_OK;
    PeerFlags pf{};
    for (int p = 0; p < n; ++p) {
        if (!d_flag_words[p]) return LLVQ_EINVAL;
        if (!aligned(d_flag_words[p], 4)) return LLVQ_EALIGN;
        pf.at[p] = d_flag_words[p];
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    signal_ranks_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(pf, n, epoch);
    return status();
}

int llvq_wait_ranks(const llvq_ctx* ctx, const uint32_t* d_flags, int world, int skip, uint32_t epoch, uint32_t max_spins, void* stream)
{
    if (!ctx || ctx->device < 0 || !d_flags || world < 1 || world > kMaxRanks || skip >= world) return LLVQ_EINVAL;
    if (!aligned(d_flags, 4)) return LLVQ_EALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    const uint32_t spins = max_spins == 0 ? kWaitSpins : (max_spins < kWaitSpins ? max_spins : kWaitSpins);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(32);
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, wait_ranks_kernel, d_flags, world, skip, epoch, spins, ctx->dev.flags) != cudaSuccess) return LLVQ_ECUDA;
    return status();
}

}  // extern "C"
