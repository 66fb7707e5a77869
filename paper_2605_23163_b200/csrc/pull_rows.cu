// fdd_pull_masked_rows: the logits rows of the MASKED positions, fetched from host memory by a kernel.
//
// The caller's logits live in pinned host memory that the device can address.  A small grid reads
// the state array on the device and pulls exactly the rows whose state is MASKED across PCIe into
// the device buffer: one launch instead of a copy per run of rows, no state read-back and no host
// synchronisation, so a step that takes its logits from the host can be issued ahead like any other.
#include "fdd_internal.h"

namespace {

constexpr int kPullThreads = 256;
constexpr int kPullCtas = 32;          // enough loads in flight to fill the link (measured: 16 CTAs already do)
constexpr int kPullUnroll = 8;         // 16-byte loads in flight per thread

__global__ void __launch_bounds__(kPullThreads)
pull_rows_kernel(const unsigned char* __restrict__ src, unsigned char* __restrict__ dst,
                 const uint8_t* __restrict__ state, int rows, size_t row_bytes, int vec_ok,
                 unsigned long long* __restrict__ bytes_pulled) {
    for (int r = blockIdx.x; r < rows; r += gridDim.x) {
        if (state[r] != FDD_MASKED) continue;            // (the same byte for every thread of the CTA)
        const size_t off = static_cast<size_t>(r) * row_bytes;
        if (vec_ok) {
            const uint4* s = reinterpret_cast<const uint4*>(src + off);
            uint4* d = reinterpret_cast<uint4*>(dst + off);
            const size_t n16 = row_bytes / 16;
            size_t i = threadIdx.x;
            for (; i + (kPullUnroll - 1) * kPullThreads < n16; i += kPullUnroll * kPullThreads) {
                uint4 v[kPullUnroll];
#pragma unroll
                for (int u = 0; u < kPullUnroll; ++u) v[u] = s[i + u * kPullThreads];
#pragma unroll
                for (int u = 0; u < kPullUnroll; ++u) d[i + u * kPullThreads] = v[u];
            }
            for (; i < n16; i += kPullThreads) d[i] = s[i];
        } else {
            // rows that are not a multiple of 16 bytes apart: two bytes at a time (logits are 2 or 4 bytes wide)
            const uint16_t* s = reinterpret_cast<const uint16_t*>(src + off);
            uint16_t* d = reinterpret_cast<uint16_t*>(dst + off);
            for (size_t i = threadIdx.x; i < row_bytes / 2; i += kPullThreads) d[i] = s[i];
        }
        if (threadIdx.x == 0 && bytes_pulled != nullptr) atomicAdd(bytes_pulled, static_cast<unsigned long long>(row_bytes));
    }
}

}  // namespace

fdd_status fdd_pull_masked_rows(fdd_ctx* ctx, const void* host_logits, void* dev_logits, const uint8_t* dev_state,
                                int rows, unsigned long long* bytes_pulled, void* stream) {
    CallRange range("fdd_pull_masked_rows");
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (!host_logits || !dev_logits || !dev_state || rows < 0) {
        ctx->last_error = "fdd_pull_masked_rows: host_logits/dev_logits/dev_state is NULL or rows < 0";
        return FDD_ERR_INVALID_ARG;
    }
    if (rows == 0) return FDD_OK;
    // the address a kernel can use for the host buffer (pinned memory only)
    cudaPointerAttributes attr;
    cudaError_t e = cudaPointerGetAttributes(&attr, host_logits);
    if (e != cudaSuccess || attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) {
        (void)cudaGetLastError();
        ctx->last_error = "fdd_pull_masked_rows: host_logits must be pinned host memory that the device can address "
                          "(cudaHostAlloc / cudaHostRegister)";
        return FDD_ERR_INVALID_ARG;
    }
    const size_t row_bytes = static_cast<size_t>(ctx->cfg.vocab) * (ctx->cfg.logits_dtype == FDD_LOGITS_BF16 ? 2 : 4);
    const int vec_ok = row_bytes % 16 == 0 && reinterpret_cast<uintptr_t>(attr.devicePointer) % 16 == 0 &&
                       reinterpret_cast<uintptr_t>(dev_logits) % 16 == 0;
    const int ctas = rows < kPullCtas ? rows : kPullCtas;
    pull_rows_kernel<<<ctas, kPullThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const unsigned char*>(attr.devicePointer), static_cast<unsigned char*>(dev_logits), dev_state, rows,
        row_bytes, vec_ok, bytes_pulled);
    ctx->launches += 1;
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        ctx->last_error = std::string("fdd_pull_masked_rows launch: ") + cudaGetErrorString(e);
        return FDD_ERR_CUDA;
    }
    return FDD_OK;
}
