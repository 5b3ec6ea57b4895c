// The library's context object and small host helpers shared by its translation units.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "decode.cuh"
#include "tables.h"

// Device tables of the encoder (point -> index): present for codes the encoder supports.
struct EncTables {
    const uint16_t* pos_by_low12 = nullptr;   // [4096] low 12 bits of a Golay codeword -> its position in the sorted table
    const uint64_t* hash_key = nullptr;       // [hash_size] signature of a class (0 = empty slot)
    const uint32_t* hash_cls = nullptr;       // [hash_size] its class number
    uint32_t hash_mask = 0;                   // hash_size - 1 (a power of two)
    const uint64_t* sig_of_value = nullptr;   // [64] signature contribution of one coordinate of absolute value a
};

struct llvq_ctx {
    int device = 0;
    llvq::HostTables host;
    llvq::DevCode dev{};
    void* d_blob = nullptr;          // one allocation holding every device table
    unsigned long long* d_err = nullptr;
    int sm_count = 0;
    float* d_scratch = nullptr;      // split-K accumulation buffer of the small-batch GEMM, kept all-zero between calls
    uint32_t* d_counters = nullptr;  // per row tile arrival counters, kept zero between calls
    void* d_shard = nullptr;         // device copy of the destinations (peers' Y and flags) of the row-sharded GEMM in flight
    bool fast = false;               // class tables fit the shared-memory image; otherwise they are read from global memory
    llvq::FastLayout fl{};
    const uint8_t* d_image = nullptr;
    bool can_encode = false;         // m_lo == 2, m_hi >= 6, indices fit 64 bits
    EncTables enc{};
    const uint32_t* d_golay = nullptr;   // [4096] sorted codewords in global memory
    const uint16_t* d_sort_rank = nullptr;   // [nclasses] (fast codes with at most 1023 classes) position of a class in the order of the sorted layout
};

namespace llvq {

struct DeviceGuard {
    int prev = -1; bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace llvq
