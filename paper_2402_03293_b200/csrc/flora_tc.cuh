// Tensor-core (tcgen05) kernels of the path: placeholder interface, nothing eligible yet.
#pragma once
#include <atomic>
#include <vector>

#include "../../include/flora.h"

namespace flora {

struct TcSet {
    bool compress_ready = false;
    bool decompress_ready = false;
};

__device__ int g_flora_error_word;

inline bool tc_supported(const flora_mat*, const flora_mat*) { return false; }
inline flora_status tc_compress_single(const flora_mat*, flora_mat*, uint64_t, float, float, cudaStream_t, std::atomic<uint64_t>&) { return FLORA_ERR_UNSUPPORTED; }
inline flora_status tc_decompress_single(flora_mat*, const flora_mat*, uint64_t, float, cudaStream_t, std::atomic<uint64_t>&) { return FLORA_ERR_UNSUPPORTED; }
inline flora_status tc_set_build(TcSet&, const std::vector<flora_mat>&, const std::vector<flora_mat>&, const std::vector<flora_mat>&) { return FLORA_OK; }
inline void tc_set_free(TcSet&) {}
inline flora_status tc_set_rebind(TcSet&, const std::vector<flora_mat>&, const std::vector<flora_mat>&) { return FLORA_OK; }
inline flora_status tc_set_compress(TcSet&, const uint64_t*, float, float, cudaStream_t, std::atomic<uint64_t>&) { return FLORA_ERR_UNSUPPORTED; }
inline flora_status tc_set_decompress(TcSet&, const uint64_t*, float, cudaStream_t, std::atomic<uint64_t>&) { return FLORA_ERR_UNSUPPORTED; }
inline bool tc_read_and_clear_error(int* word)
{
    int zero = 0;
    if (cudaMemcpyFromSymbol(word, g_flora_error_word, sizeof(int)) != cudaSuccess) return false;
    return cudaMemcpyToSymbol(g_flora_error_word, &zero, sizeof(int)) == cudaSuccess;
}

}  // namespace flora
