// Tensor-core chunk forward (tcgen05 / TMEM) -- placeholder until the kernel lands.
#include "common.cuh"

namespace kla {

bool chunk_tc_supported(int, int, int) { return false; }

cudaError_t launch_chunk_tc(const ChunkParams &, int, int, int, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace kla
