// placeholder until the tcgen05 kernel lands
#include "kernels.h"
namespace yoco {
cudaError_t launch_chunk(const ChunkParams&, const CUtensorMap&, const CUtensorMap&, const CUtensorMap&,
                         int, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t chunk_kernel_setup() { return cudaSuccess; }
}
