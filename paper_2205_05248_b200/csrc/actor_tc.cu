// Tensor-core (tcgen05) actor kernel - placeholder until the kernel lands: reports "unsupported" for
// every shape, so the runtime always selects the FFMA kernel.
#include "common.cuh"

namespace marl {
bool tc_supported(int, int, int, int, int) { return false; }
size_t tc_wpack_bytes(int, int, int, int) { return 0; }
void tc_pack_weights(int, int, int, int, const float*, const float*, const float*, const float*, const float*,
                     const float*, const float*, const float*, void*) {}
void tc_tiling(int, int, int, int* ept, int* num_tiles) { *ept = 1; *num_tiles = 0; }
int launch_actor_tc(const ActorParams&, int, cudaStream_t) { return -(int)cudaErrorNotSupported; }
}  // namespace marl
