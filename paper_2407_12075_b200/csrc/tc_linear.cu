// placeholder until the tcgen05 kernel lands
#include "common.cuh"
namespace tbn {
bool tensor_path_supported(const LayerArgs &) { return false; }
int launch_tensor_linear(const LayerArgs &, int *, cudaStream_t) { return TBN_ERR_UNSUPPORTED; }
}
