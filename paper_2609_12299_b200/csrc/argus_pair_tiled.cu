// argus_pair_tiled.cu — tiled pairing kernel (placeholder until the tiled kernel lands).
#include "argus_pair_common.cuh"

bool argus_pair_tiled_usable(const ArgusPairArgs&) { return false; }
int argus_launch_pair_tiled(const ArgusPairArgs&, cudaStream_t) { return ARGUS_ERR_INVALID_ARG; }
