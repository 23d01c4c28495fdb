// Tensor-core verifier (placeholder until the tcgen05 kernel lands): takes no shape.
#include "common.cuh"
#include "launch.h"

namespace spr {
int launch_verifier_tensor(const VerifyParams &, int, cudaStream_t) { return -1; }
}  // namespace spr
