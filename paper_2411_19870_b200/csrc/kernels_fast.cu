// Register-resident fast-DCT kernels for 2-D tensors (placeholder until implemented).
#include "demo_internal.h"

bool demo_fast_supported(int) { return false; }
cudaError_t demo_launch_compress_fast(int, const DemoCompressArgs &, int, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t demo_launch_decode_fast(int, const DemoDecodeArgs &, int, cudaStream_t) { return cudaErrorNotSupported; }
