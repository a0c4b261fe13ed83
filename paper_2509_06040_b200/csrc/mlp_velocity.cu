// Per-token MLP velocity stage (placeholder until the tcgen05 kernel lands).
#include "internal.h"

namespace bgrpo {
size_t mlp_packed_bytes(int hidden) { return static_cast<size_t>(hidden) * 64 * 2 * 2; }
cudaError_t launch_mlp_pack(const uint16_t*, const uint16_t*, int, void*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t launch_mlp(const float*, int64_t, int64_t, int, int64_t, const void*, int, float*, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace bgrpo
