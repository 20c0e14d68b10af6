// Few-token (decode) forward: placeholder until the weight-streaming kernels land.
#include "internal.h"

namespace ffsp {

bool decode_path_applies(const ffsplit_ctx*, const BlobHeader&, long long) { return false; }
size_t decode_workspace_bytes(const BlobHeader&, long long) { return 0; }
ffsplit_status launch_decode_forward(ffsplit_ctx* ctx, const BlobHeader&, const char*, const void*, long long, void*,
                                     char*, cudaStream_t) {
  return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "decode path not built");
}

}  // namespace ffsp
