// K2 placeholder
#include "peagle_internal.h"
namespace peagle {
int launch_bwd(const Plan &, const BwdArgs &, EncodeTiledFn, int, cudaStream_t) { return 0; }
int launch_cast_grads(const float *, const float *, void *, void *, size_t, cudaStream_t) { return 0; }
}
