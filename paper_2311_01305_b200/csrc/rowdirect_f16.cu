// fp16 instantiations of the direct row quantiser (a translation unit of its own so that the
// two element types compile in parallel)
#include "rowdirect_impl.cuh"

namespace aweq {
aweq_status rd_launch_f16(const RowQuantParams &p, int team_warps, int V, int mode, cudaStream_t stream)
{
    return rd_launch<F16>(p, team_warps, V, mode, stream);
}
}  // namespace aweq
