// fp16 instantiations of the row quantiser (a translation unit of its own so that the
// two element types compile in parallel)
#include "rowquant_impl.cuh"

namespace aweq {
aweq_status rq_launch_f16(const RowQuantParams &p, const RowQuantPlan &pl, int mode, cudaStream_t stream)
{
    return rq_launch<F16>(p, pl, mode, stream);
}
}  // namespace aweq
