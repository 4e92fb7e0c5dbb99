// bf16 instantiations of the row quantiser
#include "rowquant_impl.cuh"

namespace aweq {
aweq_status rq_launch_bf16(const RowQuantParams &p, const RowQuantPlan &pl, int mode, cudaStream_t stream)
{
    return rq_launch<BF16>(p, pl, mode, stream);
}
}  // namespace aweq
