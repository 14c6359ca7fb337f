// Prefill dispatch: picks the kernel that serves a (shape, alignment) case.
#include "flux_internal.h"

namespace flux {

int prefill_mma_setup();
int launch_prefill_mma(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v,
                       int q_start, int Nq, void *out, cudaStream_t st);

int prefill_setup(flux_plan *p)
{
    (void)p;
    return prefill_mma_setup();
}

int launch_prefill(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v,
                   int q_start, int Nq, void *out, cudaStream_t st)
{
    return launch_prefill_mma(p, layer, req, q, k, v, q_start, Nq, out, st);
}

}  // namespace flux
