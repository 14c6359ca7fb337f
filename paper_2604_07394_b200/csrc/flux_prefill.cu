// Prefill entry: both the routed layers (Eq. 1 / Eq. 2) and the block-mask layers run on the tcgen05 kernel.
#include "flux_internal.h"

namespace flux {

int prefill_tc_setup();
int launch_prefill_tc(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v, int q_start, int Nq,
                      void *out, cudaStream_t st, const uint8_t *block_mask, int n_kv_blocks);

int prefill_setup(flux_plan *) { return prefill_tc_setup(); }

int launch_prefill(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v, int q_start, int Nq,
                   void *out, cudaStream_t st)
{
    return launch_prefill_tc(p, layer, req, q, k, v, q_start, Nq, out, st, nullptr, 0);   // TMA zero-fills ragged tiles
}

int launch_prefill_blocks(flux_plan *p, const void *q, const void *k, const void *v, int q_start, int Nq,
                          const uint8_t *block_mask, int n_kv_blocks, void *out, cudaStream_t st)
{
    return launch_prefill_tc(p, 0, 0, q, k, v, q_start, Nq, out, st, block_mask, n_kv_blocks);
}

}  // namespace flux
