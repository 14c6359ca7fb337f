// Prefill dispatch: picks the kernel that serves a launch.
#include "flux_internal.h"

namespace flux {

int prefill_mma_setup();
int launch_prefill_mma(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v,
                       int q_start, int Nq, void *out, cudaStream_t st);
int prefill_tc_setup();
int prefill_blocks_setup();
int launch_prefill_tc(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v,
                      int q_start, int Nq, void *out, cudaStream_t st, const uint8_t *block_mask, int n_kv_blocks);
int prefill_pair_setup();
bool prefill_pair_supports(const flux_plan *p);
int launch_prefill_pair(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v, int q_start,
                        int Nq, void *out, cudaStream_t st);
int launch_prefill_blocks_mma(flux_plan *p, const void *q, const void *k, const void *v, int q_start, int Nq,
                              const uint8_t *block_mask, int n_kv_blocks, void *out, cudaStream_t st);

int prefill_setup(flux_plan *p)
{
    p->prefill_kernel = FLUX_PREFILL_AUTO;
    int rc = prefill_mma_setup();
    if (!rc) rc = prefill_tc_setup();
    if (!rc) rc = prefill_blocks_setup();
    if (!rc) rc = prefill_pair_setup();
    return rc;
}

int launch_prefill(flux_plan *p, int layer, int req, const void *q, const void *k, const void *v,
                   int q_start, int Nq, void *out, cudaStream_t st)
{
    // The tcgen05 kernel serves every shape (TMA zero-fills ragged tiles); the warp-MMA
    // kernel stays selectable for comparison.
    if (p->prefill_kernel == FLUX_PREFILL_WARP_MMA)
        return launch_prefill_mma(p, layer, req, q, k, v, q_start, Nq, out, st);
    if (p->prefill_kernel == FLUX_PREFILL_TCGEN05_PAIR && prefill_pair_supports(p))
        return launch_prefill_pair(p, layer, req, q, k, v, q_start, Nq, out, st);
    return launch_prefill_tc(p, layer, req, q, k, v, q_start, Nq, out, st, nullptr, 0);
}

int launch_prefill_blocks(flux_plan *p, const void *q, const void *k, const void *v, int q_start, int Nq,
                          const uint8_t *block_mask, int n_kv_blocks, void *out, cudaStream_t st)
{
    if (p->prefill_kernel == FLUX_PREFILL_WARP_MMA)
        return launch_prefill_blocks_mma(p, q, k, v, q_start, Nq, block_mask, n_kv_blocks, out, st);
    return launch_prefill_tc(p, 0, 0, q, k, v, q_start, Nq, out, st, block_mask, n_kv_blocks);
}

}  // namespace flux
