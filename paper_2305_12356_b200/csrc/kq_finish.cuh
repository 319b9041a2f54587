// The step that turns summed squared errors into outputs: per-candidate MSE in the caller's order and, when a record
// is wanted, Algorithm 1's comparison (strictly smaller error wins, candidates in the caller's order).
#pragma once
#include "mofq_internal.h"

namespace mofq {
namespace kqfin {

// tot: [set][canonical slot] sums of squared errors over the whole tensor
__device__ inline void write_outputs(const double *tot, const Finalize &fin, WsHeader *hdr)
{
    int status = 0;
    if (fin.res) status = atomicExch(&hdr->status, 0);
    for (int s = 0; s < fin.n_sets; ++s) {
        double err[MOFQ_MAX_CAND];
        for (int i = 0; i < fin.n_cand; ++i) {
            err[i] = tot[s * fin.nc + fin.perm[i]] * fin.inv_n;
            if (fin.mse_out) fin.mse_out[s * fin.n_cand + i] = (float)err[i];
        }
        if (fin.res) {
            // Algorithm 1: min_error = inf; replace only on a strictly smaller error, caller's order
            double best = INFINITY, second = INFINITY;
            int chosen = -1;
            for (int i = 0; i < fin.n_cand; ++i) {
                if (err[i] < best) {
                    second = best;
                    best = err[i];
                    chosen = i;
                } else if (err[i] < second) {
                    second = err[i];
                }
            }
            mofq_result r;
            r.chosen = chosen;
            r.status = status;
            for (int i = 0; i < MOFQ_MAX_CAND; ++i) {
                r.error[i] = i < fin.n_cand ? (float)err[i] : 0.0f;
                r.nsr[i] = 0.0f;
            }
            r.rel_margin = best > 0.0 ? (float)((second - best) / best) : INFINITY;
            r.reserved = 0;
            fin.res[s] = r;
        }
    }
}

}  // namespace kqfin
}  // namespace mofq
