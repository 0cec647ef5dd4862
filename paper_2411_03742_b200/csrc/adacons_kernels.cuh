// Device code of the AdaCons aggregation library (sm_100a only).
//
// Three steps per aggregation (Algorithm 1 of arXiv 2411.03742, run on one device):
//   pass1_*   stream the N x d matrix once: column sums s_k = sum_j g_jk, then per worker
//             N p_i = sum_k g_ik s_k and q_i = sum_k g_ik^2 (Eq. 7).  One partial per block.
//   coeff_*   fixed-order fp64 reduction of the partials, a_i = p_i/sqrt(q_i), sorted
//             momentum (Eq. 11), sum-to-one weights (Eq. 12-13).
//   pass2_*   stream the matrix again: out_k = cast(sum_i gamma_i g_ik) (Eq. 12).
//
// Everything is deterministic: fixed block->tile assignment, fixed per-thread order, fixed
// shuffle trees, fixed-order cross-block sums, no floating-point atomics.
#pragma once

#include "adacons_common.cuh"
#include "adacons_pass1.cuh"
#include "adacons_gram.cuh"
#include "adacons_shift.cuh"
#include "adacons_coeff.cuh"
#include "adacons_pass2.cuh"
#include "adacons_fused.cuh"
