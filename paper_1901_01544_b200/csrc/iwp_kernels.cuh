// sm_100a kernels of the importance-weighted pruning step (Algorithm 1 of the paper).
//
// Nothing here is a dense contraction, so there are no tensor-core instructions: every
// kernel is bound by HBM traffic (or, for the small ones, by launch latency).  The work is
// organised so that the W*N residual/gradient stream is touched as few times as possible
// and always with coalesced 128-bit accesses.
//
// IEEE exactness: the residual add, the eps guard and the division use the explicit
// round-to-nearest intrinsics, so the results do not depend on compiler contraction or
// fast-math flags, and denormals are kept.
//
// The kernels, by step of the path:
//   iwp_device.cuh     shared device helpers (importance arithmetic, vector loads, scans, radix select)
//   iwp_stream.cuh     (a)+(b): accumulate, threshold guess from a sample, single-read streaming pass
//   iwp_select.cuh     (c)+(d): exact radix select, ordered compaction, one-CTA path of small layers
//   iwp_reduce.cuh     (e)-(g): reduction at the index set, zero mask, sharded phases, mask accessor
//   iwp_threshold.cuh  absolute-threshold mode, random selection, layer-wise threshold
#pragma once
#include "iwp_device.cuh"
#include "iwp_reduce.cuh"
#include "iwp_select.cuh"
#include "iwp_stream.cuh"
#include "iwp_threshold.cuh"
