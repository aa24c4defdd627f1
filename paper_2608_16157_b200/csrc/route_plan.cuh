// Decode-sized calls: route, permute and plan of one layer in a single one-CTA launch.
#pragma once
#include "plan.cuh"
#include "route.cuh"

namespace ftmoe {

__global__ void __launch_bounds__(1024) route_plan_small_kernel(RouteParams rp, PlanParams pp) {
  extern __shared__ __align__(16) unsigned char s_dyn[];
  // a streaming kernel launched as a programmatic dependent may be scheduled now; it waits for this grid to
  // complete before it reads the plan
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __shared__ RouteSmem rs;
  __shared__ PlanSmem ps;
  int64_t t;
  int slot;
  plan_prefetch(pp, s_dyn, t, slot);   // state loads overlap the logits load of the routing below
  route_small_body(rp, rs);
  __syncthreads();
  const int tid = threadIdx.x;
  int c = 0, off = 0;
  if (tid < rp.E) { c = rs.cnt[tid]; off = rs.off[tid]; }
  plan_body(pp, ps, s_dyn, c, off, rp.T * rp.k, t, slot);
}

}  // namespace ftmoe
