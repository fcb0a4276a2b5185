// CaP scoring on the tensor cores (Sec. 3.3.1, Eq. 2) - interface.
#pragma once
#include "../../include/ipot.h"
#include "common.cuh"

namespace ipotk {

struct TcPlan {
    bool usable = false;
};

inline void tc_plan_init(TcPlan &, const ipot_config_t &, const void *, int) {}
inline void tc_plan_destroy(TcPlan &) {}
inline bool tc_applicable(const TcPlan &plan, const ipot_config_t &, int, int) { return plan.usable; }
inline int tc_launch(TcPlan &, const ipot_config_t &, const void *, const void *, float *, size_t, int, int, int,
                     int *, cudaStream_t, int *, int *)
{
    return IPOT_E_INVALID;
}

}  // namespace ipotk
