// One group of kernel instances (see cg_instances.h); compiled once per group.
#include "cg_kernel.cuh"
#include "cg_instances.h"

#ifndef CG_INST_GROUP
#error "compile with -DCG_INST_GROUP=<0..8>"
#endif

namespace cg {
#define CG_DEFINE(BN, CGN, KM, CV) template CG_KERNEL_SIGNATURE(BN, CGN, KM, CV)
#if CG_INST_GROUP == 0
CG_INSTANCES_GROUP0(CG_DEFINE)
#elif CG_INST_GROUP == 1
CG_INSTANCES_GROUP1(CG_DEFINE)
#elif CG_INST_GROUP == 2
CG_INSTANCES_GROUP2(CG_DEFINE)
#elif CG_INST_GROUP == 3
CG_INSTANCES_GROUP3(CG_DEFINE)
#elif CG_INST_GROUP == 4
CG_INSTANCES_GROUP4(CG_DEFINE)
#elif CG_INST_GROUP == 5
CG_INSTANCES_GROUP5(CG_DEFINE)
#elif CG_INST_GROUP == 6
CG_INSTANCES_GROUP6(CG_DEFINE)
#elif CG_INST_GROUP == 7
CG_INSTANCES_GROUP7(CG_DEFINE)
#elif CG_INST_GROUP == 8
CG_INSTANCES_GROUP8(CG_DEFINE)
#else
#error "CG_INST_GROUP out of range"
#endif
}  // namespace cg
