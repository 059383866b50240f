// The instances of gemm_epilogue_kernel<BN, CG, B_KMAJOR, MODE> (MODE 0 GEMM, 1 convolution, 2 symmetric A, 3 symmetric B), in
// nine groups of three.  Each group is one
// translation unit (cg_inst.cu compiled with -DCG_INST_GROUP=g), so that the groups compile in parallel; the
// C-ABI file only declares them.
#pragma once

#define CG_INSTANCES_GROUP0(X) X(64, 1, false, 0) X(64, 1, true, 0) X(64, 1, true, 1)
#define CG_INSTANCES_GROUP1(X) X(128, 1, false, 0) X(128, 1, true, 0) X(128, 1, true, 1)
#define CG_INSTANCES_GROUP2(X) X(256, 1, false, 0) X(256, 1, true, 0) X(256, 1, true, 1)
#define CG_INSTANCES_GROUP3(X) X(128, 2, false, 0) X(128, 2, true, 0) X(128, 2, true, 1)
#define CG_INSTANCES_GROUP4(X) X(256, 2, false, 0) X(256, 2, true, 0) X(256, 2, true, 1)
#define CG_INSTANCES_GROUP5(X) X(512, 2, false, 0) X(512, 2, true, 0) X(512, 2, true, 1)
#define CG_INSTANCES_GROUP6(X) X(128, 1, false, 2) X(128, 1, true, 2) X(256, 1, false, 2)
#define CG_INSTANCES_GROUP7(X) X(256, 1, true, 2) X(256, 2, false, 2) X(256, 2, true, 2)
#define CG_INSTANCES_GROUP8(X) X(128, 1, true, 3) X(256, 1, true, 3) X(256, 2, true, 3)
#define CG_INSTANCE_GROUPS 9
#define CG_ALL_INSTANCES(X) \
  CG_INSTANCES_GROUP0(X) CG_INSTANCES_GROUP1(X) CG_INSTANCES_GROUP2(X) CG_INSTANCES_GROUP3(X) CG_INSTANCES_GROUP4(X) CG_INSTANCES_GROUP5(X) \
  CG_INSTANCES_GROUP6(X) CG_INSTANCES_GROUP7(X) CG_INSTANCES_GROUP8(X)

#define CG_KERNEL_SIGNATURE(BN, CGN, KM, CV) \
  __global__ void gemm_epilogue_kernel<BN, CGN, KM, CV>(const __grid_constant__ CUtensorMap, const __grid_constant__ CUtensorMap, \
                                                         const __grid_constant__ CUtensorMap, const __grid_constant__ CUtensorMap, \
                                                         const KernelParams);
