// Kernel variant 1 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 1
#include "sg_variant.inc"
