// Kernel variant 7 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 7
#include "sg_variant.inc"
