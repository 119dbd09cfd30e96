// Kernel variant 8 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 8
#include "sg_variant.inc"
