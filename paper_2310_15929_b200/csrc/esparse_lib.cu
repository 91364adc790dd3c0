// Single translation unit of libesparse.so (the device status word is shared by all kernels).
#include "prune_kernels.cu"
#include "spgemm_kernels.cu"
#include "esparse_api.cu"
#include "spgemm_static.cu"
