// The whole library as one translation unit (one device status word, no device linking).
#include "api.cu"
#include "quantize.cu"
#include "layernorm_compare.cu"
#include "softmax.cu"
#include "gemm.cu"
#include "attention_fused.cu"
#include "attention.cu"
