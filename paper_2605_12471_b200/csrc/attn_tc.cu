// Tensor-core (tcgen05 / TMEM / TMA) prefix + chunk attention for bf16 caches.
#include "kvfold_internal.h"

namespace kvf {

bool attn_tc_supported(int dtype, int d, int G) { (void)dtype; (void)d; (void)G; return false; }
int attn_tc_ctas(int n, int G, int Hkv, int splits) { return ((n * G + 127) / 128) * Hkv * splits; }
cudaError_t launch_attn_tc(const AttnArgs &, const TcMaps &, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace kvf
