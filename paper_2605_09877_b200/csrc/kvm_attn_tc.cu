// Placeholder while the tcgen05 kernel is brought up: routes to the scalar-core kernel.
#include "kvm_internal.h"
namespace kvm {
int launch_attn_tc(State* st, const AttnArgs& a, cudaStream_t s) { return launch_attn_simt(st, a, s); }
}
