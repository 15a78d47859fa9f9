// Persistent cluster kernel for EF21+ (Algorithm 3), whole-block steps: instantiations and their lookup.
#define PK_BODY_FILE "persistent_body.inc"
#define PK_KERNEL_NAME persistent_plus_kernel
#define PK_LOOKUP_NAME pk_lookup_plus
#define PK_PLUS 1
#define PK_EF 0
#define PK_FLOOR 0
#include "persistent_method.inc"
