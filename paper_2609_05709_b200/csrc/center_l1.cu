// Per-centre kernel instantiations for l_max = 1.
#define SOAP_L 1
#include "center_inst.inc"
