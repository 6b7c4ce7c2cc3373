// Per-centre kernel instantiations for l_max = 2.
#define SOAP_L 2
#include "center_inst.inc"
