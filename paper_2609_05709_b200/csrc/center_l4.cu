// Per-centre kernel instantiations for l_max = 4.
#define SOAP_L 4
#include "center_inst.inc"
