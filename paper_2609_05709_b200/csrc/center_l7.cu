// Per-centre kernel instantiations for l_max = 7.
#define SOAP_L 7
#include "center_inst.inc"
