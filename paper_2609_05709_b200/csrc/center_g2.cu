// Per-centre kernel instantiations for l_max in [9, 10].
#define SOAP_GROUP 2
#define SOAP_L_LIST X(9) X(10)
#include "center_inst.inc"
