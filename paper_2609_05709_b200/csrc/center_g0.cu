// Per-centre kernel instantiations for l_max in [0, 1, 2, 3, 4, 5].
#define SOAP_GROUP 0
#define SOAP_L_LIST X(0) X(1) X(2) X(3) X(4) X(5)
#include "center_inst.inc"
