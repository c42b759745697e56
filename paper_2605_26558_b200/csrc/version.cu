#include "common.cuh"

extern "C" const char* cass_version(void) { return "cass-b200 0.1 (sm_100a)"; }
