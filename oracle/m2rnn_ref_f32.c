/*
 * fp32 build of the oracle's loops (m2rnn_ref.c, textually the same code with `double` read as
 * `float` and the libm calls as their float forms), for one use: the all-cores CPU leg that the
 * bench times beside the GPU.  TEST INFRASTRUCTURE ONLY, like the file it includes.  It is not the
 * parity reference (that is the fp64 build) and nothing compares the GPU with it.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#define double float
#define tanh tanhf
#define exp expf
#define log1p log1pf
#define sqrt sqrtf

#include "m2rnn_ref.c"
