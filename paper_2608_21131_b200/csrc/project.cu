// placeholder translation unit: packed projection kernels are added below
#include "internal.h"
