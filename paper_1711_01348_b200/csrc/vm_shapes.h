// The vector shapes (TA values per thread along the lane variable x UB along the element variable)
// the interpreter kernel is built for; each is compiled into an object file of its own.
#pragma once
#define TAD_VM_SHAPES(M) M(1, 1) M(2, 1) M(4, 1) M(8, 1) M(16, 1) M(1, 4) M(1, 8) M(2, 8) M(1, 16) M(4, 8)
