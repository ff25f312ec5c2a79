// Typed form of an elementwise program: the instruction list after the broadcast step and the
// Fig. 5 typing rules have been applied to concrete input descriptors (host side).
#pragma once
#include "common.h"

namespace relay {

constexpr int kMaxValues = RELAY_MAX_INPUTS + RELAY_MAX_INSTR;

struct TypedProgram {
    int n_in = 0, n_instr = 0, n_values = 0;
    int rank = 0;
    int64_t shape[RELAY_MAX_RANK] = {0};                       // common broadcast shape
    int64_t in_shape[RELAY_MAX_INPUTS][RELAY_MAX_RANK] = {{0}}; // inputs right-aligned to `rank`
    int32_t dtype[kMaxValues] = {0};                            // base type of every value
    relay_instr_t instr[RELAY_MAX_INSTR];
    int64_t total = 1;                                          // elements of the broadcast shape
};

// null -> rank/type of each input -> instruction typing (dtype) -> broadcast (shape)
relay_status_t type_program(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                            TypedProgram *out);

}  // namespace relay
