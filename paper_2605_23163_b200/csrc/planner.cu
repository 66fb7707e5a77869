// Section-aligned block planner (host code only): which positions of the output template form which
// block.  Section s, with E_s editable positions, is cut into ceil(E_s / d) blocks filled from the
// left; a block ends right after its last editable position, the last block of a section at the
// section's end; a section without editable positions is one block that needs no decoding.
#include "fdd_internal.h"

extern "C" fdd_status fdd_plan_blocks(const uint8_t* editable, const int32_t* section_end, int n_sections,
                                      int length, int d, int32_t* block_begin, int32_t* block_end,
                                      int32_t* block_section, int capacity, int* n_blocks) {
    CallRange range("fdd_plan_blocks");
    if (n_blocks) *n_blocks = 0;
    if (!editable || !section_end || !block_begin || !block_end || !block_section || !n_blocks) return FDD_ERR_INVALID_ARG;
    if (n_sections < 1 || length < 0 || d < 1 || capacity < 0) return FDD_ERR_INVALID_ARG;
    int prev = 0;
    for (int s = 0; s < n_sections; ++s) {
        if (section_end[s] < prev) return FDD_ERR_INVALID_ARG;
        prev = section_end[s];
    }
    if (prev != length) return FDD_ERR_INVALID_ARG;
    int n = 0;
    int begin_s = 0;
    for (int s = 0; s < n_sections; ++s) {
        const int end_s = section_end[s];
        int n_values = 0;
        for (int i = begin_s; i < end_s; ++i) n_values += editable[i] ? 1 : 0;
        if (n_values == 0) {
            if (end_s > begin_s) {
                if (n >= capacity) return FDD_ERR_CAPACITY;
                block_begin[n] = begin_s; block_end[n] = end_s; block_section[n] = s; ++n;
            }
        } else {
            int b = begin_s, seen = 0, in_block = 0;
            for (int i = begin_s; i < end_s; ++i) {
                if (!editable[i]) continue;
                ++seen; ++in_block;
                if (in_block == d && seen < n_values) {          // a full block that is not the section's last
                    if (n >= capacity) return FDD_ERR_CAPACITY;
                    block_begin[n] = b; block_end[n] = i + 1; block_section[n] = s; ++n;
                    b = i + 1; in_block = 0;
                }
            }
            if (n >= capacity) return FDD_ERR_CAPACITY;
            block_begin[n] = b; block_end[n] = end_s; block_section[n] = s; ++n;
        }
        begin_s = end_s;
    }
    *n_blocks = n;
    return FDD_OK;
}
