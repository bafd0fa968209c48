// Host-side pieces of the KSA library shared by its entry-point files (internal):
// argument validation, the sequence layout of Eq. 1 and the tile schedule of Eq. 3.
#pragma once
#include <vector>

#include "../../include/ksa.h"
#include "ksa_common.h"

struct HostSchedule {
    std::vector<int32_t> key;         // lengths and parameters this schedule was built for
    std::vector<ksa::SeqInfo> seqs;
    std::vector<ksa::WorkItem> work;       // sorted, longest first
    int64_t total_aug = 0, text_rows = 0, summ_rows = 0;
    int32_t max_text_pad = 0, max_summ_pad = 0, max_n_summ = 0;
};

struct WorkspaceLayout { size_t qt, kt, vt, ks, vs, total; };

// KSA_OK or the KSA_ERR_* code describing what is wrong with p.
int validate(const ksa_params* p);
int validate_strides(const ksa_params* p);
// Fills seqs and the stream totals of hs from p (p must have passed validate).
void build_layout(const ksa_params* p, HostSchedule& hs);
// Fills hs.work (longest first) from p and the layout already in hs.
void build_schedule(const ksa_params* p, HostSchedule& hs);
// Offsets of the packed streams inside the workspace, and its total size.
WorkspaceLayout workspace_layout(const ksa_params* p, const HostSchedule& hs);
