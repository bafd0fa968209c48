// Host-side pieces of the KSA library shared by its entry-point files (internal):
// argument validation, the sequence layout of Eq. 1 and the tile schedule of Eq. 3.
#pragma once
#include <vector>

#include "../../include/ksa.h"
#include "ksa_common.h"

// A run of consecutive query tiles of one sequence that the host entry point uploads, computes
// and downloads as one pipeline stage.  All row numbers are per sequence except aug0 / aug1.
struct RowChunk {
    int32_t seq;
    int32_t text0, text1;             // packed text-stream rows to pack (text1 includes the zero padding of the last chunk)
    int32_t summ0, summ1, summq1;     // summary-stream rows to pack [summ0, summ1), summary query rows [summ0, summq1)
    int64_t aug0, aug1;               // global augmented rows [aug0, aug1) of q / k / v / out that belong to the chunk
    int64_t work_off, work_cnt;       // its items in HostSchedule::work
};

struct HostSchedule {
    std::vector<int32_t> key;         // lengths and parameters this schedule was built for
    std::vector<ksa::SeqInfo> seqs;
    std::vector<ksa::WorkItem> work;       // sorted, longest first (within each row chunk, if chunked)
    std::vector<RowChunk> chunks;          // empty unless built with row chunks
    int64_t total_aug = 0, text_rows = 0, summ_rows = 0;
    int32_t max_text_pad = 0, max_summ_pad = 0, max_n_summ = 0;
};

struct WorkspaceLayout { size_t qt, kt, vt, ks, vs, total; };

// KSA_OK or the KSA_ERR_* code describing what is wrong with p.
int validate(const ksa_params* p);
int validate_strides(const ksa_params* p);
// True if the text kernel can read its tiles straight from the caller's tensors (nothing is packed).
bool direct_ok(const ksa_params* p);
// Fills seqs and the stream totals of hs from p (p must have passed validate).
void build_layout(const ksa_params* p, HostSchedule& hs);
// Fills hs.work (longest first) from p and the layout already in hs.
// target_chunks > 0 additionally splits the query tiles into about that many row chunks (in
// sequence order) and orders the work list chunk by chunk.
void build_schedule(const ksa_params* p, HostSchedule& hs, int target_chunks = 0);
// Offsets of the packed streams inside the workspace, and its total size.
WorkspaceLayout workspace_layout(const ksa_params* p, const HostSchedule& hs);

// Access to the context for the other entry-point files (the struct itself lives in ksa_api.cu).
int32_t* ksa_ctx_status_word(ksa_ctx* ctx);                 // device status word
int ksa_ctx_num_sms(const ksa_ctx* ctx);
void ksa_ctx_add_launches(ksa_ctx* ctx, int n);
int ksa_ctx_cuda_fail(ksa_ctx* ctx, int cuda_error);        // records the error, returns KSA_ERR_CUDA
bool* ksa_ctx_decode_ready(ksa_ctx* ctx);                   // the decode kernels' shared-memory opt-in was done on this context's device
