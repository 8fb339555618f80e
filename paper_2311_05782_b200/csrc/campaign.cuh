// Host-visible interface of the campaign's per-trial evaluation kernels.
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/mpgemmfi.h"

namespace mpg {

struct CampaignParams {
    int dtype, M, N, K;
    int detect_mode, n_trials;
    const void *A;
    const void *Bt;
    const float *C;                  // clean, unchecked product
    const mpgemmfi_site *sites;
    mpgemmfi_trial_record *records;
    // schedule (scratch): counters[0..2] = number of A / B / single-element trials, then the lists
    uint32_t *counters;
    uint32_t *list_a;
    uint32_t *list_b;
    uint32_t *list_e;
};

// bytes of schedule scratch for n_trials (256-byte header + three index lists), multiple of 256
size_t campaign_schedule_bytes(int n_trials);

// point the schedule members of p into a scratch block of campaign_schedule_bytes(p.n_trials) bytes
void campaign_bind_schedule(CampaignParams &p, void *scratch);

// Most trials a call may carry when the schedule lives in the library's built-in scratch.
constexpr int CAMPAIGN_STATIC_MAX_TRIALS = 65536;

// Device address and size of the built-in schedule scratch of the current device. The first call
// on a device resolves the address; nothing is allocated.
cudaError_t campaign_static_schedule(void **ptr, size_t *bytes);

// schedule + evaluate every trial; the clean product must already be queued on `stream`
cudaError_t launch_campaign_trials(const CampaignParams &p, int num_sms, cudaStream_t stream);

// zero *out and reduce the records into it
cudaError_t launch_campaign_summary(const mpgemmfi_trial_record *records, int n_trials, mpgemmfi_summary *out,
                                    int num_sms, cudaStream_t stream);

}  // namespace mpg
