/*
 * admmq_testing.h -- hooks for tests of the library's failure handling and accuracy.  Not part of the solver's
 * contract: nothing here is needed to quantize a layer, and the paper has no counterpart.
 */
#ifndef ADMMQ_TESTING_H_
#define ADMMQ_TESTING_H_

#include "admmq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Every device-side wait of the tensor-core product kernel (on a shared-memory barrier that a copy or a
 * tensor-core operation completes) is bounded: when the bound runs out the kernel records
 * ADMMQ_ERR_TIMEOUT in the device status word, stops issuing work, waits for what it has in flight,
 * frees its tensor memory and returns, and the context stays usable.
 * This call sets that bound for the context, in SM clock cycles (wait_limit_cycles >= 1000; the default is
 * 2e9, about a second), and, with hold_loads != 0, makes the kernel's producer warp issue no loads at
 * all, so that the first wait of every CTA runs out with nothing in flight: the safe way to see the
 * time-out path execute.  hold_loads = 0 and the default bound restore normal operation.  Host-side
 * only; takes effect from the next launch.  Returns ADMMQ_ERR_INVALID_ARG for a NULL context or a bound
 * below 1000 cycles. */
admmq_status admmq_test_set_wait(admmq_ctx* ctx, long long wait_limit_cycles, int hold_loads);

/* admmq_w_update with the result left in the form the solver itself works with: d_Z_out [d_out][d_in] fp32
 * receives W^(t+1) - W_hat' (scaled coordinates), i.e. the correction of Eq. 7 without the weight-sized term
 * W_hat' that admmq_w_update adds before it rounds to fp32.  For accuracy tests at the scale of a grid step. */
admmq_status admmq_test_w_update_correction(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                                            const unsigned char* d_codes, const float* d_scale,
                                            const float* d_zero, const float* d_V, double rho, float* d_Z_out);

/* The same correction evaluated as the later iterations do it (admmq_quant_cfg.wupdate_series): the series
 * c (I + E + E^2 + ...) R with `terms` = 0, 1 or 2 terms of E kept, on the fixed operand mu I - H~, whatever ||E|| is
 * at this penalty.  For a test that compares it with the route through the factorisation on both sides of the
 * penalties where the solver would switch to it.  ADMMQ_ERR_INVALID_ARG for any other `terms`. */
admmq_status admmq_test_w_update_series(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                                        const unsigned char* d_codes, const float* d_scale,
                                        const float* d_zero, const float* d_V, double rho, int terms,
                                        float* d_Z_out);

#ifdef __cplusplus
}
#endif
#endif /* ADMMQ_TESTING_H_ */
