// Host-side scheduler of video parallel speculative decoding (Section 5.2): which draft and verification work a
// decoding round launches, and what the verdict of the round does to the output and to the next round.  No device
// code: the caller launches hippo_draft_attention / hippo_verify_attention / hippo_accept (and its models) on two
// streams as the plan says, reads the accepted count back, and commits it here.
//
//   optimistic round  (the previous batch was accepted in full): the target verifies the current batch while the
//                     draft model already produces the next gamma tokens; a rejection drops them.
//   conservative round (after a rejection): the draft model produces x_1; the target verifies x_1 while the draft
//                     model produces x_2..x_gamma; a rejected x_1 aborts the drafting.
#include <math.h>

#include "common.cuh"

using namespace hippo;

static bool vpsd_state_ok(const hippo_vpsd_state_t *s) {
    return s && s->struct_size == sizeof(hippo_vpsd_state_t) && s->gamma >= 1 &&
           (s->mode == HIPPO_VPSD_OPTIMISTIC || s->mode == HIPPO_VPSD_CONSERVATIVE) && s->batch >= 0 &&
           (s->mode == HIPPO_VPSD_CONSERVATIVE || s->batch >= 1);
}

extern "C" int32_t hippo_vpsd_prefill_buffer(double prefill_target, double prefill_draft, double t_draft) {
    if (!(t_draft > 0.0) || !(prefill_target > prefill_draft)) return 0;
    const double n = floor((prefill_target - prefill_draft) / t_draft + 1e-9);
    return n > 2147483647.0 ? 2147483647 : (int32_t)n;
}

extern "C" int32_t hippo_vpsd_init(hippo_vpsd_state_t *state, int32_t gamma, int32_t buffered_tokens) {
    if (!state) return fail(HIPPO_ERR_INVALID_ARG, "hippo_vpsd_init: null state");
    if (gamma < 1 || buffered_tokens < 0) return fail(HIPPO_ERR_INVALID_ARG, "hippo_vpsd_init: gamma %d, buffered %d", gamma, buffered_tokens);
    state->struct_size = sizeof(hippo_vpsd_state_t);
    state->gamma = gamma;
    state->mode = buffered_tokens > 0 ? HIPPO_VPSD_OPTIMISTIC : HIPPO_VPSD_CONSERVATIVE;
    state->batch = buffered_tokens;
    state->rounds = 0;
    state->tokens_emitted = 0;
    state->tokens_drafted = buffered_tokens;
    state->tokens_discarded = 0;
    return HIPPO_OK;
}

extern "C" int32_t hippo_vpsd_plan(const hippo_vpsd_state_t *state, hippo_vpsd_round_t *round) {
    if (!vpsd_state_ok(state) || !round) return fail(HIPPO_ERR_INVALID_ARG, "hippo_vpsd_plan: bad state or null round");
    round->mode = state->mode;
    if (state->mode == HIPPO_VPSD_OPTIMISTIC) {
        round->draft_before = 0;
        round->verify_tokens = state->batch;
        round->draft_during = state->gamma;
        round->abort_on_reject = 0;
    } else {
        round->draft_before = 1;
        round->verify_tokens = 1;
        round->draft_during = state->gamma - 1;
        round->abort_on_reject = 1;
    }
    return HIPPO_OK;
}

extern "C" int32_t hippo_vpsd_commit(hippo_vpsd_state_t *state, const hippo_vpsd_round_t *round, int32_t n_accepted,
                                     int32_t drafted_during, hippo_vpsd_outcome_t *outcome) {
    if (!vpsd_state_ok(state) || !round || !outcome) return fail(HIPPO_ERR_INVALID_ARG, "hippo_vpsd_commit: bad state or null argument");
    if (round->mode != state->mode || n_accepted < 0 || n_accepted > round->verify_tokens || drafted_during < 0 ||
        drafted_during > round->draft_during)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_vpsd_commit: round does not belong to this state, or counts out of range");
    const bool all = n_accepted == round->verify_tokens;
    if (all && drafted_during != round->draft_during)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_vpsd_commit: drafting may stop early only after a rejection");
    outcome->accepted = n_accepted;
    if (round->mode == HIPPO_VPSD_OPTIMISTIC) {
        // all accepted: the batch is emitted and the tokens drafted meanwhile are next; else n + the replacement
        outcome->emitted = all ? n_accepted : n_accepted + 1;
        outcome->target_token = all ? 0 : 1;
        outcome->keep_drafted = all ? drafted_during : 0;
    } else if (!all) {
        outcome->emitted = 1;            // the replacement of x_1
        outcome->target_token = 1;
        outcome->keep_drafted = 0;
    } else if (round->draft_during == 0) {
        outcome->emitted = 2;            // gamma = 1: x_1 and the target's bonus token, nothing is left to verify
        outcome->target_token = 1;
        outcome->keep_drafted = 0;
    } else {
        outcome->emitted = 1;            // x_1; x_2..x_gamma go to standard verification
        outcome->target_token = 0;
        outcome->keep_drafted = drafted_during;
    }
    outcome->next_mode = outcome->keep_drafted > 0 ? HIPPO_VPSD_OPTIMISTIC : HIPPO_VPSD_CONSERVATIVE;
    state->mode = outcome->next_mode;
    state->batch = outcome->keep_drafted;
    state->rounds += 1;
    state->tokens_emitted += outcome->emitted;
    state->tokens_drafted += round->draft_before + drafted_during;
    state->tokens_discarded += (round->verify_tokens - n_accepted) + (drafted_during - outcome->keep_drafted);
    return HIPPO_OK;
}

extern "C" double hippo_vpsd_round_time(const hippo_vpsd_round_t *round, int32_t n_accepted, double t_draft, double t_target) {
    if (!round) return -1.0;
    if (round->mode == HIPPO_VPSD_OPTIMISTIC) return fmax(t_target, round->draft_during * t_draft);
    // conservative: x_1, then verification beside the rest of the batch; a rejected x_1 ends the round at the verdict
    if (n_accepted < round->verify_tokens) return round->draft_before * t_draft + t_target;
    return round->draft_before * t_draft + fmax(t_target, round->draft_during * t_draft);
}

extern "C" double hippo_vpsd_serial_round_time(int32_t gamma, double t_draft, double t_target) {
    return gamma * t_draft + t_target;
}
