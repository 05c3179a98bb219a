"""B200-native per-token PPO-for-RLHF hot path (arXiv 2403.17031): thin Python binding over the
C-ABI CUDA library. Importing the package does not load the library; the first call does and
fails loudly if it is missing (there is no CPU or PyTorch fallback)."""
from .binding import (PPOParams, PPOStepIO, LMHeadStepIO, lmhead_step, lmhead_step_host, step, step_host, default_params, gae, kl_rewards, last_device_status, lib, lmhead_logprob_entropy,
                      lmhead_workspace_bytes, logprob_entropy, loss_from_logprob, loss_from_logprob_static, loss_fwd_bwd, new_workspace,
                      set_option, truncate_and_score, version, whiten, workspace_bytes, PPOError, LOSS_NAMES,
                      logprob_bwd, pairwise_loss, dpo_loss, lmhead_bwd, sample_logprob_entropy, logprob_entropy_pair, rollout_curves)

__all__ = ["PPOParams", "PPOStepIO", "LMHeadStepIO", "lmhead_step", "lmhead_step_host", "step", "step_host", "default_params", "gae", "kl_rewards", "last_device_status", "lib",
           "lmhead_logprob_entropy", "lmhead_workspace_bytes", "logprob_entropy", "loss_from_logprob", "loss_from_logprob_static",
           "loss_fwd_bwd", "new_workspace", "set_option", "truncate_and_score", "version", "whiten",
           "workspace_bytes", "PPOError", "LOSS_NAMES", "logprob_bwd", "pairwise_loss", "dpo_loss", "lmhead_bwd", "sample_logprob_entropy", "logprob_entropy_pair", "rollout_curves"]
