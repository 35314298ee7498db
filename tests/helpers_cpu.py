"""CPU-only helpers shared by the multi-process tests (no CUDA import)."""
import dataclasses

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import synth

# packed rows with masked prompt rows, 4 prompts x 3 rollouts, small enough for fp64 on a CPU
DP_WORKLOAD = dataclasses.replace(synth.small_variant("14b-long", prompts=4, samples=3, live_rows=300),
                                  d=64, V=512)


def oracle_step(batch):
    npy = lambda t: t.detach().cpu().numpy()
    Hd = orc.bf16_bits_to_f64(synth.bf16_bits(batch["H"]))
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(batch["W"]))
    ref = orc.loss_fwd(Hd, Wd, npy(batch["targets"]), npy(batch["mask"]), npy(batch["seq_id"]),
                       npy(batch["group_id"]), npy(batch["reward"]), npy(batch["logp_inf"]),
                       batch["S"], batch["P"], batch["beta_v"], batch["beta_loss"], batch["loss_scale"])
    ref["dH"], ref["dW"] = orc.loss_bwd(Hd, Wd, npy(batch["targets"]), npy(batch["mask"]), npy(batch["seq_id"]),
                                        ref["coef"])
    return ref
