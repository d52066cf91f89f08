"""Trace replay behind the policy ablations: marshals a conversation trace into fl_cache_replay, which drives the
library's dependency tree and cache swapper query by query with the HBM pool reduced to a block budget, and reports
reuse, adapter cold starts, swap volume and the share of invalid KV nodes for the full policy, the three ablations of
the paper's Section 6 (no cost model, no LoRA reward, no usage dependencies) and the static LoRA/KV partition of
Section 2.2.  Nothing of the procedure runs in Python."""
from . import binding as fl

VARIANTS = ("full", "wos", "wol", "wom", "static")
_CODE = {"full": fl.FL_REPLAY_FULL, "wos": fl.FL_REPLAY_WOS, "wol": fl.FL_REPLAY_WOL, "wom": fl.FL_REPLAY_WOM,
         "static": fl.FL_REPLAY_STATIC}


class CapacityError(Exception):
    pass


def replay(events, n_lora, variant, capacity, **kw):
    try:
        return fl.fl_cache_replay(events, n_lora, _CODE[variant], capacity, **kw)
    except fl.FlError as e:
        if e.code == fl.FL_ENOMEM:
            raise CapacityError("the running query does not fit") from e
        raise


def summary(m):
    inv = m["invalid_samples"]
    return dict(hit_rate=m["hit_blocks"] / max(1, m["asked_blocks"]), lora_cold=m["lora_cold"],
                swapped_in=m["swapped_in"], swapped_out=m["swapped_out"],
                invalid_kv=sum(inv) / len(inv) if inv else 0.0)
