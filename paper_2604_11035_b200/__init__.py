"""B200-native ISD step (introspective strided decoding): C-ABI CUDA library + thin binding."""
from .binding import (Isd, IsdError, IsdBatchState, IsdConfig, IsdStepArgs, IsdVerifyOut,
                      alloc_verify_out, isd_verify_static, load, LIB_PATH, EXPORTS)
from . import workloads


def isd_for_workload(w, st, **kw):
    """Context configured for a `workloads.Workload` and the state `workloads.make_state` built."""
    args = dict(batch=w.batch, stride=w.stride, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                vocab=w.vocab, max_pages_per_slot=st["page_table"].shape[1], num_pages=st["num_pages"],
                logits_dtype=w.logits_dtype, q_mode=w.q_mode, propose_mode=w.propose_mode, seed=w.seed,
                top_k=w.top_k, top_p=w.top_p)
    args.update(kw)
    return Isd(**args)
