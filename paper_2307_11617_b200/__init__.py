"""R-FAST activation engine for one B200: CUDA library (csrc/) plus its ctypes binding."""

from .binding import (Engine, RFastError, rfast_checkpoint_load, rfast_checkpoint_save, rfast_diagnostics, rfast_append_schedule, rfast_compile_append_check, rfast_compile_digest, rfast_compile_host, rfast_create, rfast_destroy,
                      rfast_load_schedule, rfast_ls_gradient_static, rfast_query, rfast_read_packet, rfast_read_state, rfast_reset, rfast_run, rfast_seek, rfast_set_option, rfast_snapshot, rfast_snapshot_wait,
                      rfast_sync, rfast_version, rfast_write_packet, rfast_write_state)
from . import binding

__all__ = ["Engine", "RFastError", "binding", "rfast_checkpoint_load", "rfast_checkpoint_save", "rfast_diagnostics", "rfast_append_schedule", "rfast_compile_append_check", "rfast_compile_digest", "rfast_compile_host", "rfast_create", "rfast_destroy",
           "rfast_load_schedule", "rfast_ls_gradient_static", "rfast_query", "rfast_read_packet", "rfast_read_state", "rfast_reset", "rfast_run", "rfast_seek", "rfast_set_option", "rfast_snapshot", "rfast_snapshot_wait",
           "rfast_sync", "rfast_version", "rfast_write_packet", "rfast_write_state"]
