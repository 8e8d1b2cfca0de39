"""Test and benchmark harness around the library: a random-initialised decoder whose
projections, RoPE, FFN and LM head are plain torch and whose attention, consensus and commit
go through the C ABI.  Not part of the library's path."""
