"""Developer diagnostics (nothing here is on the product path): measurements that the kernels' design rests on."""
